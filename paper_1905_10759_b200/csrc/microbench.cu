// Register-only arithmetic loops that measure the rates the integer-pipe and fp32-pipe rooflines are built on:
// 32-bit population counts per second (the XOR/POPC formulation of Eq. 7 needs one per output and K-word)
// and fp32 additions per second (the sign-select formulation of the dense x packed product needs one per
// output and K-element).  Nothing is read from memory inside the loops; every thread keeps eight independent
// dependency chains so that the issue rate of the unit, not its latency, is what is timed.
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int kChains = 8;
constexpr int kBenchThreads = 1024;

// kind 0: POPC (with the XOR that feeds it), 1: FADD, 2: FFMA
template <int KIND>
__global__ void __launch_bounds__(kBenchThreads)
alu_rate_kernel(int iters, uint32_t seed, uint32_t* __restrict__ sink) {
  const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
  if (KIND == 0) {
    uint32_t a[kChains];
#pragma unroll
    for (int i = 0; i < kChains; i++) a[i] = seed * (t + 1u) + 0x9E3779B9u * i;
    const uint32_t k = seed | 1u;
    for (int it = 0; it < iters; it++) {
#pragma unroll
      for (int i = 0; i < kChains; i++) a[i] = __popc(a[i] ^ (k + i * 0x01010101u));
    }
    uint32_t r = 0;
#pragma unroll
    for (int i = 0; i < kChains; i++) r += a[i];
    if (r == 0xFFFFFFFFu) sink[t] = r;         // never true (every a[i] <= 32): keeps the chains alive without a store
  } else {
    float a[kChains];
#pragma unroll
    for (int i = 0; i < kChains; i++) a[i] = static_cast<float>(t & 255u) + i;
    const float c = __uint_as_float(0x3F800000u | (seed & 0xFFu));   // in [1, 1.00003]
    for (int it = 0; it < iters; it++) {
#pragma unroll
      for (int i = 0; i < kChains; i++) a[i] = KIND == 1 ? a[i] + c : fmaf(a[i], c, c);
    }
    float r = 0.0f;
#pragma unroll
    for (int i = 0; i < kChains; i++) r += a[i];
    if (r == -1.0f) sink[t] = __float_as_uint(r);   // never true: every chain stays positive
  }
}

}  // namespace

// blocks x 1024 threads x iters x 8 operations; *ops receives that product.
cudaError_t launch_alu_rate(int kind, int blocks, int iters, uint32_t* sink, int64_t* ops, cudaStream_t stream) {
  if (blocks <= 0 || iters <= 0) return cudaErrorInvalidValue;
  if (ops) *ops = static_cast<int64_t>(blocks) * kBenchThreads * iters * kChains;
  switch (kind) {
    case 0: alu_rate_kernel<0><<<blocks, kBenchThreads, 0, stream>>>(iters, 0x2545F491u, sink); break;
    case 1: alu_rate_kernel<1><<<blocks, kBenchThreads, 0, stream>>>(iters, 0x2545F491u, sink); break;
    case 2: alu_rate_kernel<2><<<blocks, kBenchThreads, 0, stream>>>(iters, 0x2545F491u, sink); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace hbmm
