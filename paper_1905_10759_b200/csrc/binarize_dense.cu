// Hadamard binarization written out as a dense tensor: X~ = delta (.) Sign(X) (Eq. 2 for weights, Eq. 3-4 for
// activations), delta the mean |x| of each run of beta consecutive row elements, every element of the run
// replaced by +-delta.  With rows = the rows of an activation map (batch x channel x height) and K = its
// width this is Eq. 3 as printed: groups of beta_a neighbours along a map row, before any convolution.
// A pure stream: 4 bytes read and 4 (fp32) or 2 (bf16) written per element, HBM bound.
//
// Fast kernel (unpadded fp32 rows, K a multiple of beta, beta a power of two up to 128, element count a multiple of 4):
// the tensor is one contiguous run whose groups never straddle a row; a lane owns four consecutive elements
// (one 16-byte load, one 16- or 8-byte store) and a group is a run inside one lane or several neighbouring
// lanes whose |x| sums meet in an xor-shuffle tree.
// General kernel (any beta >= 1, any K, padded rows): one thread per (row, group), two passes over the group.
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float with_sign_of(float mag, float x) {      // mag * Sign(x), Sign(+-0) = +1
  return __uint_as_float(__float_as_uint(mag) ^ (__float_as_uint(x + 0.0f) & 0x80000000u));
}

__device__ __forceinline__ void store_run(float* out, int64_t i, const float (&o)[4]) {
  reinterpret_cast<float4*>(out)[i] = make_float4(o[0], o[1], o[2], o[3]);
}
__device__ __forceinline__ uint32_t bf16_pair(float lo, float hi) {
  const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&p);
}
__device__ __forceinline__ void store_run(__nv_bfloat16* out, int64_t i, const float (&o)[4]) {
  reinterpret_cast<uint2*>(out)[i] = make_uint2(bf16_pair(o[0], o[1]), bf16_pair(o[2], o[3]));
}
__device__ __forceinline__ void store1(float* out, int64_t i, float v) { out[i] = v; }
__device__ __forceinline__ void store1(__nv_bfloat16* out, int64_t i, float v) { out[i] = __float2bfloat16_rn(v); }

// E = consecutive elements per lane.  Four, for either output type: a warp's 16-byte loads then cover one
// contiguous 512-byte run.  (Eight per lane, which makes the bf16 store 16 bytes wide too, leaves every load
// instruction touching half of each 32-byte sector and measured 13 % slower.)
template <int BETA, int E, typename OUT>
__global__ void __launch_bounds__(kThreads)
binarize_dense_stream(const float4* __restrict__ x, OUT* __restrict__ out, int64_t n_items) {
  constexpr int LANES = BETA > E ? BETA / E : 1;          // lanes per group
  constexpr int RUN = BETA < E ? BETA : E;                // elements of one group inside a lane
  constexpr float inv = 1.0f / static_cast<float>(BETA);
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  // whole warps walk together: the shuffles below need every lane, so the loop bound is rounded up to a warp
  const int64_t n_round = (n_items + 31) / 32 * 32;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < n_round; i += stride) {
    const bool live = i < n_items;
    float xv[E];
#pragma unroll
    for (int q = 0; q < E / 4; q++) {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (live) v = __ldg(x + i * (E / 4) + q);
      xv[4 * q] = v.x; xv[4 * q + 1] = v.y; xv[4 * q + 2] = v.z; xv[4 * q + 3] = v.w;
    }
    float o[E];
#pragma unroll
    for (int r = 0; r < E / RUN; r++) {                    // the runs of this lane, each inside one group
      float sa = 0.0f;
      if constexpr (RUN == 1) {
        sa = fabsf(xv[r]);
      } else {
        float part[RUN / 2];
#pragma unroll
        for (int e = 0; e < RUN / 2; e++) part[e] = fabsf(xv[r * RUN + 2 * e]) + fabsf(xv[r * RUN + 2 * e + 1]);
#pragma unroll
        for (int w = RUN / 2; w > 1; w >>= 1)
#pragma unroll
          for (int e = 0; e < w / 2; e++) part[e] = part[2 * e] + part[2 * e + 1];
        sa = part[0];
      }
#pragma unroll
      for (int off = 1; off < LANES; off <<= 1) sa += __shfl_xor_sync(0xffffffffu, sa, off);
#pragma unroll
      for (int e = 0; e < RUN; e++) o[r * RUN + e] = with_sign_of(sa * inv, xv[r * RUN + e]);
    }
    if (live) store_run(out, i, o);
  }
}

template <typename OUT>
__global__ void __launch_bounds__(kThreads)
binarize_dense_general(const float* __restrict__ x, int64_t ldx, int64_t rows, int64_t K, int64_t beta, int64_t G,
                       OUT* __restrict__ out, int64_t ldo) {
  const int64_t total = rows * G;
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; idx < total;
       idx += static_cast<int64_t>(gridDim.x) * kThreads) {
    const int64_t r = idx / G, g = idx - r * G;
    const int64_t k0 = g * beta, k1 = k0 + beta < K ? k0 + beta : K;
    float sa = 0.0f;
    for (int64_t k = k0; k < k1; k++) sa += fabsf(x[r * ldx + k]);
    const float delta = sa / static_cast<float>(k1 - k0);
    for (int64_t k = k0; k < k1; k++) store1(out, r * ldo + k, with_sign_of(delta, x[r * ldx + k]));
  }
}

template <typename OUT>
cudaError_t launch_typed(const float* x, int64_t ldx, int64_t rows, int64_t K, int64_t beff, OUT* out, int64_t ldo, int sms,
                         cudaStream_t stream) {
  constexpr int E = 4;                                   // elements per lane
  const bool aligned = reinterpret_cast<uintptr_t>(x) % 16 == 0 && reinterpret_cast<uintptr_t>(out) % 16 == 0;
  const bool pow2 = (beff & (beff - 1)) == 0;
  const int64_t cap = static_cast<int64_t>(sms) * 32;
  if (aligned && ldx == K && ldo == K && pow2 && beff <= 128 && K % beff == 0 && (rows * K) % E == 0) {
    const int64_t n_items = rows * K / E;
    int64_t blocks = (n_items + kThreads - 1) / kThreads;
    if (blocks > cap) blocks = cap;
    const unsigned b = static_cast<unsigned>(blocks < 1 ? 1 : blocks);
    const float4* xv = reinterpret_cast<const float4*>(x);
    switch (beff) {
      case 1: binarize_dense_stream<1, E, OUT><<<b, kThreads, 0, stream>>>(xv, out, n_items); break;
      case 2: binarize_dense_stream<2, E, OUT><<<b, kThreads, 0, stream>>>(xv, out, n_items); break;
      case 4: binarize_dense_stream<4, E, OUT><<<b, kThreads, 0, stream>>>(xv, out, n_items); break;
      case 8: binarize_dense_stream<8, E, OUT><<<b, kThreads, 0, stream>>>(xv, out, n_items); break;
      case 16: binarize_dense_stream<16, E, OUT><<<b, kThreads, 0, stream>>>(xv, out, n_items); break;
      case 32: binarize_dense_stream<32, E, OUT><<<b, kThreads, 0, stream>>>(xv, out, n_items); break;
      case 64: binarize_dense_stream<64, E, OUT><<<b, kThreads, 0, stream>>>(xv, out, n_items); break;
      default: binarize_dense_stream<128, E, OUT><<<b, kThreads, 0, stream>>>(xv, out, n_items); break;
    }
    return cudaGetLastError();
  }
  const int64_t G = (K + beff - 1) / beff;
  int64_t blocks = (rows * G + kThreads - 1) / kThreads;
  if (blocks > cap) blocks = cap;
  binarize_dense_general<OUT><<<static_cast<unsigned>(blocks < 1 ? 1 : blocks), kThreads, 0, stream>>>(x, ldx, rows, K, beff, G, out, ldo);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_binarize_dense(const float* x, int64_t ldx, int64_t rows, int64_t K, int32_t beta, void* out, bool out_bf16,
                                  int64_t ldo, cudaStream_t stream) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t beff = beta >= K ? K : beta;
  if (out_bf16) return launch_typed(x, ldx, rows, K, beff, static_cast<__nv_bfloat16*>(out), ldo, sms, stream);
  return launch_typed(x, ldx, rows, K, beff, static_cast<float*>(out), ldo, sms, stream);
}

}  // namespace hbmm
