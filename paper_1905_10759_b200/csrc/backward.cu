// Gradient through the Hadamard binarization X~ = delta (.) Sign(X) (Section 3.1.3): Eq. 6 with the
// straight-through estimator of Eq. 5,
//   gx[i] = (1/n_g) s_i sum_{j in group(i)} gy[j] s_j  +  delta_g gy[i] [|x_i| <= 1],
// s = Sign(x) (+1 for x >= 0), delta_g the mean |x| of the group, n_g its length.
// A pure stream: 8 bytes read and 4 written per element, HBM bound.
//
// Fast kernel (unpadded fp32 rows, K a multiple of beta, beta a power of two up to 128, K a multiple of 4):
// the tensor is one contiguous run whose groups never straddle a row; a lane owns four consecutive
// elements (one 16-byte load of x, one of gy, one 16-byte store), a group is one lane (beta <= 4) or
// beta / 4 neighbouring lanes, whose two sums (|x| and gy s) are xor-shuffle trees.  The first term's
// sign factor is applied by XOR-ing the sign bit of x into the group sum.
// General kernel (any beta >= 1, any K, padded rows): one thread per (row, group), two passes over the group.
#include <cstdint>
#include <cuda_runtime.h>
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float signed_like(float mag, float x) {      // mag * Sign(x), Sign(+-0) = +1
  return __uint_as_float(__float_as_uint(mag) ^ (__float_as_uint(x + 0.0f) & 0x80000000u));
}

template <int BETA>
__global__ void __launch_bounds__(kThreads)
binarize_backward_stream(const float4* __restrict__ x, const float4* __restrict__ gy, float4* __restrict__ gx, int64_t n_vec) {
  constexpr int LANES = BETA > 4 ? BETA / 4 : 1;          // lanes per group
  constexpr float inv = 1.0f / static_cast<float>(BETA);
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  // whole warps walk together: the shuffles below need every lane, so the loop bound is rounded up to a warp
  const int64_t n_round = (n_vec + 31) / 32 * 32;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < n_round; i += stride) {
    const bool live = i < n_vec;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f), g = v;
    if (live) { v = __ldg(x + i); g = __ldg(gy + i); }
    const float xv[4] = {v.x, v.y, v.z, v.w}, gv[4] = {g.x, g.y, g.z, g.w};
    float a[4], d[4];                                      // |x| and gy * Sign(x)
#pragma unroll
    for (int e = 0; e < 4; e++) { a[e] = fabsf(xv[e]); d[e] = signed_like(gv[e], xv[e]); }
    float asum[4], dsum[4];                                // group sums as seen by each element
    if (BETA == 1) {
#pragma unroll
      for (int e = 0; e < 4; e++) { asum[e] = a[e]; dsum[e] = d[e]; }
    } else if (BETA == 2) {
      asum[0] = asum[1] = a[0] + a[1]; asum[2] = asum[3] = a[2] + a[3];
      dsum[0] = dsum[1] = d[0] + d[1]; dsum[2] = dsum[3] = d[2] + d[3];
    } else {
      float sa = (a[0] + a[1]) + (a[2] + a[3]), sd = (d[0] + d[1]) + (d[2] + d[3]);
#pragma unroll
      for (int off = 1; off < LANES; off <<= 1) {
        sa += __shfl_xor_sync(0xffffffffu, sa, off);
        sd += __shfl_xor_sync(0xffffffffu, sd, off);
      }
#pragma unroll
      for (int e = 0; e < 4; e++) { asum[e] = sa; dsum[e] = sd; }
    }
    float o[4];
#pragma unroll
    for (int e = 0; e < 4; e++) {
      const float first = signed_like(dsum[e] * inv, xv[e]);                      // (1/n) s_i sum_j gy_j s_j
      const float ste = a[e] <= 1.0f ? (asum[e] * inv) * gv[e] : 0.0f;            // delta_g gy_i [|x_i| <= 1]
      o[e] = first + ste;
    }
    if (live) gx[i] = make_float4(o[0], o[1], o[2], o[3]);
  }
}

__global__ void __launch_bounds__(kThreads)
binarize_backward_general(const float* __restrict__ x, int64_t ldx, const float* __restrict__ gy, int64_t ldg, int64_t rows, int64_t K,
                          int64_t beta, int64_t G, float* __restrict__ gx, int64_t ldo) {
  const int64_t total = rows * G;
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; idx < total;
       idx += static_cast<int64_t>(gridDim.x) * kThreads) {
    const int64_t r = idx / G, g = idx - r * G;
    const int64_t k0 = g * beta, k1 = k0 + beta < K ? k0 + beta : K;
    float sa = 0.0f, sd = 0.0f;
    for (int64_t k = k0; k < k1; k++) {
      const float v = x[r * ldx + k];
      sa += fabsf(v);
      sd += signed_like(gy[r * ldg + k], v);
    }
    const float n = static_cast<float>(k1 - k0);
    const float delta = sa / n, mean_d = sd / n;
    for (int64_t k = k0; k < k1; k++) {
      const float v = x[r * ldx + k];
      const float ste = fabsf(v) <= 1.0f ? delta * gy[r * ldg + k] : 0.0f;
      gx[r * ldo + k] = signed_like(mean_d, v) + ste;
    }
  }
}

template <int BETA>
void launch_stream(unsigned blocks, cudaStream_t stream, const float* x, const float* gy, float* gx, int64_t n_vec) {
  binarize_backward_stream<BETA><<<blocks, kThreads, 0, stream>>>(reinterpret_cast<const float4*>(x), reinterpret_cast<const float4*>(gy),
                                                               reinterpret_cast<float4*>(gx), n_vec);
}

}  // namespace

cudaError_t launch_binarize_backward(const float* x, int64_t ldx, const float* gy, int64_t ldg, int64_t rows, int64_t K, int32_t beta,
                                     float* gx, int64_t ldo, cudaStream_t stream) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t beff = beta >= K ? K : beta;
  const bool aligned = reinterpret_cast<uintptr_t>(x) % 16 == 0 && reinterpret_cast<uintptr_t>(gy) % 16 == 0 &&
                       reinterpret_cast<uintptr_t>(gx) % 16 == 0;
  const bool pow2 = (beff & (beff - 1)) == 0;
  if (aligned && ldx == K && ldg == K && ldo == K && pow2 && beff <= 128 && K % beff == 0 && K % 4 == 0) {
    const int64_t n_vec = rows * K / 4;
    int64_t blocks = (n_vec + kThreads - 1) / kThreads;
    const int64_t cap = static_cast<int64_t>(sms) * 32;
    if (blocks > cap) blocks = cap;
    const unsigned b = static_cast<unsigned>(blocks < 1 ? 1 : blocks);
    switch (beff) {
      case 1: launch_stream<1>(b, stream, x, gy, gx, n_vec); break;
      case 2: launch_stream<2>(b, stream, x, gy, gx, n_vec); break;
      case 4: launch_stream<4>(b, stream, x, gy, gx, n_vec); break;
      case 8: launch_stream<8>(b, stream, x, gy, gx, n_vec); break;
      case 16: launch_stream<16>(b, stream, x, gy, gx, n_vec); break;
      case 32: launch_stream<32>(b, stream, x, gy, gx, n_vec); break;
      case 64: launch_stream<64>(b, stream, x, gy, gx, n_vec); break;
      default: launch_stream<128>(b, stream, x, gy, gx, n_vec); break;
    }
    return cudaGetLastError();
  }
  const int64_t G = (K + beff - 1) / beff;
  int64_t blocks = (rows * G + kThreads - 1) / kThreads;
  const int64_t cap = static_cast<int64_t>(sms) * 32;
  if (blocks > cap) blocks = cap;
  binarize_backward_general<<<static_cast<unsigned>(blocks < 1 ? 1 : blocks), kThreads, 0, stream>>>(x, ldx, gy, ldg, rows, K, beff, G, gx, ldo);
  return cudaGetLastError();
}

}  // namespace hbmm
