// Convolution front end: implicit im2col gather from an NCHW activation tensor.
//   A[m,k] = x[b, c, yo*sh + i - ph, xo*sw + j - pw]  (0 outside the image),
//   m = (b, yo, xo), k = (c, i, j) with c slowest -- the column order of Reshape(W, (filters, -1)).
// The packed variant binarizes each gathered row along k on the fly (Eq. 1-4 applied to the
// im2col row, the grouping Eq. 7 is stated for) and never writes the fp32 matrix; the dense
// variant writes bf16 rows for the HBWN mode.
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int kThreads = 128;

__device__ __forceinline__ float load_x(const void* p, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(p) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(p) + idx);
}
__device__ __forceinline__ void store_scale(void* scales, int bf16, int64_t idx, float v) {
  if (bf16) reinterpret_cast<__nv_bfloat16*>(scales)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(scales)[idx] = v;
}

// One thread per output row m: consecutive lanes hold consecutive xo, so every tap is a
// coalesced read along the image row.  Words and scales are produced in k order.
__global__ void __launch_bounds__(kThreads)
im2col_quantize_kernel(const void* __restrict__ x, int x_bf16, const ConvGeom g, int64_t M, int64_t K,
                       int64_t beta, int64_t G, uint32_t* __restrict__ bits, int64_t ld_words,
                       void* __restrict__ scales, int64_t ld_scales, int scale_bf16) {
  const int64_t m = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
  if (m >= M) return;
  const int xo = static_cast<int>(m % g.Wo);
  const int yo = static_cast<int>((m / g.Wo) % g.Ho);
  const int64_t b = m / (static_cast<int64_t>(g.Wo) * g.Ho);
  uint32_t* brow = bits + m * ld_words;
  uint32_t word = 0;
  float wsum[4] = {0.f, 0.f, 0.f, 0.f};
  float gsum = 0.0f;
  int64_t k = 0, grp = 0, in_grp = 0;
  for (int c = 0; c < g.C; c++) {
    const int64_t plane = (b * g.C + c) * static_cast<int64_t>(g.H) * g.W;
    for (int i = 0; i < g.kh; i++) {
      const int y = yo * g.sh + i - g.ph;
      const bool yin = y >= 0 && y < g.H;
      for (int j = 0; j < g.kw; j++) {
        const int xx = xo * g.sw + j - g.pw;
        float v = 0.0f;
        if (yin && xx >= 0 && xx < g.W) v = load_x(x, x_bf16, plane + static_cast<int64_t>(y) * g.W + xx);
        word |= (v >= 0.0f ? 1u : 0u) << (k & 31);
        wsum[k & 3] += fabsf(v);
        k++;
        in_grp++;
        if ((k & 31) == 0) { brow[(k >> 5) - 1] = word; word = 0; }
        if ((k & 31) == 0 || in_grp == beta) {
          gsum += (wsum[0] + wsum[1]) + (wsum[2] + wsum[3]);
          wsum[0] = wsum[1] = wsum[2] = wsum[3] = 0.0f;
        }
        if (in_grp == beta) {
          store_scale(scales, scale_bf16, m * ld_scales + grp, gsum / static_cast<float>(beta));
          grp++; in_grp = 0; gsum = 0.0f;
        }
      }
    }
  }
  if (k & 31) brow[k >> 5] = word;
  for (int64_t w = (k + 31) >> 5; w < ld_words; w++) brow[w] = 0u;
  if (in_grp > 0) {
    gsum += (wsum[0] + wsum[1]) + (wsum[2] + wsum[3]);
    store_scale(scales, scale_bf16, m * ld_scales + grp, gsum / static_cast<float>(in_grp));
    grp++;
  }
  for (int64_t z = grp; z < ld_scales; z++) store_scale(scales, scale_bf16, m * ld_scales + z, 0.0f);
}

// One thread per (row m, scale group g): the 32 lanes of a warp hold 32 consecutive m for the
// same group, so every tap is a coalesced read along an image row and each thread emits whole
// words plus the group's scale.  Used when beta < K; blocks are 32 rows x 8 groups.
__global__ void __launch_bounds__(256)
im2col_quantize_groups_kernel(const void* __restrict__ x, int x_bf16, const ConvGeom g, int64_t M, int64_t K,
                              int beta_words, int64_t G, int64_t n_words, uint32_t* __restrict__ bits,
                              int64_t ld_words, void* __restrict__ scales, int64_t ld_scales, int scale_bf16) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t m = static_cast<int64_t>(blockIdx.x) * 32 + lane;
  const int64_t grp = static_cast<int64_t>(blockIdx.y) * 8 + warp;
  if (m >= M || grp >= G) return;
  const int xo = static_cast<int>(m % g.Wo);
  const int yo = static_cast<int>((m / g.Wo) % g.Ho);
  const int64_t b = m / (static_cast<int64_t>(g.Wo) * g.Ho);
  const int taps = g.kh * g.kw;
  const int64_t HW = static_cast<int64_t>(g.H) * g.W;
  const int y0 = yo * g.sh - g.ph, x0 = xo * g.sw - g.pw;
  const int64_t k_begin = grp * beta_words * 32;
  int64_t k_end = k_begin + static_cast<int64_t>(beta_words) * 32;
  if (k_end > K) k_end = K;
  int c = static_cast<int>(k_begin / taps);
  int r = static_cast<int>(k_begin - static_cast<int64_t>(c) * taps);
  int i = r / g.kw, j = r - i * g.kw;
  const int64_t base = b * g.C * HW;
  uint32_t* brow = bits + m * ld_words;
  float gsum = 0.0f;
  for (int64_t kw0 = k_begin; kw0 < k_end; kw0 += 32) {
    uint32_t word = 0;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    const int nk = (k_end - kw0 < 32) ? static_cast<int>(k_end - kw0) : 32;
#pragma unroll 4
    for (int e = 0; e < nk; e++) {
      const int y = y0 + i, xx = x0 + j;
      float v = 0.0f;
      if (y >= 0 && y < g.H && xx >= 0 && xx < g.W) v = load_x(x, x_bf16, base + c * HW + static_cast<int64_t>(y) * g.W + xx);
      word |= (v >= 0.0f ? 1u : 0u) << e;
      const float av = fabsf(v);
      if ((e & 3) == 0) s0 += av; else if ((e & 3) == 1) s1 += av; else if ((e & 3) == 2) s2 += av; else s3 += av;
      if (++j == g.kw) { j = 0; if (++i == g.kh) { i = 0; c++; } }
    }
    brow[kw0 >> 5] = word;
    gsum += (s0 + s1) + (s2 + s3);
  }
  store_scale(scales, scale_bf16, m * ld_scales + grp, gsum / static_cast<float>(k_end - k_begin));
  if (grp == G - 1) {
    for (int64_t w = n_words; w < ld_words; w++) brow[w] = 0u;
    for (int64_t z = G; z < ld_scales; z++) store_scale(scales, scale_bf16, m * ld_scales + z, 0.0f);
  }
}

__global__ void __launch_bounds__(256)
im2col_bf16_kernel(const void* __restrict__ x, int x_bf16, const ConvGeom g, int64_t M, int64_t K,
                   __nv_bfloat16* __restrict__ out, int64_t ld) {
  const int64_t total = M * ld;
  const int taps = g.kh * g.kw;
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; idx < total;
       idx += static_cast<int64_t>(gridDim.x) * 256) {
    const int64_t m = idx / ld;
    const int k = static_cast<int>(idx - m * ld);
    float v = 0.0f;
    if (k < K) {
      const int c = k / taps, r = k - c * taps, i = r / g.kw, j = r - i * g.kw;
      const int xo = static_cast<int>(m % g.Wo);
      const int yo = static_cast<int>((m / g.Wo) % g.Ho);
      const int64_t b = m / (static_cast<int64_t>(g.Wo) * g.Ho);
      const int y = yo * g.sh + i - g.ph, xx = xo * g.sw + j - g.pw;
      if (y >= 0 && y < g.H && xx >= 0 && xx < g.W)
        v = load_x(x, x_bf16, ((b * g.C + c) * static_cast<int64_t>(g.H) + y) * g.W + xx);
    }
    out[idx] = __float2bfloat16_rn(v);
  }
}

}  // namespace

cudaError_t launch_im2col_quantize(const void* x, int x_bf16, const ConvGeom& g, int32_t beta,
                                   uint32_t* bits, int64_t ld_words, void* scales, int64_t ld_scales,
                                   int scale_bf16, cudaStream_t stream) {
  const int64_t M = static_cast<int64_t>(g.B) * g.Ho * g.Wo, K = static_cast<int64_t>(g.C) * g.kh * g.kw;
  const int64_t beta_eff = beta >= K ? K : beta;
  const int64_t G = num_groups(K, beta);
  if (beta < K && beta % 32 == 0) {
    dim3 grid(static_cast<unsigned>((M + 31) / 32), static_cast<unsigned>((G + 7) / 8));
    im2col_quantize_groups_kernel<<<grid, 256, 0, stream>>>(x, x_bf16, g, M, K, beta / 32, G, (K + 31) / 32, bits,
                                                             ld_words, scales, ld_scales, scale_bf16);
    return cudaGetLastError();
  }
  const int64_t blocks = (M + kThreads - 1) / kThreads;
  im2col_quantize_kernel<<<static_cast<unsigned>(blocks), kThreads, 0, stream>>>(
      x, x_bf16, g, M, K, beta_eff, G, bits, ld_words, scales, ld_scales, scale_bf16);
  return cudaGetLastError();
}

cudaError_t launch_im2col_bf16(const void* x, int x_bf16, const ConvGeom& g, void* out, int64_t ld,
                               cudaStream_t stream) {
  const int64_t M = static_cast<int64_t>(g.B) * g.Ho * g.Wo, K = static_cast<int64_t>(g.C) * g.kh * g.kw;
  int64_t blocks = (M * ld + 255) / 256;
  if (blocks > 148 * 64) blocks = 148 * 64;
  im2col_bf16_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(x, x_bf16, g, M, K,
                                                                         reinterpret_cast<__nv_bfloat16*>(out), ld);
  return cudaGetLastError();
}

}  // namespace hbmm
