// Hadamard binarization + bit-packing of a row-major tensor (Section 3, Eq. 1-4; packing Section 4).
//
// HBM-bound streaming kernel: every input element is read once with 16-byte loads that are
// contiguous across a warp, the sign bits and |x| sums of a 32-element word are combined with
// xor-shuffles inside the 8 (fp32) or 4 (bf16) lanes that hold the word, and group sums for
// beta = 64 / 128 (/256 for bf16) continue the same shuffle tree across words.  All sums are
// fp32 pairwise trees, so a scale differs from the exactly rounded mean by at most
// (log2(beta) + 2) * 2^-24 relative.
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int kThreads = 256;

template <bool BF16> struct In;
template <> struct In<false> {
  static constexpr int EPT = 4;  // elements per thread and 16-byte load
  using Vec = float4;
  __device__ static void unpack(const Vec& v, float* o) { o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w; }
  __device__ static float scalar(const void* p, int64_t i) { return __ldg(reinterpret_cast<const float*>(p) + i); }
};
template <> struct In<true> {
  static constexpr int EPT = 8;
  using Vec = uint4;
  __device__ static void unpack(const Vec& v, float* o) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; i++) {  // a bf16 is the upper half of the fp32 with the same value
      o[2 * i] = __uint_as_float(w[i] << 16);
      o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  __device__ static float scalar(const void* p, int64_t i) {
    return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(p) + i)) << 16);
  }
};

__device__ __forceinline__ void store_scale(void* scales, int bf16, int64_t idx, float v) {
  if (bf16) reinterpret_cast<__nv_bfloat16*>(scales)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(scales)[idx] = v;
}

// Loads the EPT elements starting at column k0 of a row; columns >= K read as "absent"
// (value 0, sign bit 0).  Returns the sign nibble/byte and the pairwise sum of |x|.
template <bool BF16>
__device__ __forceinline__ void load_signs_abs(const void* x, int64_t row_off, int64_t k0, int64_t K, bool vec_ok,
                                               uint32_t& sbits, float& asum) {
  using L = In<BF16>;
  constexpr int EPT = L::EPT;
  float v[EPT];
  sbits = 0;
  if (vec_ok && k0 + EPT <= K) {
    const typename L::Vec* p = reinterpret_cast<const typename L::Vec*>(
        reinterpret_cast<const char*>(x) + (row_off + k0) * (BF16 ? 2 : 4));
    L::unpack(__ldg(p), v);
#pragma unroll
    for (int e = 0; e < EPT; e++) sbits |= (v[e] >= 0.0f ? 1u : 0u) << e;
  } else {
#pragma unroll
    for (int e = 0; e < EPT; e++) {
      const bool in = k0 + e < K;
      v[e] = in ? L::scalar(x, row_off + k0 + e) : 0.0f;
      sbits |= ((in && v[e] >= 0.0f) ? 1u : 0u) << e;
    }
  }
#pragma unroll
  for (int e = 0; e < EPT; e++) v[e] = fabsf(v[e]);
#pragma unroll
  for (int w = 1; w < EPT; w <<= 1)
#pragma unroll
    for (int e = 0; e < EPT; e += 2 * w) v[e] += v[e + w];
  asum = v[0];
}

// Fast path: beta/32 is a power of two no larger than the words one warp covers.
// One warp item = WPW consecutive words of one row.
template <bool BF16>
__global__ void __launch_bounds__(kThreads)
quantize_small_beta(const void* __restrict__ x, int64_t rows, int64_t K, int64_t ldx, bool vec_ok,
                    uint32_t* __restrict__ bits, int64_t ld_words, void* __restrict__ scales, int64_t ld_scales,
                    int scale_bf16, int beta_words, int64_t G) {
  constexpr int EPT = In<BF16>::EPT;
  constexpr int LPW = 32 / EPT;  // lanes per word
  constexpr int WPW = EPT;       // words per warp item (32 lanes * EPT elements / 32)
  const int lane = threadIdx.x & 31;
  const int64_t chunks = (ld_words + WPW - 1) / WPW;
  const int64_t items = rows * chunks;
  const int64_t warp0 = (static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = (static_cast<int64_t>(gridDim.x) * kThreads) >> 5;
  const int64_t beta = static_cast<int64_t>(beta_words) * 32;
  for (int64_t it = warp0; it < items; it += nwarps) {
    const int64_t row = it / chunks, chunk = it - row * chunks;
    const int64_t k0 = (chunk * WPW * 32) + lane * EPT;
    uint32_t sb;
    float s;
    load_signs_abs<BF16>(x, row * ldx, k0, K, vec_ok, sb, s);
    uint32_t word = sb << (EPT * (lane % LPW));
#pragma unroll
    for (int off = 1; off < LPW; off <<= 1) {
      word |= __shfl_xor_sync(0xffffffffu, word, off);
      s += __shfl_xor_sync(0xffffffffu, s, off);
    }
    for (int off = LPW; off < LPW * beta_words; off <<= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    const int64_t wi = chunk * WPW + lane / LPW;
    if ((lane % LPW) == 0 && wi < ld_words) bits[row * ld_words + wi] = word;
    if ((lane % (LPW * beta_words)) == 0) {
      const int64_t g = wi / beta_words;
      if (g < G) {
        const int64_t cnt = (K - g * beta < beta) ? (K - g * beta) : beta;
        store_scale(scales, scale_bf16, row * ld_scales + g, s / static_cast<float>(cnt));
        if (g == G - 1)
          for (int64_t z = G; z < ld_scales; z++) store_scale(scales, scale_bf16, row * ld_scales + z, 0.0f);
      }
    }
  }
}

// Sub-word groups (beta = 2, 4, 8 or 16 < K): the paper's own settings (Section 5 uses beta 2 .. 16).
// Same warp item as above (32 lanes x EPT consecutive elements of one row); a group lies inside one
// thread's elements (beta <= EPT) or inside beta / EPT neighbouring lanes, so its sum is a pairwise tree
// in registers followed by at most two shuffle steps.  Scales leave as EPT / beta consecutive values
// per thread, i.e. contiguous across the warp.
template <bool BF16, int BETA>
__global__ void __launch_bounds__(kThreads)
quantize_subword(const void* __restrict__ x, int64_t rows, int64_t K, int64_t ldx, bool vec_ok,
                 uint32_t* __restrict__ bits, int64_t ld_words, void* __restrict__ scales, int64_t ld_scales,
                 int scale_bf16, int64_t G) {
  using L = In<BF16>;
  constexpr int EPT = L::EPT;
  constexpr int LPW = 32 / EPT;
  constexpr int WPW = EPT;
  constexpr int GPT = EPT >= BETA ? EPT / BETA : 1;     // groups per thread
  constexpr int LPG = EPT >= BETA ? 1 : BETA / EPT;     // lanes per group
  const int lane = threadIdx.x & 31;
  const int64_t chunks = (ld_words + WPW - 1) / WPW;
  const int64_t items = rows * chunks;
  const int64_t warp0 = (static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = (static_cast<int64_t>(gridDim.x) * kThreads) >> 5;
  for (int64_t it = warp0; it < items; it += nwarps) {
    const int64_t row = it / chunks, chunk = it - row * chunks;
    const int64_t k0 = (chunk * WPW * 32) + lane * EPT;
    float v[EPT];
    uint32_t sb = 0;
    if (vec_ok && k0 + EPT <= K) {
      const typename L::Vec* p = reinterpret_cast<const typename L::Vec*>(
          reinterpret_cast<const char*>(x) + (row * ldx + k0) * (BF16 ? 2 : 4));
      L::unpack(__ldg(p), v);
#pragma unroll
      for (int e = 0; e < EPT; e++) sb |= (v[e] >= 0.0f ? 1u : 0u) << e;
    } else {
#pragma unroll
      for (int e = 0; e < EPT; e++) {
        const bool in = k0 + e < K;
        v[e] = in ? L::scalar(x, row * ldx + k0 + e) : 0.0f;      // absent columns: value 0, sign bit 0
        sb |= ((in && v[e] >= 0.0f) ? 1u : 0u) << e;
      }
    }
    uint32_t word = sb << (EPT * (lane % LPW));
#pragma unroll
    for (int off = 1; off < LPW; off <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, off);
    const int64_t wi = chunk * WPW + lane / LPW;
    if ((lane % LPW) == 0 && wi < ld_words) bits[row * ld_words + wi] = word;
    // group sums of |x|
#pragma unroll
    for (int e = 0; e < EPT; e++) v[e] = fabsf(v[e]);
    constexpr int SPAN = EPT >= BETA ? BETA : EPT;     // elements of one group inside a thread
#pragma unroll
    for (int w = 1; w < SPAN; w <<= 1)
#pragma unroll
      for (int e = 0; e < EPT; e += 2 * w) v[e] += v[e + w];
#pragma unroll
    for (int off = 1; off < LPG; off <<= 1) v[0] += __shfl_xor_sync(0xffffffffu, v[0], off);
    if ((lane % LPG) == 0) {
#pragma unroll
      for (int i = 0; i < GPT; i++) {
        const int64_t g = k0 / BETA + i;
        if (g < G) {
          const int64_t cnt = (K - g * BETA < BETA) ? (K - g * BETA) : BETA;
          store_scale(scales, scale_bf16, row * ld_scales + g, v[i * SPAN] / static_cast<float>(cnt));
          if (g == G - 1)
            for (int64_t z = G; z < ld_scales; z++) store_scale(scales, scale_bf16, row * ld_scales + z, 0.0f);
        }
      }
    }
  }
}

template <bool BF16>
void launch_subword(int beta, unsigned blocks, cudaStream_t stream, const void* x, int64_t rows, int64_t K, int64_t ldx, bool vec_ok,
                    uint32_t* bits, int64_t ld_words, void* scales, int64_t ld_scales, int scale_bf16, int64_t G) {
  switch (beta) {
    case 2: quantize_subword<BF16, 2><<<blocks, kThreads, 0, stream>>>(x, rows, K, ldx, vec_ok, bits, ld_words, scales, ld_scales, scale_bf16, G); break;
    case 4: quantize_subword<BF16, 4><<<blocks, kThreads, 0, stream>>>(x, rows, K, ldx, vec_ok, bits, ld_words, scales, ld_scales, scale_bf16, G); break;
    case 8: quantize_subword<BF16, 8><<<blocks, kThreads, 0, stream>>>(x, rows, K, ldx, vec_ok, bits, ld_words, scales, ld_scales, scale_bf16, G); break;
    default: quantize_subword<BF16, 16><<<blocks, kThreads, 0, stream>>>(x, rows, K, ldx, vec_ok, bits, ld_words, scales, ld_scales, scale_bf16, G); break;
  }
}

// General path: beta any multiple of 32, or one group per row (beta >= K).  One block per row;
// the per-word |x| sums are kept in shared memory and each group is then summed by one warp
// (lane-strided partial sums followed by a shuffle tree).
template <bool BF16>
__global__ void __launch_bounds__(kThreads)
quantize_any_beta(const void* __restrict__ x, int64_t rows, int64_t K, int64_t ldx, bool vec_ok,
                  uint32_t* __restrict__ bits, int64_t ld_words, void* __restrict__ scales, int64_t ld_scales,
                  int scale_bf16, int64_t beta_words, int64_t beta, int64_t G) {
  extern __shared__ float word_sum[];  // [ld_words]
  constexpr int EPT = In<BF16>::EPT;
  constexpr int LPW = 32 / EPT;
  constexpr int WPW = EPT;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kWarps = kThreads / 32;
  const int64_t chunks = (ld_words + WPW - 1) / WPW;
  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
    for (int64_t chunk = warp; chunk < chunks; chunk += kWarps) {
      const int64_t k0 = (chunk * WPW * 32) + lane * EPT;
      uint32_t sb;
      float s;
      load_signs_abs<BF16>(x, row * ldx, k0, K, vec_ok, sb, s);
      uint32_t word = sb << (EPT * (lane % LPW));
#pragma unroll
      for (int off = 1; off < LPW; off <<= 1) {
        word |= __shfl_xor_sync(0xffffffffu, word, off);
        s += __shfl_xor_sync(0xffffffffu, s, off);
      }
      const int64_t wi = chunk * WPW + lane / LPW;
      if ((lane % LPW) == 0 && wi < ld_words) {
        bits[row * ld_words + wi] = word;
        word_sum[wi] = s;
      }
    }
    __syncthreads();
    for (int64_t g = warp; g < ld_scales; g += kWarps) {
      float s = 0.0f;
      if (g < G) {
        const int64_t w0 = g * beta_words;
        int64_t w1 = w0 + beta_words;
        if (w1 > ld_words) w1 = ld_words;
        for (int64_t w = w0 + lane; w < w1; w += 32) s += word_sum[w];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        const int64_t cnt = (K - g * beta < beta) ? (K - g * beta) : beta;
        s = s / static_cast<float>(cnt);
      }
      if (lane == 0) store_scale(scales, scale_bf16, row * ld_scales + g, s);
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t launch_quantize(const void* x, int x_bf16, int64_t rows, int64_t K, int64_t ldx,
                            uint32_t* bits, int64_t ld_words, void* scales, int64_t ld_scales,
                            int scale_bf16, int32_t beta, cudaStream_t stream) {
  const int64_t esz = x_bf16 ? 2 : 4;
  const bool vec_ok = (reinterpret_cast<uintptr_t>(x) % 16 == 0) && ((ldx * esz) % 16 == 0);
  const int64_t G = num_groups(K, beta);
  const bool one_group = beta >= K;
  const int64_t beta_words = one_group ? ld_words : beta / 32;
  const int wpw = x_bf16 ? 8 : 4;
  const bool pow2 = (beta_words & (beta_words - 1)) == 0;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (!one_group && beta < 32) {
    if (beta != 2 && beta != 4 && beta != 8 && beta != 16) return cudaErrorInvalidValue;
    const int64_t chunks = (ld_words + wpw - 1) / wpw;
    const int64_t items = rows * chunks;
    int64_t blocks = (items + (kThreads / 32) - 1) / (kThreads / 32);
    const int64_t cap = static_cast<int64_t>(sms) * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (x_bf16) launch_subword<true>(beta, static_cast<unsigned>(blocks), stream, x, rows, K, ldx, vec_ok, bits, ld_words, scales, ld_scales, scale_bf16, G);
    else launch_subword<false>(beta, static_cast<unsigned>(blocks), stream, x, rows, K, ldx, vec_ok, bits, ld_words, scales, ld_scales, scale_bf16, G);
    return cudaGetLastError();
  }
  if (!one_group && pow2 && beta_words <= wpw) {
    const int64_t chunks = (ld_words + wpw - 1) / wpw;
    const int64_t items = rows * chunks;
    int64_t blocks = (items + (kThreads / 32) - 1) / (kThreads / 32);
    const int64_t cap = static_cast<int64_t>(sms) * 16;  // grid-stride beyond 8 resident blocks/SM x2
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (x_bf16)
      quantize_small_beta<true><<<static_cast<unsigned>(blocks), kThreads, 0, stream>>>(
          x, rows, K, ldx, vec_ok, bits, ld_words, scales, ld_scales, scale_bf16, static_cast<int>(beta_words), G);
    else
      quantize_small_beta<false><<<static_cast<unsigned>(blocks), kThreads, 0, stream>>>(
          x, rows, K, ldx, vec_ok, bits, ld_words, scales, ld_scales, scale_bf16, static_cast<int>(beta_words), G);
  } else {
    const size_t smem = static_cast<size_t>(ld_words) * sizeof(float);
    if (smem > 48 * 1024) return cudaErrorInvalidValue;  // rows longer than 393216 elements
    int64_t blocks = rows < static_cast<int64_t>(sms) * 8 ? rows : static_cast<int64_t>(sms) * 8;
    const int64_t beta_eff = one_group ? K : beta;
    if (x_bf16)
      quantize_any_beta<true><<<static_cast<unsigned>(blocks), kThreads, smem, stream>>>(
          x, rows, K, ldx, vec_ok, bits, ld_words, scales, ld_scales, scale_bf16, beta_words, beta_eff, G);
    else
      quantize_any_beta<false><<<static_cast<unsigned>(blocks), kThreads, smem, stream>>>(
          x, rows, K, ldx, vec_ok, bits, ld_words, scales, ld_scales, scale_bf16, beta_words, beta_eff, G);
  }
  return cudaGetLastError();
}

}  // namespace hbmm
