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

// Loads only (no reduction): the EPT elements starting at column k0 of a row; columns >= K read as 0 with
// the `in` mask cleared, so that several loads can be issued before the first one is used.
template <bool BF16>
__device__ __forceinline__ void load_elems(const void* x, int64_t row_off, int64_t k0, int64_t K, bool vec_ok,
                                           float (&v)[In<BF16>::EPT], uint32_t& in_mask) {
  using L = In<BF16>;
  constexpr int EPT = L::EPT;
  if (vec_ok && k0 + EPT <= K) {
    const typename L::Vec* p = reinterpret_cast<const typename L::Vec*>(
        reinterpret_cast<const char*>(x) + (row_off + k0) * (BF16 ? 2 : 4));
    L::unpack(__ldg(p), v);
    in_mask = (1u << EPT) - 1u;
  } else {
    in_mask = 0;
#pragma unroll
    for (int e = 0; e < EPT; e++) {
      const bool in = k0 + e < K;
      v[e] = in ? L::scalar(x, row_off + k0 + e) : 0.0f;
      in_mask |= (in ? 1u : 0u) << e;
    }
  }
}
template <int EPT>
__device__ __forceinline__ void signs_and_abs_sum(float (&v)[EPT], uint32_t in_mask, uint32_t& sbits, float& asum) {
  sbits = 0;
#pragma unroll
  for (int e = 0; e < EPT; e++) sbits |= (v[e] >= 0.0f ? 1u : 0u) << e;
  sbits &= in_mask;
#pragma unroll
  for (int e = 0; e < EPT; e++) v[e] = fabsf(v[e]);
#pragma unroll
  for (int w = 1; w < EPT; w <<= 1)
#pragma unroll
    for (int e = 0; e < EPT; e += 2 * w) v[e] += v[e + w];
  asum = v[0];
}

// Fast path: beta/32 is a power of two no larger than the words one warp covers.
// One warp item = WPW consecutive words of one row; a warp takes kUnroll items per trip and issues all
// their loads before it touches the first value (the kernel is a pure stream: what limits it is the
// number of bytes in flight).
constexpr int kUnroll = 4;
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
  const int bw_shift = __ffs(beta_words) - 1;                 // beta_words is a power of two on this path
  // (row, chunk) of the next item are carried along instead of divided out of the item number
  const int64_t step_rows = nwarps / chunks, step_chunks = nwarps - step_rows * chunks;
  int64_t nrow = warp0 / chunks, nchunk = warp0 - nrow * chunks;
  for (int64_t it0 = warp0; it0 < items; it0 += nwarps * kUnroll) {
    float v[kUnroll][EPT];
    uint32_t in_mask[kUnroll];
    int64_t row[kUnroll], chunk[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; u++) {
      const int64_t it = it0 + u * nwarps;
      row[u] = nrow;
      chunk[u] = nchunk;
      nrow += step_rows;
      nchunk += step_chunks;
      if (nchunk >= chunks) { nchunk -= chunks; nrow++; }
      in_mask[u] = 0;
      if (it < items) load_elems<BF16>(x, row[u] * ldx, (chunk[u] * WPW * 32) + lane * EPT, K, vec_ok, v[u], in_mask[u]);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; u++) {
      if (it0 + u * nwarps >= items) break;
      uint32_t sb;
      float s;
      signs_and_abs_sum<EPT>(v[u], in_mask[u], sb, s);
      uint32_t word = sb << (EPT * (lane % LPW));
#pragma unroll
      for (int off = 1; off < LPW; off <<= 1) {
        word |= __shfl_xor_sync(0xffffffffu, word, off);
        s += __shfl_xor_sync(0xffffffffu, s, off);
      }
      for (int off = LPW; off < LPW * beta_words; off <<= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
      const int64_t wi = chunk[u] * WPW + lane / LPW;
      if ((lane % LPW) == 0 && wi < ld_words) bits[row[u] * ld_words + wi] = word;
      if ((lane % (LPW * beta_words)) == 0) {
        const int64_t g = wi >> bw_shift;
        if (g < G) {
          const int64_t cnt = (K - g * beta < beta) ? (K - g * beta) : beta;
          store_scale(scales, scale_bf16, row[u] * ld_scales + g, s / static_cast<float>(cnt));
          if (g == G - 1)
            for (int64_t z = G; z < ld_scales; z++) store_scale(scales, scale_bf16, row[u] * ld_scales + z, 0.0f);
        }
      }
    }
  }
}

// Stream path: rows without padding (ldx == K), K a multiple of 32 and of beta, beta a power of two from
// 2 to 512.  The tensor is then one contiguous run of elements whose words and groups never straddle a
// row, and the kernel is written for instructions per element: a lane owns 16 consecutive elements
// (64 bytes of fp32, 32 of bf16), so a packed word is two lanes and a beta = 32 group sum one shuffle.
// Sign(x) = +1 for x >= 0 including -0: adding +0.0 turns -0 into +0, after which the IEEE sign bit
// decides; it is shifted into the lane's 16-bit sign field with one funnel shift per element.
template <bool BF16, int BETA>
__global__ void __launch_bounds__(kThreads)
quantize_stream(const void* __restrict__ x, int64_t total_words, uint32_t n_words, uint32_t* __restrict__ bits, int64_t ld_words,
                void* __restrict__ scales, int64_t ld_scales, int scale_bf16, uint32_t G) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = (static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = (static_cast<int64_t>(gridDim.x) * kThreads) >> 5;
  const int64_t items = (total_words + 15) / 16;                  // 16 words = 512 elements per warp and trip
  for (int64_t it = warp0; it < items; it += nwarps) {
    const int64_t fw = it * 16 + (lane >> 1);                      // this lane's word, counted over the whole tensor
    const bool live = fw < total_words;
    float v[16];
    if (live) {
      if (BF16) {
        const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned short*>(x) + fw * 32 + (lane & 1) * 16);
        const uint4 a = __ldg(p), b = __ldg(p + 1);
        In<true>::unpack(a, v);
        In<true>::unpack(b, v + 8);
      } else {
        const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(x) + fw * 32 + (lane & 1) * 16);
        const float4 a = __ldg(p), b = __ldg(p + 1), c = __ldg(p + 2), d = __ldg(p + 3);
        In<false>::unpack(a, v); In<false>::unpack(b, v + 4); In<false>::unpack(c, v + 8); In<false>::unpack(d, v + 12);
      }
    } else {
#pragma unroll
      for (int e = 0; e < 16; e++) v[e] = 0.0f;
    }
    uint32_t neg = 0;                                             // bit e set <=> element e is negative
#pragma unroll
    for (int e = 15; e >= 0; e--) neg = __funnelshift_l(__float_as_uint(v[e] + 0.0f), neg, 1);
    const uint32_t sb = ~neg & 0xFFFFu;
    const uint32_t other = __shfl_xor_sync(0xffffffffu, sb, 1);
    const uint32_t row = static_cast<uint32_t>(fw / n_words), wi = static_cast<uint32_t>(fw - static_cast<int64_t>(row) * n_words);
    if (live && (lane & 1) == 0) {
      uint32_t* brow = bits + static_cast<int64_t>(row) * ld_words;
      brow[wi] = sb | (other << 16);
      if (wi == 0) {                                              // the row's zero padding
        for (int64_t z = n_words; z < ld_words; z++) brow[z] = 0u;
        for (int64_t z = G; z < ld_scales; z++) store_scale(scales, scale_bf16, static_cast<int64_t>(row) * ld_scales + z, 0.0f);
      }
    }
    // pairwise sums of |x|: after the level of width w, v[e] (e a multiple of 2w) holds the sum of 2w elements
#pragma unroll
    for (int e = 0; e < 16; e++) v[e] = fabsf(v[e]);
    constexpr int IN_LANE = BETA < 16 ? BETA : 16;
#pragma unroll
    for (int w = 1; w < IN_LANE; w <<= 1)
#pragma unroll
      for (int e = 0; e < 16; e += 2 * w) v[e] += v[e + w];
    constexpr float inv = 1.0f / static_cast<float>(BETA);        // beta is a power of two: the same as dividing
    if constexpr (BETA <= 16) {
      constexpr int GPL = 16 / BETA;                              // groups per lane, consecutive in the scale row
      const int64_t g0 = static_cast<int64_t>(row) * ld_scales + (wi * 32u + (lane & 1) * 16u) / BETA;
      if (live) {
#pragma unroll
        for (int i = 0; i < GPL; i++) store_scale(scales, scale_bf16, g0 + i, v[i * BETA] * inv);
      }
    } else {
      constexpr int LANES = BETA / 16;                            // lanes per group
      float sum = v[0];
#pragma unroll
      for (int off = 1; off < LANES; off <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
      if (live && (lane % LANES) == 0)
        store_scale(scales, scale_bf16, static_cast<int64_t>(row) * ld_scales + wi / (BETA / 32), sum * inv);
    }
  }
}

template <bool BF16>
bool launch_stream(int beta, unsigned blocks, cudaStream_t stream, const void* x, int64_t total_words, uint32_t n_words, uint32_t* bits,
                   int64_t ld_words, void* scales, int64_t ld_scales, int scale_bf16, uint32_t G) {
#define HBMM_QS(B) case B: quantize_stream<BF16, B><<<blocks, kThreads, 0, stream>>>(x, total_words, n_words, bits, ld_words, scales, ld_scales, scale_bf16, G); return true;
  switch (beta) {
    HBMM_QS(2) HBMM_QS(4) HBMM_QS(8) HBMM_QS(16) HBMM_QS(32) HBMM_QS(64) HBMM_QS(128) HBMM_QS(256) HBMM_QS(512)
    default: return false;
  }
#undef HBMM_QS
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
  const int64_t step_rows = nwarps / chunks, step_chunks = nwarps - step_rows * chunks;
  int64_t nrow = warp0 / chunks, nchunk = warp0 - nrow * chunks;
  for (int64_t it = warp0; it < items; it += nwarps) {
    const int64_t row = nrow, chunk = nchunk;
    nrow += step_rows;
    nchunk += step_chunks;
    if (nchunk >= chunks) { nchunk -= chunks; nrow++; }
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
  if (!one_group && vec_ok && ldx == K && K % 32 == 0 && K % beta == 0 && K / 32 < (int64_t{1} << 31) && rows < (int64_t{1} << 31)) {
    const int64_t total_words = rows * (K / 32);
    int64_t blocks = ((total_words + 15) / 16 + (kThreads / 32) - 1) / (kThreads / 32);
    const int64_t cap = static_cast<int64_t>(sms) * 16;
    if (blocks > cap) blocks = cap;
    const bool ok = x_bf16 ? launch_stream<true>(beta, static_cast<unsigned>(blocks), stream, x, total_words, static_cast<uint32_t>(K / 32), bits,
                                                 ld_words, scales, ld_scales, scale_bf16, static_cast<uint32_t>(G))
                           : launch_stream<false>(beta, static_cast<unsigned>(blocks), stream, x, total_words, static_cast<uint32_t>(K / 32), bits,
                                                  ld_words, scales, ld_scales, scale_bf16, static_cast<uint32_t>(G));
    if (ok) return cudaGetLastError();
  }
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
