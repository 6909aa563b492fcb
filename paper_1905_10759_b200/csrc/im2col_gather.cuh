// Inner loop of the packed convolution front end for a full 32-channel chunk whose filter size is
// known at compile time (shared by the two tiled front-end kernels).
#pragma once
#include <cstdint>

namespace hbmm {

// One K-word: element e of word WORD is chunk-local k = 32 * WORD + e = (c, i, j) with
// c = k / (KH * KW), read from a staged fp32 tile in shared memory at byte address
// base + c * cs_bytes + i * pitch_bytes + 4 * j (one address per (c, i), the tap column as an
// immediate).  Each element costs one shared-memory load, one add of +0 (so that -0 counts as +0 and
// the sign bit alone decides Sign(x): x >= 0 <=> bit clear), one funnel shift that collects the sign
// bit, and one add of |x|.  Returns the packed word (bit e = 1 <=> x >= 0) and the sum of |x|.
// MASKED: the tile has no zero halo; bit j of `mask` says that filter column j, bit 8 + i that filter
// row i lies inside the image for this pixel, and taps outside are taken as 0 without being loaded.
template <int KH, int KW, int WORD, bool MASKED>
__device__ __forceinline__ void gather_word_static(uint32_t base, uint32_t cs_bytes, uint32_t pitch_bytes, uint32_t mask,
                                                   uint32_t& word, float& sum) {
  constexpr int T = KH * KW;
  uint32_t pat = 0;
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int e = 0; e < 32; e += 4) {
    float v[4];
#pragma unroll
    for (int u = 0; u < 4; u++) {
      const int k = 32 * WORD + e + u, c = k / T, t = k % T, i = t / KW, j = t % KW;
      const uint32_t row = base + c * cs_bytes + i * pitch_bytes;
      float x = 0.0f;
      if (!MASKED || ((mask >> j) & (mask >> (8 + i)) & 1u))
        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(x) : "r"(row + 4 * j));   // the constant folds into the load
      v[u] = x + 0.0f;
      pat = __funnelshift_l(__float_as_uint(v[u]), pat, 1);     // pat = pat << 1 | sign bit
    }
    s0 += fabsf(v[0]); s1 += fabsf(v[1]); s2 += fabsf(v[2]); s3 += fabsf(v[3]);
  }
  word = ~__brev(pat);                                            // element e at bit e
  sum = (s0 + s1) + (s2 + s3);
}

// The same with the sum of |x| kept per scale group of 32 / SUB elements (groups shorter than a word, SUB = 2 .. 16 of
// them): sums[i] covers elements i * beta .. (i + 1) * beta - 1 of the word.
template <int KH, int KW, int WORD, bool MASKED, int SUB>
__device__ __forceinline__ void gather_word_static_sub(uint32_t base, uint32_t cs_bytes, uint32_t pitch_bytes, uint32_t mask,
                                                       uint32_t& word, float (&sums)[SUB]) {
  constexpr int T = KH * KW, BETA = 32 / SUB;
  uint32_t pat = 0;
  float acc[SUB][2];            // two partial sums per group where a group has that many elements
#pragma unroll
  for (int i = 0; i < SUB; i++) { acc[i][0] = 0.f; acc[i][1] = 0.f; }
#pragma unroll
  for (int e = 0; e < 32; e++) {
    const int k = 32 * WORD + e, c = k / T, t = k % T, i = t / KW, j = t % KW;
    const uint32_t row = base + c * cs_bytes + i * pitch_bytes;
    float x = 0.0f;
    if (!MASKED || ((mask >> j) & (mask >> (8 + i)) & 1u))
      asm volatile("ld.shared.f32 %0, [%1];" : "=f"(x) : "r"(row + 4 * j));
    const float v = x + 0.0f;
    pat = __funnelshift_l(__float_as_uint(v), pat, 1);
    acc[e / BETA][e & 1] += fabsf(v);
  }
  word = ~__brev(pat);
#pragma unroll
  for (int i = 0; i < SUB; i++) sums[i] = acc[i][0] + acc[i][1];
}

template <int KH, int KW, bool MASKED, int SUB, int WORD = 0>
__device__ __forceinline__ void gather_word_dispatch_sub(int w, uint32_t base, uint32_t cs_bytes, uint32_t pitch_bytes, uint32_t mask,
                                                         uint32_t& word, float (&sums)[SUB]) {
  if constexpr (WORD < KH * KW) {
    if (w == WORD) gather_word_static_sub<KH, KW, WORD, MASKED, SUB>(base, cs_bytes, pitch_bytes, mask, word, sums);
    else gather_word_dispatch_sub<KH, KW, MASKED, SUB, WORD + 1>(w, base, cs_bytes, pitch_bytes, mask, word, sums);
  }
}

// w (warp-uniform) selects the word of the chunk: KH * KW words per 32 channels.
template <int KH, int KW, bool MASKED = false, int WORD = 0>
__device__ __forceinline__ void gather_word_dispatch(int w, uint32_t base, uint32_t cs_bytes, uint32_t pitch_bytes, uint32_t mask,
                                                     uint32_t& word, float& sum) {
  if constexpr (WORD < KH * KW) {
    if (w == WORD) gather_word_static<KH, KW, WORD, MASKED>(base, cs_bytes, pitch_bytes, mask, word, sum);
    else gather_word_dispatch<KH, KW, MASKED, WORD + 1>(w, base, cs_bytes, pitch_bytes, mask, word, sum);
  }
}

}  // namespace hbmm
