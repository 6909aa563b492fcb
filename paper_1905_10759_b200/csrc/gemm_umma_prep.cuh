// Pieces of the tcgen05 HBMM kernel that other translation units need: the argument block, the
// shared-memory stage layout, and the routine that expands the weight operand into that layout (the
// packed convolution front end runs it in a few extra CTAs of its own launch, so the expansion costs
// no launch of its own).
#pragma once
#include <cuda_bf16.h>
#include <cstdint>
#include "kernels.h"
#include "umma_common.cuh"

namespace hbmm {
namespace umma_prep {

using namespace umma;
using Args = UmmaArgs;

constexpr int WPS = 4;            // K-words per stage
constexpr int STAGES = 3;

__device__ __forceinline__ float load_scale(const void* s, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(s) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(s) + idx);
}
// Four sign bits (in bits 0..3 or 4..7 of `v`, selected by the multiplier) -> four e4m3 bytes:
// the multiply copies bit i to bit 8*i+7, the sign position of byte i; 0xB8 = -1.0, 0x38 = +1.0.
__device__ __forceinline__ uint32_t signs_lo(uint32_t v) { return (((v & 0x0Fu) * 0x10204080u) & 0x80808080u) ^ 0xB8B8B8B8u; }
__device__ __forceinline__ uint32_t signs_hi(uint32_t v) { return (((v & 0xF0u) * 0x01020408u) & 0x80808080u) ^ 0xB8B8B8B8u; }

// Four packed K-words of one tile row -> 4 x 32 e4m3 bytes (pieces 0..7 of the row).
__device__ __forceinline__ void expand_words(unsigned char* tile, int row, const uint4& w4) {
  const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
  for (int q = 0; q < 4; q++) {
    const uint32_t y0 = w[q] & 0xFF, y1 = (w[q] >> 8) & 0xFF, y2 = (w[q] >> 16) & 0xFF, y3 = w[q] >> 24;
    *reinterpret_cast<uint4*>(swz(tile, row, 2 * q)) = make_uint4(signs_lo(y0), signs_hi(y0), signs_lo(y1), signs_hi(y1));      // K bytes 0..15
    *reinterpret_cast<uint4*>(swz(tile, row, 2 * q + 1)) = make_uint4(signs_lo(y2), signs_hi(y2), signs_lo(y3), signs_hi(y3));  // K bytes 16..31
  }
}

// fp32 scale -> three bf16 pieces with a = a1 + a2 + a3 up to 2^-26 |a| (each remainder is exact in fp32).
__device__ __forceinline__ void split3(float a, uint32_t& h1, uint32_t& h2, uint32_t& h3) {
  const __nv_bfloat16 b1 = __float2bfloat16_rn(a);
  const float r1 = a - __bfloat162float(b1);
  const __nv_bfloat16 b2 = __float2bfloat16_rn(r1);
  const float r2 = r1 - __bfloat162float(b2);
  const __nv_bfloat16 b3 = __float2bfloat16_rn(r2);
  h1 = __bfloat16_as_ushort(b1); h2 = __bfloat16_as_ushort(b2); h3 = __bfloat16_as_ushort(b3);
}
// One row of the scale operands of a segment: eight bf16 (K columns 0..7; columns 8..15 are a piece of
// zeros next to it).  Row of A': (a1, a1, a2, a2, a1, a3, 0, 0); row of B': (w1, w2, w1, w2, w3, w1, 0, 0):
// their dot product is a1w1 + a1w2 + a2w1 + a2w2 + a1w3 + a3w1.
template <bool IS_B>
__device__ __forceinline__ uint4 scale_row(float v) {
  uint32_t h1, h2, h3;
  split3(v, h1, h2, h3);
  if (IS_B) return make_uint4(h1 | (h2 << 16), h1 | (h2 << 16), h3 | (h1 << 16), 0u);
  return make_uint4(h1 | (h1 << 16), h2 | (h2 << 16), h1 | (h3 << 16), 0u);
}

template <int TN>
struct Smem {
  static constexpr int A_STAGE = TM * 128;                // sign bytes of the A tile: 128 rows x 4 words x 32 bytes
  static constexpr int SA_STAGE = TM * 128;               // scale pieces: per word slot 16 bytes of pieces + 16 of zeros
  static constexpr int B_SIGNS = TN * 128;
  static constexpr int B_STAGE = 2 * B_SIGNS;             // signs then scale pieces: one bulk copy
  static constexpr int OFF_A = 0;
  static constexpr int OFF_SA = OFF_A + STAGES * A_STAGE;
  static constexpr int OFF_B = OFF_SA + STAGES * SA_STAGE;
  static constexpr int OFF_BAR = OFF_B + STAGES * B_STAGE;
  static constexpr int NBUF = 512 / (2 * TN);                           // TMEM buffers: D and S side by side
  // barriers: full[STAGES], empty[STAGES], tfull[NBUF], tempty[NBUF], drain
  static constexpr int NBAR = 2 * STAGES + 2 * NBUF + 1;
  static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;                   // tmem base, abort flag
  static constexpr int USED = OFF_MISC + 16;
  // at least 120 KB so that two CTAs never share an SM (each one allocates all of TMEM)
  static constexpr int BYTES = USED > 120 * 1024 ? USED : 120 * 1024;
};

// Expands one (stage, column tile) of the weight operand into the stage layout the main kernel reads:
// the e4m3 sign bytes followed by the bf16 scale pieces, exactly as they sit in shared memory.
// p = row of the tile (0 .. TN-1), one thread per row.
template <int TN>
__device__ __forceinline__ void prepare_w_task(const Args& g, unsigned char* __restrict__ out, int64_t st, int64_t tile_n, int p) {
  using S = Smem<TN>;
  const int64_t n_stages = (g.n_words + WPS - 1) / WPS;
  const int64_t n = tile_n * TN + p;
  const bool in = n < g.N;
  const int64_t kw = st * WPS;
  uint4 w = make_uint4(0, 0, 0, 0);
  if (in && kw < g.ldw_w) w = __ldg(reinterpret_cast<const uint4*>(g.w_bits + n * g.ldw_w + kw));
  unsigned char* base = out + (tile_n * n_stages + st) * S::B_STAGE;
  expand_words(base, p, w);
#pragma unroll
  for (int q = 0; q < WPS; q++) {
    float f = 0.0f;
    const int64_t grp = ((kw + q) / g.seg_words) / g.rw;
    if (in && kw + q < g.n_words && grp < g.Gw) f = load_scale(g.w_scales, g.w_bf16, n * g.ldw_s + grp);
    *reinterpret_cast<uint4*>(swz(base + S::B_SIGNS, p, 2 * q)) = scale_row<true>(f);
    *reinterpret_cast<uint4*>(swz(base + S::B_SIGNS, p, 2 * q + 1)) = make_uint4(0, 0, 0, 0);
  }
}

}  // namespace umma_prep
}  // namespace hbmm
