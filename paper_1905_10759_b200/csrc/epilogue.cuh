// What a contraction kernel can do with a finished product tile besides storing it as fp32: the chain the
// paper's layer order asks for (Section 5: ... convolution -> activation -> [pooling] -> batch normalisation ->
// binarization of the next block), applied to 32 consecutive columns of one output row at a time while they
// are still in registers.
//   y = act(C)                       (none or max(0, .))
//   z = bn_scale[n] * y + bn_shift[n]   (a batch normalisation folded to inference form; null pointers: 1 and 0)
// and then either z stored dense as fp32 or bf16 ([M, ld]: for a convolution that is NHWC, what the next
// dense-activation convolution reads directly), or the row Hadamard-binarized along n (Eq. 3-4) and only its
// packed form stored (what a following fully connected layer or 1 x 1 convolution reads as its operand).
#pragma once
#include <cuda_bf16.h>
#include <cstdint>
#include "kernels.h"

namespace hbmm {

namespace epi {

__device__ __forceinline__ void store_next_scale(void* s, int bf16, int64_t idx, float v) {
  if (bf16) reinterpret_cast<__nv_bfloat16*>(s)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(s)[idx] = v;
}

// 32 consecutive columns of one row of z (columns n0 .. n0 + 31, `valid` of them inside the output) become one
// packed word (bit e = 1 <=> z[e] >= 0, -0 counting as +0; bits of absent columns 0) and the scales of the
// groups that end inside the chunk (mean |z| over the group's columns inside the output).
// BETA > 32: the chunk's |z| sum is added to `carry`, and the group is closed by its last chunk.
template <int BETA>
__device__ __forceinline__ void emit_next_chunk(const float (&z)[32], int valid, int64_t n0, int64_t N, uint32_t* bits_row, void* scales,
                                                int bf16, int64_t srow, int64_t ld_scales, float& carry) {
  uint32_t neg = 0;
#pragma unroll
  for (int e = 31; e >= 0; e--) neg = __funnelshift_l(__float_as_uint(z[e] + 0.0f), neg, 1);
  const uint32_t vmask = valid >= 32 ? 0xFFFFFFFFu : (valid <= 0 ? 0u : ((1u << valid) - 1u));
  bits_row[n0 >> 5] = ~neg & vmask;
  float a[16];                                            // pairwise tree of |z|, first level formed on the fly
#pragma unroll
  for (int e = 0; e < 16; e++)
    a[e] = (2 * e < valid ? fabsf(z[2 * e]) : 0.0f) + (2 * e + 1 < valid ? fabsf(z[2 * e + 1]) : 0.0f);
  constexpr int SPAN = (BETA < 32 ? BETA : 32) / 2;       // pairs per group inside the chunk
#pragma unroll
  for (int w = 1; w < SPAN; w <<= 1)
#pragma unroll
    for (int e = 0; e < 16; e += 2 * w) a[e] += a[e + w];
  if constexpr (BETA <= 32) {
#pragma unroll
    for (int gi = 0; gi < 32 / BETA; gi++) {
      const int64_t gidx = n0 / BETA + gi;
      const int cnt = valid - gi * BETA < BETA ? valid - gi * BETA : BETA;
      if (gidx < ld_scales) store_next_scale(scales, bf16, srow + gidx, cnt > 0 ? a[gi * SPAN] / static_cast<float>(cnt) : 0.0f);
    }
  } else {
    carry += a[0];
    if ((n0 + 32) % BETA == 0) {
      const int64_t g0 = n0 + 32 - BETA, gidx = g0 / BETA;
      const int64_t cnt = N - g0 < BETA ? N - g0 : BETA;
      if (gidx < ld_scales) store_next_scale(scales, bf16, srow + gidx, cnt > 0 ? carry / static_cast<float>(cnt) : 0.0f);
      carry = 0.0f;
    }
  }
}

// One chunk of a row through the chain.  c[e]: the product at column n0 + e; fs / fh: the 32 affine factors of
// these columns (already 1 / 0 where there is no map).  tile_end: first column past the tile the chunk belongs to
// (the last tile of a row also writes the row's zero padding in packed mode).
__device__ __forceinline__ void finish_chunk(const EpiArgs& ep, float (&c)[32], const float (&fs)[32], const float (&fh)[32],
                                             int64_t m, int64_t n0, int64_t N, bool last_chunk_of_row_tile, int64_t tile_end,
                                             float& carry) {
  float z[32];
#pragma unroll
  for (int e = 0; e < 32; e++) {
    const float y = ep.act == 1 ? fmaxf(c[e], 0.0f) : c[e];
    z[e] = fmaf(y, fs[e], fh[e]);
  }
  const int valid = N - n0 >= 32 ? 32 : static_cast<int>(N - n0 > 0 ? N - n0 : 0);
  if (ep.mode == kEpiDense) {
    if (ep.out_bf16) {
      __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(ep.out) + m * ep.ld_out + n0;
      if (valid == 32 && ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0)) {
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; e++) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(z[j + 2 * e], z[j + 2 * e + 1]);
            w[e] = *reinterpret_cast<const uint32_t*>(&h);
          }
          *reinterpret_cast<uint4*>(dst + j) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      } else {
        for (int e = 0; e < valid; e++) dst[e] = __float2bfloat16_rn(z[e]);
      }
    } else {
      float* dst = reinterpret_cast<float*>(ep.out) + m * ep.ld_out + n0;
      if (valid == 32 && ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0)) {
#pragma unroll
        for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(dst + j) = make_float4(z[j], z[j + 1], z[j + 2], z[j + 3]);
      } else {
        for (int e = 0; e < valid; e++) dst[e] = z[e];
      }
    }
    return;
  }
  uint32_t* brow = ep.nx_bits + m * ep.nx_ld_words;
  const int64_t srow = m * ep.nx_ld_scales;
  switch (ep.nx_beta) {
    case 2: emit_next_chunk<2>(z, valid, n0, N, brow, ep.nx_scales, ep.nx_bf16, srow, ep.nx_ld_scales, carry); break;
    case 4: emit_next_chunk<4>(z, valid, n0, N, brow, ep.nx_scales, ep.nx_bf16, srow, ep.nx_ld_scales, carry); break;
    case 8: emit_next_chunk<8>(z, valid, n0, N, brow, ep.nx_scales, ep.nx_bf16, srow, ep.nx_ld_scales, carry); break;
    case 16: emit_next_chunk<16>(z, valid, n0, N, brow, ep.nx_scales, ep.nx_bf16, srow, ep.nx_ld_scales, carry); break;
    case 32: emit_next_chunk<32>(z, valid, n0, N, brow, ep.nx_scales, ep.nx_bf16, srow, ep.nx_ld_scales, carry); break;
    case 64: emit_next_chunk<64>(z, valid, n0, N, brow, ep.nx_scales, ep.nx_bf16, srow, ep.nx_ld_scales, carry); break;
    default: emit_next_chunk<128>(z, valid, n0, N, brow, ep.nx_scales, ep.nx_bf16, srow, ep.nx_ld_scales, carry); break;
  }
  if (last_chunk_of_row_tile && tile_end >= N) {
    // last column tile: the row's zero padding past what the tiles cover
    for (int64_t wz = tile_end >> 5; wz < ep.nx_ld_words; wz++) brow[wz] = 0u;
    for (int64_t sz = tile_end / ep.nx_beta; sz < ep.nx_ld_scales; sz++) store_next_scale(ep.nx_scales, ep.nx_bf16, srow + sz, 0.0f);
  }
}

}  // namespace epi
}  // namespace hbmm
