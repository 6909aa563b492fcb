// Pieces of the folded-scale tcgen05 HBMM kernel that other translation units need: the shared-memory
// stage layout, the routine that turns packed words + group scales into fp16 operand tiles, and the
// weight-expansion task (the packed convolution front end runs it in a few extra CTAs of its launch).
//
// Folded scales.  A Hadamard-binary operand X~ = delta (.) Sign(X) (Eq. 2 / Eq. 4) is written as the sum of
// two fp16 matrices X1 + X2: the group scale, multiplied by a power of two 2^u chosen per row so that the
// row's largest scale lies in [2^14, 2^15), is split as delta * 2^u = d1 + d2 with d1 = fp16(delta * 2^u) and
// d2 = fp16(delta * 2^u - d1) (the remainder is exact in fp32), and element k of piece i is +-d_i.  d1 + d2
// carries 22 significant bits of every scale that is within 2^-17 of its row's largest (below that d2
// becomes subnormal and the error is at most 2^-39 of the row's largest scale).  fp16 x fp16 products are
// exact in fp32, so A~ W~^T = (A1 + A2)(W1 + W2)^T accumulated in fp32 reproduces Eq. 7's per-group
// full-precision scaling with no per-group step at all; the powers of two are divided out once per output.
#pragma once
#include <cuda_fp16.h>
#include <cstdint>
#include "kernels.h"
#include "umma_common.cuh"

namespace hbmm {
namespace fold {

using namespace umma;
using Args = FoldArgs;

constexpr int KB = 64;            // K elements per stage: one 128-byte row of fp16
constexpr int WPS = 2;            // packed K-words per stage
constexpr int kRowSlots = 8;      // ring of per-tile row factors (scouts -> producers and epilogue)

// The weight stages live in shared memory (streamed from the prepared workspace by bulk copies); the
// activation pieces live in TENSOR memory: the producers write them there straight from registers and the
// MMA reads its A operand from there, so the activation operand never touches shared memory.
template <int TN>
struct Smem {
  static constexpr int A_COLS = 2 * (KB / 2);             // TMEM columns of one A stage: two pieces x 64 fp16 (two per 32-bit column)
  // A tensor-core instruction costs about the same for 64 and for 128 columns, so the narrow tile stacks
  // the two weight pieces along N: one MMA of 2 TN columns forms A1 W1 and A1 W2 side by side (the epilogue
  // adds the two blocks) and a second one of TN columns adds A2 W1.  The wide tile has no room for a
  // 256-column accumulator pair beside the A ring and adds all three products into the same TN columns.
  static constexpr bool STACKED = TN == 64;
  static constexpr int ACC_COLS = STACKED ? 2 * TN : TN;  // one fp32 accumulator
  static constexpr int STAGES = (512 - 2 * ACC_COLS) / A_COLS;        // 4: the rest of the 512 columns
  static constexpr int A_BASE = 2 * ACC_COLS;             // first TMEM column of the A ring
  static constexpr int TMEM_COLS = 512;
  static constexpr int B_PIECE = TN * 128;
  static constexpr int B_STAGE = 2 * B_PIECE;             // W1 rows then W2 rows
  static constexpr int OFF_B = 0;
  static constexpr int OFF_ROWF = OFF_B + STAGES * B_STAGE;
  static constexpr int OFF_COLF = OFF_ROWF + 2 * kRowSlots * TM * 4;  // per slot and row: normalising power of two and its inverse
  static constexpr int OFF_BAR = OFF_COLF + 3 * 4 * TN * 4;           // the tile's column factors (power of two, affine scale and shift), one copy per epilogue warp
  static constexpr int NBAR = 2 * STAGES + 4 + 1 + 2 * kRowSlots;     // full, empty, tfull[2], tempty[2], drain, rowfull, rowempty
  static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
  static constexpr int USED = OFF_MISC + 16;
  // more than half of an SM's shared memory is requested whatever is used: one CTA per SM, which owns all 512
  // columns of tensor memory
  static constexpr int BYTES = USED > 120 * 1024 ? USED : 120 * 1024;
  static_assert(STAGES >= 3 && A_BASE + STAGES * A_COLS <= 512, "accumulators and the A ring share 512 columns");
};

__device__ __forceinline__ float load_scale(const void* s, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(s) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(s) + idx);
}

// Largest scale of one operand row.  Rows are 16-byte vectors (the leading dimension is a multiple of 4
// fp32 / 8 bf16 entries) and entries past the last group are stored zeros.  Scales are >= 0, so their bit
// patterns order like the values.
__device__ __forceinline__ float row_max_scale(const void* s, int bf16, int64_t row_off, int64_t ld) {
  uint32_t mx = 0;
  if (bf16) {
    const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned short*>(s) + row_off);
#pragma unroll 4
    for (int64_t i = 0; i < ld / 8; i++) {
      const uint4 v = __ldg(p + i);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; e++) { mx = max(mx, w[e] << 16); mx = max(mx, w[e] & 0xFFFF0000u); }
    }
  } else {
    const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(s) + row_off);
#pragma unroll 4
    for (int64_t i = 0; i < ld / 4; i++) {
      const uint4 v = __ldg(p + i);
      mx = max(max(mx, v.x), max(v.y, max(v.z, v.w)));
    }
  }
  return __uint_as_float(mx);
}

// The same for two rows at once (both rows' loads in flight together).
__device__ __forceinline__ void row_max_scale2(const void* s, int bf16, int64_t off_a, int64_t off_b, int64_t ld, float& max_a, float& max_b) {
  uint32_t ma = 0, mb = 0;
  if (bf16) {
    const uint4* pa = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned short*>(s) + off_a);
    const uint4* pb = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned short*>(s) + off_b);
#pragma unroll 2
    for (int64_t i = 0; i < ld / 8; i++) {
      const uint4 va = __ldg(pa + i), vb = __ldg(pb + i);
      const uint32_t wa[4] = {va.x, va.y, va.z, va.w}, wb[4] = {vb.x, vb.y, vb.z, vb.w};
#pragma unroll
      for (int e = 0; e < 4; e++) {
        ma = max(ma, wa[e] << 16); ma = max(ma, wa[e] & 0xFFFF0000u);
        mb = max(mb, wb[e] << 16); mb = max(mb, wb[e] & 0xFFFF0000u);
      }
    }
  } else {
    const uint4* pa = reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(s) + off_a);
    const uint4* pb = reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(s) + off_b);
    // eight 16-byte loads of each row in flight: rows of a few hundred scales are scanned at a rate set by how much
    // is in flight, and the scouts have little else in registers
    int64_t i = 0;
    for (; i + 8 <= ld / 4; i += 8) {
      uint4 va[8], vb[8];
#pragma unroll
      for (int u = 0; u < 8; u++) { va[u] = __ldg(pa + i + u); vb[u] = __ldg(pb + i + u); }
#pragma unroll
      for (int u = 0; u < 8; u++) {
        ma = max(max(ma, va[u].x), max(va[u].y, max(va[u].z, va[u].w)));
        mb = max(max(mb, vb[u].x), max(vb[u].y, max(vb[u].z, vb[u].w)));
      }
    }
    for (; i < ld / 4; i++) {
      const uint4 va = __ldg(pa + i), vb = __ldg(pb + i);
      ma = max(max(ma, va.x), max(va.y, max(va.z, va.w)));
      mb = max(max(mb, vb.x), max(vb.y, max(vb.z, vb.w)));
    }
  }
  max_a = __uint_as_float(ma);
  max_b = __uint_as_float(mb);
}

// Powers of two for a row whose largest scale is mx: mx * up lies in [2^14, 2^15), down = 1 / up.
// Rows whose scales are all below 2^-100 (an all-zero row included) are treated as if their largest
// were 2^-100, which keeps both factors normal numbers.
__device__ __forceinline__ void norm_factors(float mx, float& up, float& down) {
  uint32_t e = (__float_as_uint(mx) >> 23) & 0xFFu;      // biased exponent
  e = e < 27u ? 27u : e;
  up = __uint_as_float((268u - e) << 23);                // 2^(14 - (e - 127))
  down = __uint_as_float((e - 14u) << 23);               // 2^((e - 127) - 14)
}

// One packed K-word of tile row `row` -> its 32 elements in both fp16 pieces.  `scaled` is the word's
// group scale times the row's power of two (0 for words past K or rows past the operand: +-0).
// Word slot q of the stage fills the 16-byte chunks 4q .. 4q+3 of the 128-byte row; 32-bit position j of
// the slot holds the elements of bits j (low half) and j + 16 (high half).  Both operands use this
// order, and a dot product does not depend on the order of its terms.  Bit 1 <=> +1, bit 0 <=> -1: the
// inverted bit is moved onto the fp16 sign.
__device__ __forceinline__ void expand_word(unsigned char* piece1, unsigned char* piece2, int row, int q, uint32_t word, float scaled) {
  const __half d1 = __float2half_rn(scaled);
  const __half d2 = __float2half_rn(scaled - __half2float(d1));
  const uint32_t h1 = static_cast<uint32_t>(__half_as_ushort(d1)) * 0x10001u;
  const uint32_t h2 = static_cast<uint32_t>(__half_as_ushort(d2)) * 0x10001u;
  const uint32_t nw = ~word;
#pragma unroll
  for (int c = 0; c < 4; c++) {
    uint32_t m[4];
#pragma unroll
    for (int i = 0; i < 4; i++) m[i] = (nw << (15 - (4 * c + i))) & 0x80008000u;
    *reinterpret_cast<uint4*>(swz(piece1, row, 4 * q + c)) = make_uint4(m[0] ^ h1, m[1] ^ h1, m[2] ^ h1, m[3] ^ h1);
    *reinterpret_cast<uint4*>(swz(piece2, row, 4 * q + c)) = make_uint4(m[0] ^ h2, m[1] ^ h2, m[2] ^ h2, m[3] ^ h2);
  }
}

// The same 32 elements as 16 + 16 register values (one per 32-bit column of tensor memory): column j of the
// word's 16 columns holds the elements of bits j (low half) and j + 16 (high half), exactly the pairs
// expand_word stores at 32-bit position j.
__device__ __forceinline__ void expand_word_regs(uint32_t word, float scaled, uint32_t (&p1)[16], uint32_t (&p2)[16]) {
  const __half d1 = __float2half_rn(scaled);
  const __half d2 = __float2half_rn(scaled - __half2float(d1));
  const uint32_t h1 = static_cast<uint32_t>(__half_as_ushort(d1)) * 0x10001u;
  const uint32_t h2 = static_cast<uint32_t>(__half_as_ushort(d2)) * 0x10001u;
  const uint32_t nw = ~word;
#pragma unroll
  for (int j = 0; j < 16; j++) {
    const uint32_t m = (nw << (15 - j)) & 0x80008000u;
    p1[j] = m ^ h1;
    p2[j] = m ^ h2;
  }
}
template <int SUB>
__device__ __forceinline__ void expand_word_sub_regs(uint32_t word, const float (&scaled)[SUB], uint32_t (&p1)[16], uint32_t (&p2)[16]) {
  static_assert(SUB == 2 || SUB == 4 || SUB == 8 || SUB == 16, "beta = 16, 8, 4, 2");
  constexpr int BETA = 32 / SUB, HALF = SUB / 2;
  uint32_t h1[HALF], h2[HALF];
#pragma unroll
  for (int t = 0; t < HALF; t++) {
    const __half2 d1 = __floats2half2_rn(scaled[t], scaled[t + HALF]);          // low half: group t, high half: group t + SUB/2
    const float2 back = __half22float2(d1);
    const __half2 d2 = __floats2half2_rn(scaled[t] - back.x, scaled[t + HALF] - back.y);
    h1[t] = *reinterpret_cast<const uint32_t*>(&d1);
    h2[t] = *reinterpret_cast<const uint32_t*>(&d2);
  }
  const uint32_t nw = ~word;
#pragma unroll
  for (int j = 0; j < 16; j++) {
    const uint32_t m = (nw << (15 - j)) & 0x80008000u;
    p1[j] = m ^ h1[j / BETA];
    p2[j] = m ^ h2[j / BETA];
  }
}

// The same for sub-word groups (beta = 32 / SUB = 2 .. 16, the settings of the paper's experiments): the
// word has SUB scales, group i covering bits [i * beta, (i + 1) * beta).  Position j holds bits j and j + 16,
// i.e. groups j / beta and j / beta + SUB / 2, so there are SUB / 2 distinct pairs of fp16 values per piece.
template <int SUB>
__device__ __forceinline__ void expand_word_sub(unsigned char* piece1, unsigned char* piece2, int row, int q, uint32_t word,
                                                const float (&scaled)[SUB]) {
  static_assert(SUB == 2 || SUB == 4 || SUB == 8 || SUB == 16, "beta = 16, 8, 4, 2");
  constexpr int BETA = 32 / SUB, HALF = SUB / 2;
  uint32_t h1[HALF], h2[HALF];
#pragma unroll
  for (int t = 0; t < HALF; t++) {
    const __half2 d1 = __floats2half2_rn(scaled[t], scaled[t + HALF]);          // low half: group t, high half: group t + SUB/2
    const float2 back = __half22float2(d1);
    const __half2 d2 = __floats2half2_rn(scaled[t] - back.x, scaled[t + HALF] - back.y);
    h1[t] = *reinterpret_cast<const uint32_t*>(&d1);
    h2[t] = *reinterpret_cast<const uint32_t*>(&d2);
  }
  const uint32_t nw = ~word;
#pragma unroll
  for (int c = 0; c < 4; c++) {
    uint32_t m[4], o1[4], o2[4];
#pragma unroll
    for (int i = 0; i < 4; i++) {
      const int j = 4 * c + i;
      m[i] = (nw << (15 - j)) & 0x80008000u;
      o1[i] = m[i] ^ h1[j / BETA];
      o2[i] = m[i] ^ h2[j / BETA];
    }
    *reinterpret_cast<uint4*>(swz(piece1, row, 4 * q + c)) = make_uint4(o1[0], o1[1], o1[2], o1[3]);
    *reinterpret_cast<uint4*>(swz(piece2, row, 4 * q + c)) = make_uint4(o2[0], o2[1], o2[2], o2[3]);
  }
}

// SUB scales of one word (index of the first one given), times the row's power of two.
template <int SUB>
__device__ __forceinline__ void load_scaled(const void* s, int bf16, int64_t idx, float up, float (&out)[SUB]) {
  if (!bf16) {
    const float* p = reinterpret_cast<const float*>(s) + idx;       // idx is a multiple of SUB: vectors stay aligned
    if (SUB == 2) {
      const float2 v = __ldg(reinterpret_cast<const float2*>(p));
      out[0] = v.x * up; out[1] = v.y * up;
    } else {
#pragma unroll
      for (int i = 0; i < SUB / 4; i++) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(p) + i);
        out[4 * i] = v.x * up; out[4 * i + 1] = v.y * up; out[4 * i + 2] = v.z * up; out[4 * i + 3] = v.w * up;
      }
    }
  } else {
    const uint32_t* p = reinterpret_cast<const uint32_t*>(reinterpret_cast<const unsigned short*>(s) + idx);
#pragma unroll
    for (int i = 0; i < SUB / 2; i++) {
      const uint32_t v = __ldg(p + i);
      out[2 * i] = __uint_as_float(v << 16) * up;
      out[2 * i + 1] = __uint_as_float(v & 0xFFFF0000u) * up;
    }
  }
}

// One word of a weight row with a run-time number of groups per word.
__device__ __forceinline__ void expand_weight_word(unsigned char* p1, unsigned char* p2, int row, int q, uint32_t word, const void* scales,
                                                   int bf16, int64_t idx, int sub, float up, bool valid) {
  if (!valid) { expand_word(p1, p2, row, q, 0u, 0.0f); return; }
  switch (sub) {
    case 2: { float sc[2]; load_scaled<2>(scales, bf16, idx, up, sc); expand_word_sub<2>(p1, p2, row, q, word, sc); break; }
    case 4: { float sc[4]; load_scaled<4>(scales, bf16, idx, up, sc); expand_word_sub<4>(p1, p2, row, q, word, sc); break; }
    case 8: { float sc[8]; load_scaled<8>(scales, bf16, idx, up, sc); expand_word_sub<8>(p1, p2, row, q, word, sc); break; }
    case 16: { float sc[16]; load_scaled<16>(scales, bf16, idx, up, sc); expand_word_sub<16>(p1, p2, row, q, word, sc); break; }
    default: expand_word(p1, p2, row, q, word, load_scale(scales, bf16, idx) * up); break;
  }
}

// Expands kPrepStages consecutive stages (short tasks: many of them run side by side) of one column tile of the weight operand into the stage layout
// the main kernel streams: rows 0 .. TN-1 piece 1, rows TN .. 2TN-1 piece 2, exactly as they sit in
// shared memory.  The task of the first stages also stores the rows' inverse powers of two.
// p = row of the tile, one thread per row (it scans its row's scales once per task).
constexpr int kPrepStages = 2;
template <int TN>
__device__ __forceinline__ void prepare_w_task(const Args& g, unsigned char* __restrict__ out, float* __restrict__ w_down,
                                               int64_t chunk, int64_t tile_n, int p) {
  using S = Smem<TN>;
  const int64_t n_stages = (g.n_words + WPS - 1) / WPS;
  const int64_t n = tile_n * TN + p;
  const bool in = n < g.N;
  float up = 0.0f, down = 1.0f;
  if (in) norm_factors(row_max_scale(g.w_scales, g.w_bf16, n * g.ldw_s, g.ldw_s), up, down);
  if (chunk == 0) w_down[n] = down;
  if (g.sk_counters != nullptr) {
    // the per-tile arrival counters of the balanced schedule start at zero; every launch leaves them there
    const int64_t n_chunks = (n_stages + kPrepStages - 1) / kPrepStages, tiles_n = (g.N + TN - 1) / TN;
    for (int64_t i = (tile_n * n_chunks + chunk) * TN + p; i < g.sk_counter_count; i += tiles_n * n_chunks * TN) g.sk_counters[i] = 0;
  }
  const int64_t st0 = chunk * kPrepStages;
  const int64_t st1 = st0 + kPrepStages < n_stages ? st0 + kPrepStages : n_stages;
  for (int64_t st = st0; st < st1; st++) {
    unsigned char* base = out + (tile_n * n_stages + st) * S::B_STAGE;
#pragma unroll
    for (int q = 0; q < WPS; q++) {
      const int64_t wi = st * WPS + q;
      const bool valid = in && wi < g.n_words;
      const uint32_t word = valid ? __ldg(g.w_bits + n * g.ldw_w + wi) : 0u;
      const int64_t idx = n * g.ldw_s + (g.w_sub > 1 ? wi * g.w_sub : wi / g.w_gw);
      expand_weight_word(base, base + S::B_PIECE, p, q, word, g.w_scales, g.w_bf16, idx, g.w_sub, up, valid);
    }
  }
}

}  // namespace fold
}  // namespace hbmm
