// HBMM contraction of two packed operands on the 5th-generation tensor cores with the group scales
// folded into the operands (tcgen05 / TMEM).
//
// Section 4.2, Eq. 7 computes  C[m,n] = sum_g deltaA[m,g] deltaW[n,g] D_g[m,n]  with D_g the signed +-1 dot
// of group g.  That is the plain product of the Hadamard-product operands A~ = deltaA (.) Sign(A) and
// W~ = deltaW (.) Sign(W) (Eq. 2 / Eq. 4).  Here each operand is expanded on the fly into two fp16
// matrices whose sum carries its fp32 group scales to 22 bits (see gemm_fold_prep.cuh), every fp16 x fp16
// product is exact in the fp32 accumulator, and the cross products
//     A1 W1^T + A1 W2^T + A2 W1^T
// are one accumulation in tensor memory over the whole of K: per 16 K-elements three MMAs of 128 x TN x 16
// (A1 against W1, A2 against W1, A1 against W2) add into the same TN accumulator columns (the 64-column tile
// forms A1 W1 and A1 W2 with one MMA of 128 columns instead and adds the blocks in the epilogue).  The fourth product A2 W2^T is left out: both second pieces are
// constant inside a scale group and at most 2^-11 of the first, so it equals sum_g (a2_g w2_g) D_g, at
// most 2^-22 of sum_g |deltaA deltaW D_g| -- forty times below the 1e-5 the result is held to.
// There is no per-group step; the epilogue runs once per tile and divides the rows' and columns' powers of
// two out again (exact).  Compared with forming D_g and the scale
// product per group this trades 3x the tensor work for the removal of the per-group TMEM round trip
// that bounded the e4m3 kernel.
//
// CTA tile = 128 rows x TN columns; one persistent CTA per SM walks the tiles of the output.
//   warps 0-3   : epilogue, once per tile (TMEM lanes 32*w ..)
//   warps 4-11  : A producers: thread = (tile row, stage parity); packed words + group scales -> the
//                 64 elements of both fp16 pieces, written from registers straight into TENSOR memory (the
//                 MMA takes its A operand from there: the activation operand never passes through shared
//                 memory, whose bandwidth bounded the kernel while it did), with the global loads issued
//                 several stages ahead
//   warps 14-15 : scouts: one thread per two tile rows finds a row's largest scale (the power of two that
//                 normalises the row) a few tiles ahead of everyone else
//   warp  12    : TMEM allocation and the single MMA-issuing thread
//   warp  13    : one thread streams the prepared W stages (cp.async.bulk, completion on the stage's
//                 mbarrier); W is expanded once per call (or once per weight tensor) into a workspace
// A stage holds 64 K-elements (two packed words): 64 TMEM columns of A pieces and the W stage in shared
// memory.  Tensor memory: two accumulators of TN columns, the rest is the ring of A stages.  Stages and the
// accumulators are mbarrier rings.  Every wait is bounded: on expiry the thread records a code, raises a
// CTA-wide abort flag that all other waits observe, and the kernel drains and frees its TMEM before returning.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "kernels.h"
#include "tensor_map.h"
#include "umma_common.cuh"
#include "gemm_fold_prep.cuh"
#include "epilogue.cuh"
#include "pdl.cuh"

namespace hbmm {
namespace {

using namespace umma;
using namespace fold;

constexpr int kEpilogueWarps = 4;
constexpr int kProducerWarps = 8;
constexpr int kFirstProducerWarp = kEpilogueWarps;
constexpr int kMmaWarp = kEpilogueWarps + kProducerWarps;   // 12
constexpr int kLoaderWarp = kMmaWarp + 1;                   // 13
constexpr int kFirstScoutWarp = kLoaderWarp + 1;            // 14..17
constexpr int kScoutWarps = 2;                              // 16 warps in all: 128 registers per thread
constexpr int kThreads = (kFirstScoutWarp + kScoutWarps) * 32;
// Stages of packed words + scales each producer thread keeps in flight; fewer when a word has many scales.
template <int SUBW> struct DepthFor { static constexpr int value = SUBW == 1 ? 4 : (SUBW <= 4 ? 2 : 1); };

// Sub-word groups (beta_a = 32 / ASUB): a stage of a tile needs 2 ASUB scales per row -- up to 128 bytes a row, 16 KB a
// stage, against 1 KB of packed words.  Loaded by the producer threads themselves (one row per lane) these are
// hundreds of scattered 16-byte requests per stage with nothing to hide their latency behind; instead the loader
// thread brings the stage's [128 rows][2 ASUB] block of fp32 scales with one tensor copy into a ring beside the
// weight stages, and the producers read their rows from shared memory.  The copy swizzles the rows' 16-byte
// pieces (by the row number, as wide as the row is long), so 8 consecutive rows read 8 different bank groups.
constexpr int kStagedFrom = 4;          // groups per word from which the scales go through shared memory (beta_a <= 8)
constexpr int64_t kRowMaxFrom = 512;    // scales per row from which a kernel of its own finds the rows' largest scales
template <int TN, int ASUB>
struct ScaleRing {
  static constexpr int ROW_BYTES = 8 * ASUB;                       // two words' scales
  static constexpr int STAGE = TM * ROW_BYTES;
  // The ring is deeper than the ring of weight stages: the block of stage g + LEAD is requested when stage g's weight
  // copy is (its slot last served stage g - STAGES, whose MMAs -- hence whose producers -- are done by then).
  static constexpr int NS = ASUB == 16 ? Smem<TN>::STAGES + 1 : 2 * Smem<TN>::STAGES;
  static constexpr int LEAD = NS - Smem<TN>::STAGES;
  static constexpr int OFF = (Smem<TN>::USED + 1023) / 1024 * 1024;
  static constexpr int OFF_BAR = OFF + NS * STAGE;                 // sfull[NS]
  static constexpr int BYTES = ASUB == 1 ? Smem<TN>::BYTES : OFF_BAR + NS * 8 + 16;
  // byte offset of the 16-byte piece c of row p inside a stage block
  __device__ static __forceinline__ int piece(int p, int c) {
    if (ASUB == 16) return p * 128 + ((c ^ (p & 7)) << 4);
    if (ASUB == 8) return p * 64 + ((c ^ ((p >> 1) & 3)) << 4);
    if (ASUB == 4) return p * 32 + ((c ^ ((p >> 2) & 1)) << 4);
    return p * 16;
  }
};

template <int TN>
__global__ void __launch_bounds__(TN)
prepare_w_fold_kernel(const Args g, unsigned char* __restrict__ out, float* __restrict__ w_down) {
  prepare_w_task<TN>(g, out, w_down, blockIdx.x, blockIdx.y, threadIdx.x);
}

// Largest scale of every row of an operand with many scales per row (sub-word groups): one warp per row, consecutive
// lanes on consecutive 16-byte vectors.  Scales are >= 0, so their bit patterns order like the values; entries past the
// last group are stored zeros.
__global__ void __launch_bounds__(256)
row_max_kernel(const float* __restrict__ scales, int64_t ld, int64_t M, float* __restrict__ out) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t m = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (m >= M) return;
  const uint4* p = reinterpret_cast<const uint4*>(scales + m * ld);
  const int64_t n_vec = ld / 4;
  uint32_t x0 = 0, x1 = 0, x2 = 0, x3 = 0;
  int64_t j = lane;
  for (; j + 96 < n_vec; j += 128) {
    const uint4 a = __ldg(p + j), b = __ldg(p + j + 32), c = __ldg(p + j + 64), d = __ldg(p + j + 96);
    x0 = max(max(x0, a.x), max(a.y, max(a.z, a.w)));
    x1 = max(max(x1, b.x), max(b.y, max(b.z, b.w)));
    x2 = max(max(x2, c.x), max(c.y, max(c.z, c.w)));
    x3 = max(max(x3, d.x), max(d.y, max(d.z, d.w)));
  }
  for (; j < n_vec; j += 32) {
    const uint4 a = __ldg(p + j);
    x0 = max(max(x0, a.x), max(a.y, max(a.z, a.w)));
  }
  uint32_t x = max(max(x0, x1), max(x2, x3));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = max(x, __shfl_xor_sync(0xFFFFFFFFu, x, o));
  if (lane == 0) out[m] = __uint_as_float(x);
}

// Walks the stages a producer thread owns (every second stage of the CTA's stream of tiles) and keeps
// the row pointers of the tile it is in.
struct StageCursor {
  int64_t ti, st;            // tile (in this CTA's sequence) and stage inside it
  int64_t end;               // one past the last stage of the segment (ti)
  const uint32_t* bptr;      // packed words of this thread's row
  int64_t srow;              // first scale of the row
  bool in;                   // the row exists
};

// ASUB: scale groups per packed word of A (1: groups of whole words; 2 .. 16: beta_a = 16 .. 2).
// FUSE: the epilogue runs the activation / affine map / dense or binarized output chain of epilogue.cuh instead of
// storing the product as fp32.
// BAL: the balanced schedule (runs of (tile, stage) pairs, partial tiles reduced by the last CTA to arrive); the plain
// instantiation carries none of its code.
template <int TN, int ASUB, bool FUSE, bool BAL>
__global__ void __launch_bounds__(kThreads, 1)
hbmm_fold_kernel(const Args g, const __grid_constant__ CUtensorMap s_map) {
  using S = Smem<TN>;
  using SR = ScaleRing<TN, ASUB>;
  const bool staged = ASUB > 1 && g.a_staged;                    // the stage's scales come through shared memory
  constexpr int kDepth = DepthFor<ASUB>::value;
  constexpr int STAGES = S::STAGES;
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + S::OFF_BAR);
  uint64_t* sfull = reinterpret_cast<uint64_t*>(smem + (ASUB > 1 ? SR::OFF_BAR : S::OFF_BAR));   // the scale block of a stage has arrived
  uint64_t* empty = full + STAGES;
  uint64_t* tfull = empty + STAGES;
  uint64_t* tempty = tfull + 2;
  uint64_t* drain = tempty + 2;
  uint64_t* rowfull = drain + 1;                 // the scouts have stored a tile's row factors
  uint64_t* rowempty = rowfull + kRowSlots;      // the epilogue has read them
  float* rowup = reinterpret_cast<float*>(smem + S::OFF_ROWF);
  float* rowdown = rowup + kRowSlots * TM;
  float* colf = reinterpret_cast<float*>(smem + S::OFF_COLF);
  uint32_t* tmem_base_ptr = reinterpret_cast<uint32_t*>(smem + S::OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + S::OFF_MISC + 4);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t tiles_n = (g.N + TN - 1) / TN, tiles_m = (g.M + TM - 1) / TM;
  const int64_t n_tiles = tiles_m * tiles_n;
  const int64_t n_stages = (g.n_words + WPS - 1) / WPS;      // per tile
  // The CTA's work is a list of segments (tile, first stage, one past the last stage).  Plain schedule: whole tiles
  // blockIdx.x, blockIdx.x + gridDim.x, ...  Balanced schedule: the run [u0, u1) of the tile-major (tile, stage)
  // sequence -- consecutive tiles, the first possibly entered mid-way, the last possibly left early.
  constexpr bool balanced = BAL;
  const int64_t u0 = balanced ? static_cast<int64_t>(blockIdx.x) * g.sk_units : 0;
  const int64_t u_end = balanced ? ((u0 + g.sk_units < n_tiles * n_stages) ? u0 + g.sk_units : n_tiles * n_stages) : 0;
  const int64_t sk_t0 = balanced ? u0 / n_stages : 0;                                  // first tile of the run
  const int64_t sk_first = balanced ? u0 - sk_t0 * n_stages : 0;                       // first stage inside it
  const int64_t sk_t1 = (balanced && u_end > u0) ? (u_end - 1) / n_stages : 0;         // last tile of the run
  const int64_t sk_last_end = (balanced && u_end > u0) ? u_end - sk_t1 * n_stages : 0; // one past its last stage
  const int64_t my_tiles = balanced ? (u_end > u0 ? sk_t1 - sk_t0 + 1 : 0)
                                    : (blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0);
  const int64_t my_stages = balanced ? (u_end > u0 ? u_end - u0 : 0) : my_tiles * n_stages;
  // Order of work in a balanced run: the two tiles shared with the neighbouring runs first (the tail of the run's first
  // tile, then the head of its last), the whole tiles after them -- so partial accumulators are handed in early and
  // the CTA that completes a shared tile does so in the shadow of the MMAs of its whole tiles, not at the kernel's end.
  const bool reorder = balanced && my_tiles >= 3;
  auto seg_nat = [&](int64_t ti) -> int64_t { return !reorder ? ti : (ti == 0 ? 0 : (ti == 1 ? my_tiles - 1 : ti - 1)); };
  auto seg_tile = [&](int64_t ti) -> int64_t { return balanced ? sk_t0 + seg_nat(ti) : blockIdx.x + ti * gridDim.x; };
  auto seg_begin = [&](int64_t ti) -> int64_t { return (balanced && ti < my_tiles && seg_nat(ti) == 0) ? sk_first : 0; };
  auto seg_end = [&](int64_t ti) -> int64_t { return (balanced && ti < my_tiles && seg_nat(ti) == my_tiles - 1) ? sk_last_end : n_stages; };

  pdl_launch_dependents();      // the next kernel of the stream may start its own set-up
  if (tid == 0) {
    for (int s = 0; s < STAGES; s++) {
      mbar_init(&full[s], kProducerWarps / 2 + 1);  // the four producer warps of the stage + the loader's expect_tx arrival
      mbar_init(&empty[s], 1);                      // MMA commit: the stage's bytes have been read
    }
    for (int b = 0; b < 2; b++) { mbar_init(&tfull[b], 1); mbar_init(&tempty[b], kEpilogueWarps); }
    mbar_init(drain, 1);
    if (ASUB > 1)
      for (int s = 0; s < SR::NS; s++) mbar_init(&sfull[s], 1);        // the loader's expect_tx arrival; the copy completes the bytes
    for (int r = 0; r < kRowSlots; r++) { mbar_init(&rowfull[r], kScoutWarps); mbar_init(&rowempty[r], kEpilogueWarps); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    tmem_alloc(tmem_base_ptr, S::TMEM_COLS);
    tmem_relinquish();
  }
  pdl_wait();                   // everything before this line touched no global memory
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_ptr;

  // The CTA is persistent: it walks tiles blockIdx.x, blockIdx.x + gridDim.x, ... and the stage ring
  // simply continues across tiles (gst counts stages since launch).
  if (warp >= kFirstProducerWarp && warp < kMmaWarp) {
    // =========================== A producers ===========================
    // Thread = (tile row p, parity q): it expands both words of every stage whose number since launch
    // has parity q.  Packed words and scales are loaded kDepth of its stages (2 kDepth stages of the
    // CTA) ahead, across tile boundaries, so that no global-memory latency is left in the stage loop.
    const int pt = tid - kFirstProducerWarp * 32;
    const int q = pt >> 7;
    const int p = pt & (TM - 1);
    const uint32_t t_lane = static_cast<uint32_t>((warp & 3) * 32) << 16;     // this warp's quarter of the TMEM lanes = its tile rows
    const uint32_t n_words = static_cast<uint32_t>(g.n_words), gw = static_cast<uint32_t>(g.a_gw);
    const bool vec_scales = ASUB == 1 && !g.a_bf16 && gw == 1;      // one fp32 scale per word: a stage's two scales are one 8-byte load
    const int64_t total = my_stages;
    auto set_tile = [&](StageCursor& c) {
      const int64_t tile = seg_tile(c.ti);
      const int64_t m = (tile / tiles_n) * TM + p;
      c.in = c.ti < my_tiles && m < g.M;
      c.bptr = g.a_bits + (c.in ? m : 0) * g.lda_w;
      c.srow = (c.in ? m : 0) * g.lda_s;
    };
    auto carry_over = [&](StageCursor& c) {        // moves a stage index past its segment's end into the segments after it
      if (c.st >= c.end) {
        if (!balanced) {
          do { c.st -= n_stages; c.ti++; } while (c.st >= n_stages);
        } else {
          do { const int64_t over = c.st - c.end; c.ti++; c.st = seg_begin(c.ti) + over; c.end = seg_end(c.ti); } while (c.st >= c.end);
        }
        set_tile(c);
      }
    };
    auto advance = [&](StageCursor& c) {
      c.st += 2;
      carry_over(c);
    };
    // raw scales of the stage's two words: sc[0 .. ASUB) of the first, sc[ASUB .. 2 ASUB) of the second
    auto fetch = [&](const StageCursor& c, uint2& w, float (&sc)[2 * ASUB]) {
      w = make_uint2(0u, 0u);
#pragma unroll
      for (int i = 0; i < 2 * ASUB; i++) sc[i] = 0.0f;
      const uint32_t wi = static_cast<uint32_t>(c.st) * WPS;
      if (c.in && wi < n_words) {
        w = __ldg(reinterpret_cast<const uint2*>(c.bptr + wi));      // the row is padded with zero words to a multiple of four
        if (ASUB > 1 && staged) {
          // the scales arrive in shared memory
        } else if (ASUB > 1) {
          // K is a multiple of 32 here, so every word has all its ASUB groups
          float lo[ASUB], hi[ASUB];
          load_scaled<(ASUB > 1 ? ASUB : 2)>(g.a_scales, g.a_bf16, c.srow + static_cast<int64_t>(wi) * ASUB, 1.0f,
                                             reinterpret_cast<float(&)[(ASUB > 1 ? ASUB : 2)]>(lo));
#pragma unroll
          for (int i = 0; i < ASUB; i++) { sc[i] = lo[i]; hi[i] = 0.0f; }
          if (wi + 1 < n_words)
            load_scaled<(ASUB > 1 ? ASUB : 2)>(g.a_scales, g.a_bf16, c.srow + static_cast<int64_t>(wi + 1) * ASUB, 1.0f,
                                               reinterpret_cast<float(&)[(ASUB > 1 ? ASUB : 2)]>(hi));
#pragma unroll
          for (int i = 0; i < ASUB; i++) sc[ASUB + i] = hi[i];
        } else if (vec_scales) {
          const float2 v = __ldg(reinterpret_cast<const float2*>(reinterpret_cast<const float*>(g.a_scales) + c.srow + wi));
          sc[0] = v.x;
          sc[ASUB] = v.y;                                              // past the last group: a stored zero
        } else {
          sc[0] = load_scale(g.a_scales, g.a_bf16, c.srow + wi / gw);
          if (wi + 1 < n_words) sc[ASUB] = load_scale(g.a_scales, g.a_bf16, c.srow + (wi + 1) / gw);
        }
      }
    };
    StageCursor pf, cur;
    pf.ti = 0; pf.st = seg_begin(0) + q; pf.end = seg_end(0);      // the stage walk continues from segment to segment
    carry_over(pf);
    set_tile(pf);
    cur = pf;
    uint2 w[kDepth];
    float sc[kDepth][2 * ASUB];
#pragma unroll
    for (int u = 0; u < kDepth; u++) { fetch(pf, w[u], sc[u]); advance(pf); }
    int64_t up_tile = -1;
    float up = 0.0f;
    bool ok = true;
    for (int64_t gst = q; gst < total && ok; gst += 2 * kDepth) {
#pragma unroll
      for (int u = 0; u < kDepth; u++) {
        const int64_t my = gst + 2 * u;
        if (my < total && ok) {
          if (cur.ti != up_tile) {
            // the row's power of two comes from the scouts, who run ahead of the tile being filled
            const int slot = static_cast<int>(cur.ti & (kRowSlots - 1));
            if (!mbar_wait(&rowfull[slot], static_cast<uint32_t>((cur.ti / kRowSlots) & 1), abort_flag, 7)) { ok = false; }
            up = rowup[slot * TM + p];
            up_tile = cur.ti;
          }
          const int s = static_cast<int>(my % STAGES);
          if (ok && my >= STAGES && !mbar_wait(&empty[s], static_cast<uint32_t>(((my / STAGES) & 1) ^ 1), abort_flag, 1)) ok = false;
          ok = __all_sync(0xFFFFFFFFu, ok);      // the tensor-memory stores below are warp-wide: all lanes or none
          if (ok) {
            // stage s: columns [0, 32) piece 1, [32, 64) piece 2; word slot q in columns 16 q .. 16 q + 15 of its piece
            const uint32_t a_col = tmem_base + t_lane + S::A_BASE + static_cast<uint32_t>(s) * S::A_COLS;
            if (ASUB > 1 && staged) {
              // this row's 2 ASUB scales of the stage, from the block the loader's tensor copy laid down
              const int ss = static_cast<int>(my % SR::NS);
              if (!mbar_wait(&sfull[ss], static_cast<uint32_t>((my / SR::NS) & 1), abort_flag, 9)) ok = false;
              ok = __all_sync(0xFFFFFFFFu, ok);
              if (!ok) break;
              const unsigned char* blk = smem + SR::OFF + ss * SR::STAGE;
#pragma unroll
              for (int c = 0; c < (2 * ASUB) / 4; c++) {
                const float4 v = *reinterpret_cast<const float4*>(blk + SR::piece(p, c));
                sc[u][4 * c] = v.x; sc[u][4 * c + 1] = v.y; sc[u][4 * c + 2] = v.z; sc[u][4 * c + 3] = v.w;
              }
            }
#pragma unroll
            for (int qw = 0; qw < WPS; qw++) {
              uint32_t p1[16], p2[16];
              const uint32_t word = qw == 0 ? w[u].x : w[u].y;
              if (ASUB == 1) {
                expand_word_regs(word, sc[u][qw * ASUB] * up, p1, p2);
              } else {
                constexpr int SB = ASUB > 1 ? ASUB : 2;
                float sw[SB];
#pragma unroll
                for (int i = 0; i < ASUB; i++) sw[i] = sc[u][qw * ASUB + i] * up;
                expand_word_sub_regs<SB>(word, sw, p1, p2);
              }
              tmem_st16(a_col + qw * 16, p1);
              tmem_st16(a_col + KB / 2 + qw * 16, p2);
            }
            tmem_st_wait();               // the pieces are in tensor memory ...
            tc_fence_before();            // ... before the arrival that lets the MMA read them
            __syncwarp();
            if (lane == 0) mbar_arrive(&full[s]);
            fetch(pf, w[u], sc[u]);         // this register slot is free again: load kDepth of my stages ahead
            advance(pf);
            advance(cur);
          }
        }
      }
    }
  } else if (warp >= kFirstScoutWarp) {
    // =========================== scouts ===========================
    // One thread per tile row finds the row's largest scale and stores the two powers of two, up to
    // kRowSlots tiles ahead of the epilogue.
    const int p0 = tid - kFirstScoutWarp * 32;
    for (int64_t ti = 0; ti < my_tiles; ti++) {
      const int slot = static_cast<int>(ti & (kRowSlots - 1));
      if (ti >= kRowSlots && !mbar_wait(&rowempty[slot], static_cast<uint32_t>(((ti / kRowSlots) & 1) ^ 1), abort_flag, 8)) break;
      const int64_t tile = seg_tile(ti);
      if (ASUB > 1 && g.a_rowmax) {
        // long rows of scales: a kernel of its own has reduced every row to its largest scale
        const int64_t ma = (tile / tiles_n) * TM + p0, mb = ma + kScoutWarps * 32;
        float up = 0.0f, down = 1.0f;
        if (ma < g.M) norm_factors(__ldg(g.a_rowmax + ma), up, down);
        rowup[slot * TM + p0] = up;
        rowdown[slot * TM + p0] = down;
        up = 0.0f; down = 1.0f;
        if (mb < g.M) norm_factors(__ldg(g.a_rowmax + mb), up, down);
        rowup[slot * TM + p0 + kScoutWarps * 32] = up;
        rowdown[slot * TM + p0 + kScoutWarps * 32] = down;
      } else {
        // rows p0 and p0 + 64, scanned together so that both rows' loads are in flight at once
        const int64_t ma = (tile / tiles_n) * TM + p0, mb = ma + kScoutWarps * 32;
        float xa, xb;
        row_max_scale2(g.a_scales, g.a_bf16, (ma < g.M ? ma : 0) * g.lda_s, (mb < g.M ? mb : 0) * g.lda_s, g.lda_s, xa, xb);
        float up = 0.0f, down = 1.0f;
        if (ma < g.M) norm_factors(xa, up, down);
        rowup[slot * TM + p0] = up;
        rowdown[slot * TM + p0] = down;
        up = 0.0f; down = 1.0f;
        if (mb < g.M) norm_factors(xb, up, down);
        rowup[slot * TM + p0 + kScoutWarps * 32] = up;
        rowdown[slot * TM + p0 + kScoutWarps * 32] = down;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&rowfull[slot]);
    }
  } else if (warp == kLoaderWarp) {
    // =========================== W loader ===========================
    if (lane == 0) {
      int64_t gst = 0;
      bool ok = true;
      // sub-word groups: the next scale block to request -- [128 rows][2 ASUB scales] of one stage; rows past M and groups
      // past the last one arrive as zeros
      int64_t sc_ti = 0, sc_st = seg_begin(0), sc_g = 0;
      auto issue_scales = [&]() {
        const int slot = static_cast<int>(sc_g % SR::NS);
        mbar_arrive_expect_tx(&sfull[slot], SR::STAGE);
        tma_load_2d(smem + SR::OFF + slot * SR::STAGE, &s_map, static_cast<int32_t>(sc_st * (2 * ASUB)),
                    static_cast<int32_t>((seg_tile(sc_ti) / tiles_n) * TM), &sfull[slot]);
        sc_g++;
        if (++sc_st >= seg_end(sc_ti)) { sc_ti++; sc_st = seg_begin(sc_ti); }
      };
      if (ASUB > 1 && staged)
        for (int i = 0; i < SR::LEAD && sc_g < my_stages; i++) issue_scales();
      for (int64_t ti = 0; ti < my_tiles && ok; ti++) {
        const int64_t tile = seg_tile(ti);
        const unsigned char* src = g.w_prep + (tile % tiles_n) * n_stages * S::B_STAGE;
        const int64_t st_end = seg_end(ti);
        for (int64_t st = seg_begin(ti); st < st_end; st++, gst++) {
          const int s = static_cast<int>(gst % STAGES);
          if (gst >= STAGES && !mbar_wait(&empty[s], static_cast<uint32_t>(((gst / STAGES) & 1) ^ 1), abort_flag, 6)) { ok = false; break; }
          mbar_arrive_expect_tx(&full[s], S::B_STAGE);
          bulk_copy_g2s(smem + S::OFF_B + s * S::B_STAGE, src + st * S::B_STAGE, S::B_STAGE, &full[s]);
          if (ASUB > 1 && staged && sc_g < my_stages) issue_scales();      // the block of stage gst + LEAD
        }
      }
      if (!ok || *abort_flag) {
        if (ASUB > 1 && staged) {
          const int64_t pend = sc_g < SR::NS ? sc_g : SR::NS;
          for (int64_t q = 1; q <= pend; q++) {
            const int64_t idx = sc_g - q;
            mbar_wait_quiet(&sfull[idx % SR::NS], static_cast<uint32_t>((idx / SR::NS) & 1), kDrainPolls);
          }
        }
        // aborted: the copies already issued (at most one per stage) must land before the CTA's shared memory
        // goes away.  Their barriers also count producer arrivals that may never come, so each wait is a
        // short bounded one that ignores the abort flag: it ends when the phase completes or after a time
        // that is long next to a copy.
        const int64_t pending = gst < STAGES ? gst : STAGES;
        for (int64_t q = 1; q <= pending; q++) {
          const int64_t idx = gst - q;
          mbar_wait_quiet(&full[idx % STAGES], static_cast<uint32_t>((idx / STAGES) & 1), kDrainPolls);
        }
      }
    }
    __syncwarp();
  } else if (warp == kMmaWarp) {
    // =========================== MMA issuer ===========================
    // The whole warp walks the loop so that ring indices and descriptors stay warp-uniform values; one
    // lane issues the MMAs and commits.
    {
      constexpr uint32_t idesc = instr_desc(TN, kFmtF16);
      constexpr uint32_t idesc2 = instr_desc(2 * TN, kFmtF16);     // stacked: both weight pieces in one instruction
      const uint64_t db0 = smem_desc(smem_u32(smem + S::OFF_B));
      const uint64_t db_hi = db0 & 0xFFFFFFFF00000000ull;
      const uint32_t db_lo = static_cast<uint32_t>(db0);
      const uint32_t full_a = smem_u32(full), empty_a = smem_u32(empty), tfull_a = smem_u32(tfull), tempty_a = smem_u32(tempty);
      const bool leader = lane == 0;
      uint32_t s = 0, full_par = 0;
      bool ok = true;
      for (int64_t ti = 0; ti < my_tiles && ok; ti++) {
        const uint32_t buf = static_cast<uint32_t>(ti & 1);
        if (ti >= 2) {      // the epilogue must have drained this accumulator (used by tile ti - 2)
          if (!mbar_wait_a(tempty_a + buf * 8, static_cast<uint32_t>(((ti >> 1) & 1) ^ 1), abort_flag, 3)) { ok = false; break; }
          tc_fence_after();
        }
        const uint32_t d_tmem = tmem_base + buf * S::ACC_COLS;
        const uint32_t n_st = static_cast<uint32_t>(seg_end(ti) - seg_begin(ti));      // the segment starts a fresh accumulation
        for (uint32_t st = 0; st < n_st; st++) {
          if (!mbar_wait_a(full_a + s * 8, full_par, abort_flag, 2)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a1 = tmem_base + S::A_BASE + s * S::A_COLS, a2 = a1 + KB / 2;
          const uint32_t b1_lo = db_lo + s * (S::B_STAGE >> 4), b2_lo = b1_lo + (S::B_PIECE >> 4);
          if (leader) {
#pragma unroll
            for (int ks = 0; ks < KB / 16; ks++) {        // 16 K-elements = 8 TMEM columns of A, 32 bytes along the swizzled rows of W
              if constexpr (S::STACKED) {
                umma_f16_ts(d_tmem, a1 + ks * 8, db_hi | (b1_lo + ks * 2), idesc2, (st | ks) != 0 ? 1u : 0u);   // A1 [W1; W2]
                umma_f16_ts(d_tmem, a2 + ks * 8, db_hi | (b1_lo + ks * 2), idesc, 1u);                           // A2 W1
              } else {
                umma_f16_ts(d_tmem, a1 + ks * 8, db_hi | (b1_lo + ks * 2), idesc, (st | ks) != 0 ? 1u : 0u);
                umma_f16_ts(d_tmem, a2 + ks * 8, db_hi | (b1_lo + ks * 2), idesc, 1u);
                umma_f16_ts(d_tmem, a1 + ks * 8, db_hi | (b2_lo + ks * 2), idesc, 1u);
              }
            }
            umma_commit_a(empty_a + s * 8);     // the stage (TMEM columns and W bytes) is free once these MMAs have read it
          }
          __syncwarp();
          if (++s == STAGES) { s = 0; full_par ^= 1; }
        }
        if (ok && leader) umma_commit_a(tfull_a + buf * 8);
        __syncwarp();
      }
      if (leader) {
        // every MMA issued so far has retired before TMEM is released -- also after an abort, so this wait
        // does not look at the abort flag (the commit arrives once the tensor core is done, whatever the
        // other warps do)
        umma_commit(drain);
        if (!mbar_wait_quiet(drain, 0, g_spin_limit < kDrainPolls ? kDrainPolls : g_spin_limit)) {
          atomicCAS(&g_error_word, 0, 4);
          *abort_flag = 1;
        }
      }
    }
    __syncwarp();
  } else if (warp < kEpilogueWarps) {
    // =========================== epilogue ===========================
    const int row = warp * 32 + lane;               // TMEM lane = tile row
    const uint32_t t_lane = static_cast<uint32_t>(warp * 32) << 16;
    for (int64_t ti = 0; ti < my_tiles; ti++) {
      const uint32_t buf = static_cast<uint32_t>(ti & 1);
      const int slot = static_cast<int>(ti & (kRowSlots - 1));
      const int64_t tile = seg_tile(ti);
      const int64_t m = (tile / tiles_n) * TM + row, nb = (tile % tiles_n) * TN;
      // the tile's column factors go through shared memory (one copy per warp, so no warp waits for
      // another): requested before the wait for the accumulator, read back as broadcasts
      float fcol[TN / 32], fsc[TN / 32], fsh[TN / 32];
#pragma unroll
      for (int i = 0; i < TN / 32; i++) {
        const int64_t n = nb + i * 32 + lane;
        fcol[i] = __ldg(g.w_down + n);                                                     // w_down holds a whole number of tiles
        fsc[i] = (FUSE && g.ep.bn_scale && n < g.N) ? __ldg(g.ep.bn_scale + n) : 1.0f;
        fsh[i] = (FUSE && g.ep.bn_shift && n < g.N) ? __ldg(g.ep.bn_shift + n) : 0.0f;
      }
      if (!mbar_wait(&tfull[buf], static_cast<uint32_t>((ti >> 1) & 1), abort_flag, 5)) break;
      if (!mbar_wait(&rowfull[slot], static_cast<uint32_t>((ti / kRowSlots) & 1), abort_flag, 5)) break;   // long complete
      tc_fence_after();
      const float fa = rowdown[slot * TM + row];
      float* cf = colf + warp * (3 * TN);
#pragma unroll
      for (int i = 0; i < TN / 32; i++) {
        cf[i * 32 + lane] = fcol[i];
        if (FUSE) {
          cf[TN + i * 32 + lane] = fsc[i];
          cf[2 * TN + i * 32 + lane] = fsh[i];
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&rowempty[slot]);
      float* dst = g.C + m * g.ldc + nb;
      float carry = 0.0f;                                   // |z| sum of a group wider than a 32-column chunk
      // raw accumulator of chunk c (32 columns of this thread's row): the two stacked blocks added for the narrow tile
      auto load_chunk = [&](int c, uint32_t (&v1)[32]) {
        const uint32_t t_addr = tmem_base + t_lane + buf * S::ACC_COLS + c * 32;
        tmem_ld32(t_addr, v1);
        if constexpr (S::STACKED) {      // the A1 W2 block sits TN columns further on
          uint32_t v2[32];
          tmem_ld32(t_addr + TN, v2);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; j++) v1[j] = __float_as_uint(__uint_as_float(v1[j]) + __uint_as_float(v2[j]));
        } else {
          tmem_ld_wait();
        }
      };
      // the tile's complete accumulator values of chunk c -> the output (powers of two divided out; epilogue chain or fp32 store)
      auto finish = [&](int c, const uint32_t (&v1)[32]) {
        if constexpr (FUSE) {
          if (m < g.M) {
            // the product of the chunk's 32 columns, then activation, affine map and dense or binarized output
            float cv[32], fs[32], fh[32];
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const float4 fw = *reinterpret_cast<const float4*>(cf + c * 32 + j);
              const float4 bs = *reinterpret_cast<const float4*>(cf + TN + c * 32 + j);
              const float4 bh = *reinterpret_cast<const float4*>(cf + 2 * TN + c * 32 + j);
              const float w4[4] = {fw.x, fw.y, fw.z, fw.w}, s4[4] = {bs.x, bs.y, bs.z, bs.w}, h4[4] = {bh.x, bh.y, bh.z, bh.w};
#pragma unroll
              for (int e = 0; e < 4; e++) {
                cv[j + e] = __uint_as_float(v1[j + e]) * fa * w4[e];
                fs[j + e] = s4[e];
                fh[j + e] = h4[e];
              }
            }
            epi::finish_chunk(g.ep, cv, fs, fh, m, nb + c * 32, g.N, c == TN / 32 - 1, nb + TN, carry);
          }
        } else if (m < g.M) {
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float4 fw = *reinterpret_cast<const float4*>(cf + c * 32 + j);
            float o[4];
#pragma unroll
            for (int e = 0; e < 4; e++) o[e] = __uint_as_float(v1[j + e]) * fa;
            o[0] *= fw.x; o[1] *= fw.y; o[2] *= fw.z; o[3] *= fw.w;
            const int64_t n = nb + c * 32 + j;
            if (n + 3 < g.N) *reinterpret_cast<float4*>(dst + c * 32 + j) = make_float4(o[0], o[1], o[2], o[3]);
            else
              for (int e = 0; e < 4; e++)
                if (n + e < g.N) dst[c * 32 + j + e] = o[e];
          }
        }
      };
      const bool whole = !BAL || (seg_begin(ti) == 0 && seg_end(ti) == n_stages);
      if (whole) {
#pragma unroll
        for (int c = 0; c < TN / 32; c++) {
          uint32_t v1[32];
          load_chunk(c, v1);
          finish(c, v1);
        }
        tc_fence_before();
        __syncwarp();          // also: every lane is done with the warp's column factors
        if (lane == 0) mbar_arrive(&tempty[buf]);
      } else if constexpr (BAL) {
        // Part of the tile's K range: the raw partial accumulator goes to this CTA's slot (first slot for the tile
        // its run starts in, second for the tile it ends in), the accumulator is handed back, and the warp
        // counts itself in.  Whoever arrives last adds the tile's partials in CTA order -- the same sum whoever
        // that is -- and finishes the rows.  Nobody waits for anybody.
        // slot layout [column][row]: a warp's store of one column is 32 consecutive floats
        float* slot = g.sk_partials + static_cast<int64_t>(2 * blockIdx.x + (seg_nat(ti) == 0 ? 0 : 1)) * (TM * TN) + row;
#pragma unroll
        for (int c = 0; c < TN / 32; c++) {
          uint32_t v1[32];
          load_chunk(c, v1);
#pragma unroll
          for (int j = 0; j < 32; j++) __stcg(slot + (c * 32 + j) * TM, __uint_as_float(v1[j]));
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty[buf]);
        __threadfence();       // the partial is visible device-wide before the count says so
        __syncwarp();
        const int64_t c_first = (tile * n_stages) / g.sk_units, c_last = ((tile + 1) * n_stages - 1) / g.sk_units;
        int arrived = 0;
        if (lane == 0) arrived = atomicAdd(g.sk_counters + tile * kEpilogueWarps + warp, 1);
        arrived = __shfl_sync(0xFFFFFFFFu, arrived, 0);
        if (arrived == static_cast<int>(c_last - c_first)) {
          __threadfence();
#pragma unroll 1
          for (int c = 0; c < TN / 32; c++) {
            uint32_t v1[32];
#pragma unroll
            for (int j = 0; j < 32; j++) v1[j] = 0u;                 // +0.0f
            for (int64_t cc = c_first; cc <= c_last; cc++) {
              const int64_t first_tile_of_cc = (cc * g.sk_units) / n_stages;
              const float* src = g.sk_partials + (2 * cc + (first_tile_of_cc == tile ? 0 : 1)) * (TM * TN) + (c * 32) * TM + row;
#pragma unroll
              for (int j = 0; j < 32; j++) v1[j] = __float_as_uint(__uint_as_float(v1[j]) + __ldcg(src + j * TM));
            }
            finish(c, v1);
          }
          if (lane == 0) g.sk_counters[tile * kEpilogueWarps + warp] = 0;      // as the next launch expects to find it
        }
        __syncwarp();          // every lane is done with the warp's column factors
      }

    }
  }

  // ---- teardown: everyone meets here (aborted threads too), then the allocating warp frees TMEM
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, S::TMEM_COLS);
  }
}

// Test only: thread 0 waits, with the bounded wait every role of the kernel above uses, on a barrier that
// nobody arrives at and that guards nothing (no copy, no MMA in flight).  The wait runs out after the
// limit in force, records code 9 and raises the abort flag, which the other threads then see.
__global__ void wait_expiry_selftest_kernel(int* saw_abort) {
  __shared__ uint64_t bar;
  __shared__ int flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  volatile int* abort_flag = &flag;
  bool done = true;
  if (threadIdx.x == 0) done = mbar_wait(&bar, 0, abort_flag, 9);
  __syncthreads();
  if (threadIdx.x == 1 && saw_abort) *saw_abort = (*abort_flag != 0 && done) ? 1 : 0;
}

Args make_args(const PackedView& A, const PackedView& W, float* C, int64_t ldc) {
  Args g;
  g.a_bits = A.bits; g.a_scales = A.scales; g.w_bits = W.bits; g.w_scales = W.scales; g.C = C;
  g.M = A.rows; g.N = W.rows; g.lda_w = A.ld_words; g.ldw_w = W.ld_words; g.lda_s = A.ld_scales; g.ldw_s = W.ld_scales;
  g.ldc = ldc; g.a_bf16 = A.scale_bf16; g.w_bf16 = W.scale_bf16;
  g.n_words = A.K / 32;
  const bool a_subword = A.beta < 32 && A.beta < A.K, w_subword = W.beta < 32 && W.beta < W.K;
  g.a_sub = a_subword ? 32 / A.beta : 1;
  g.w_sub = w_subword ? 32 / W.beta : 1;
  g.a_gw = A.beta >= A.K ? g.n_words : (a_subword ? 1 : A.beta / 32);
  g.w_gw = W.beta >= W.K ? g.n_words : (w_subword ? 1 : W.beta / 32);
  g.w_prep = nullptr;
  g.w_down = nullptr;
  g.ep = plain_epilogue();
  g.sk_units = 0; g.sk_counters = nullptr; g.sk_counter_count = 0; g.sk_partials = nullptr;
  g.a_staged = 0; g.a_rowmax = nullptr;
  return g;
}

template <int TN>
size_t stage_bytes(const Args& g) {
  const int64_t tiles_n = (g.N + TN - 1) / TN, n_stages = (g.n_words + WPS - 1) / WPS;
  return static_cast<size_t>(tiles_n * n_stages) * Smem<TN>::B_STAGE;
}
// Balanced schedule: worth its reduction traffic when the tiles are few waves of the machine and a tile's K walk is
// long enough to cut.  The workspace is sized for any device of up to kMaxBalancedCtas multiprocessors.
constexpr int64_t kMaxBalancedCtas = 256;
constexpr int64_t kBalancedWaves = 4;
constexpr int64_t kBalancedMinStages = 4;
constexpr int64_t kBalancedMaxShare = 4;
template <int TN>
int64_t tile_count(const Args& g) { return ((g.M + TM - 1) / TM) * ((g.N + TN - 1) / TN); }
template <int TN>
bool balanced_possible(const Args& g, int64_t sms) {
  const int64_t n_stages = (g.n_words + WPS - 1) / WPS;
  return sms <= kMaxBalancedCtas && n_stages >= kBalancedMinStages && tile_count<TN>(g) < kBalancedWaves * sms;
}
template <int TN>
size_t counters_bytes(const Args& g) { return (static_cast<size_t>(tile_count<TN>(g)) * kEpilogueWarps * sizeof(int32_t) + 255) / 256 * 256; }
template <int TN>
size_t balanced_bytes(const Args& g) {
  if (!balanced_possible<TN>(g, kMaxBalancedCtas)) return 0;
  const int64_t n_stages = (g.n_words + WPS - 1) / WPS, units = tile_count<TN>(g) * n_stages;
  const int64_t ctas = units < kMaxBalancedCtas ? units : kMaxBalancedCtas;
  return counters_bytes<TN>(g) + static_cast<size_t>(2 * ctas) * TM * TN * sizeof(float);
}
// [W stages][one float per weight row][counters][partial slots]
template <int TN>
size_t down_offset(const Args& g) { return stage_bytes<TN>(g); }
template <int TN>
size_t balanced_offset(const Args& g) {
  return (stage_bytes<TN>(g) + static_cast<size_t>((g.N + TN - 1) / TN) * TN * sizeof(float) + 255) / 256 * 256;
}
// ... then, for activation groups shorter than a word, one float per activation row (its largest scale)
template <int TN>
size_t rowmax_offset(const Args& g) { return (balanced_offset<TN>(g) + balanced_bytes<TN>(g) + 255) / 256 * 256; }
template <int TN>
size_t prep_bytes(const Args& g) {
  return g.a_sub > 1 ? rowmax_offset<TN>(g) + static_cast<size_t>(g.M) * sizeof(float) : balanced_offset<TN>(g) + balanced_bytes<TN>(g);
}
// Points the argument block at the balanced schedule's part of the workspace (when the shape has one).
template <int TN>
void set_balanced_area(Args& g, void* workspace) {
  if (balanced_bytes<TN>(g) == 0) return;
  unsigned char* area = static_cast<unsigned char*>(workspace) + balanced_offset<TN>(g);
  g.sk_counters = reinterpret_cast<int32_t*>(area);
  g.sk_counter_count = tile_count<TN>(g) * kEpilogueWarps;
  g.sk_partials = reinterpret_cast<float*>(area + counters_bytes<TN>(g));
}

template <int TN, int ASUB, bool FUSE = false>
cudaError_t launch_fold(Args g, void* workspace, cudaStream_t stream, bool w_prepared) {
  using S = Smem<TN>;
  constexpr bool kHasBalanced = ASUB == 1;           // the balanced schedule is built for activation groups of whole words
  constexpr int kBytes = ScaleRing<TN, ASUB>::BYTES;
  static_assert(kBytes <= 227 * 1024, "weight stages and the scale ring fit one CTA's shared memory");
  static DeviceOnce configured;
  int dev = 0, sms = 0;
  if (current_device(&dev, &sms) != cudaSuccess) return cudaErrorInvalidDevice;
  if (configured.pending(dev)) {
    cudaError_t e = cudaFuncSetAttribute(hbmm_fold_kernel<TN, ASUB, FUSE, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kBytes);
    if (e != cudaSuccess) return e;
    if (kHasBalanced) {
      e = cudaFuncSetAttribute(hbmm_fold_kernel<TN, ASUB, FUSE, kHasBalanced>, cudaFuncAttributeMaxDynamicSharedMemorySize, kBytes);
      if (e != cudaSuccess) return e;
    }
    configured.mark(dev);
  }
  const int64_t tiles_n = (g.N + TN - 1) / TN, n_stages = (g.n_words + WPS - 1) / WPS;
  unsigned char* stages = static_cast<unsigned char*>(workspace);
  float* down = reinterpret_cast<float*>(stages + stage_bytes<TN>(g));
  set_balanced_area<TN>(g, workspace);
  if (!w_prepared) {
    dim3 pgrid(static_cast<unsigned>((n_stages + kPrepStages - 1) / kPrepStages), static_cast<unsigned>(tiles_n));
    prepare_w_fold_kernel<TN><<<pgrid, TN, 0, stream>>>(g, stages, down);
  }
  g.w_prep = stages;
  g.w_down = down;
  // sub-word groups: the activation scales as a 2-D tensor [M][lda_s] of fp32 for the per-stage block copies
  CUtensorMap s_map = {};
  g.a_staged = 0;
  if (ASUB >= kStagedFrom && !g.a_bf16 && reinterpret_cast<uintptr_t>(g.a_scales) % 16 == 0 && g.lda_s % 4 == 0 &&
      g.lda_s < (int64_t{1} << 31) && g.M < (int64_t{1} << 31)) {
    if (EncodeTiledFn fn = encode_tiled_fn()) {
      const cuuint64_t dims[2] = {static_cast<cuuint64_t>(g.lda_s), static_cast<cuuint64_t>(g.M)};
      const cuuint64_t strides[1] = {static_cast<cuuint64_t>(g.lda_s) * 4};
      const cuuint32_t box[2] = {2 * ASUB, TM};
      const cuuint32_t elem[2] = {1, 1};
      const CUtensorMapSwizzle swz_mode = ASUB == 16 ? CU_TENSOR_MAP_SWIZZLE_128B : (ASUB == 8 ? CU_TENSOR_MAP_SWIZZLE_64B
                                          : (ASUB == 4 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE));
      if (fn(&s_map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(g.a_scales), dims, strides, box, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, swz_mode, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
        g.a_staged = 1;
    }
  }
  g.a_rowmax = nullptr;
  if (ASUB > 1 && !g.a_bf16 && g.lda_s % 4 == 0 && g.lda_s >= kRowMaxFrom && reinterpret_cast<uintptr_t>(g.a_scales) % 16 == 0) {
    // many scales per row: reduce the rows to their largest scale in a kernel of its own, at streaming bandwidth
    g.a_rowmax = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + rowmax_offset<TN>(g));
    const cudaError_t e = launch_pdl(row_max_kernel, dim3(static_cast<unsigned>((g.M + 7) / 8)), dim3(256), 0, stream,
                                     reinterpret_cast<const float*>(g.a_scales), g.lda_s, g.M, g.a_rowmax);
    if (e != cudaSuccess) return e;
  }
  const int64_t tiles = ((g.M + TM - 1) / TM) * tiles_n;
  // equal runs of (tile, stage) pairs, one per CTA, when that shortens the longest CTA's walk by a tenth or more
  const int64_t units = tiles * n_stages;
  int64_t ctas = units / kBalancedMinStages < sms ? units / kBalancedMinStages : sms;
  if (ctas < 1) ctas = 1;
  int64_t run = (units + ctas - 1) / ctas;
  // a tile is shared by at most kBalancedMaxShare + 1 CTAs: the CTA that completes it adds the others' partial
  // accumulators one after the other, which costs more than the shorter walk saves beyond that
  const int64_t min_run = (n_stages + kBalancedMaxShare - 1) / kBalancedMaxShare;
  if (run < min_run) run = min_run;
  const int64_t plain_walk = ((tiles + sms - 1) / sms) * n_stages;
  if (kHasBalanced && balanced_possible<TN>(g, sms) && run * 10 <= plain_walk * 9) {
    ctas = (units + run - 1) / run;                     // no CTA without work
    g.sk_units = run;
    return launch_pdl(hbmm_fold_kernel<TN, ASUB, FUSE, kHasBalanced>, dim3(static_cast<unsigned>(ctas)), dim3(kThreads), kBytes, stream, g, s_map);
  }
  const unsigned grid = static_cast<unsigned>(tiles < sms ? tiles : sms);   // one persistent CTA per SM
  return launch_pdl(hbmm_fold_kernel<TN, ASUB, FUSE, false>, dim3(grid), dim3(kThreads), kBytes, stream, g, s_map);
}

template <int TN>
cudaError_t launch_fold_tn(const Args& g, void* workspace, cudaStream_t stream, bool w_prepared) {
  if (g.ep.mode != kEpiPlain) {      // the fused epilogue is built for activation groups of whole words
    if (g.a_sub != 1) return cudaErrorNotSupported;
    return launch_fold<TN, 1, true>(g, workspace, stream, w_prepared);
  }
  switch (g.a_sub) {
    case 2: return launch_fold<TN, 2>(g, workspace, stream, w_prepared);
    case 4: return launch_fold<TN, 4>(g, workspace, stream, w_prepared);
    case 8: return launch_fold<TN, 8>(g, workspace, stream, w_prepared);
    case 16: return launch_fold<TN, 16>(g, workspace, stream, w_prepared);
    default: return launch_fold<TN, 1>(g, workspace, stream, w_prepared);
  }
}

}  // namespace

// K a multiple of 32; scale groups of whole words, one group per row, or the sub-word groups 2, 4, 8, 16.
bool gemm_fold_supported(const PackedView& A, const PackedView& W) {
  if (A.K % 32 != 0 || A.K / 32 >= (int64_t{1} << 31)) return false;
  auto ok = [](const PackedView& v) {
    return v.beta >= v.K || v.beta % 32 == 0 || v.beta == 2 || v.beta == 4 || v.beta == 8 || v.beta == 16;
  };
  return ok(A) && ok(W);
}

// Bytes of workspace: the weight operand as fp16 piece tiles (4 bytes per element) + one float per row.
size_t gemm_fold_workspace_bytes(const PackedView& A, const PackedView& W) {
  const Args g = make_args(A, W, nullptr, 0);
  return g.N <= 64 ? prep_bytes<64>(g) : prep_bytes<128>(g);
}

// workspace: device, 16-byte aligned, at least gemm_fold_workspace_bytes.
// The fused epilogue closes a group inside one thread's row of a tile: the group must divide the tile width.
bool gemm_fold_next_supported(int64_t N, int32_t beta_next) {
  const int tn = N <= 64 ? 64 : 128;
  return (beta_next == 2 || beta_next == 4 || beta_next == 8 || beta_next == 16 || beta_next == 32 || beta_next == 64 ||
          beta_next == 128) && beta_next <= tn;
}

cudaError_t launch_gemm_fold(const PackedView& A, const PackedView& W, float* C, int64_t ldc, void* workspace,
                             cudaStream_t stream, bool w_prepared, const EpiArgs* ep) {
  Args g = make_args(A, W, C, ldc);
  if (ep) g.ep = *ep;
  return g.N <= 64 ? launch_fold_tn<64>(g, workspace, stream, w_prepared) : launch_fold_tn<128>(g, workspace, stream, w_prepared);
}

// The weight expansion of launch_gemm_fold(A, W, ..., workspace) as a job for another kernel.
void gemm_fold_prep_job(const PackedView& A, const PackedView& W, void* workspace, UmmaPrepJob* job) {
  job->f = make_args(A, W, nullptr, 0);
  job->folded = 1;
  job->out = static_cast<unsigned char*>(workspace);
  job->tn = job->f.N <= 64 ? 64 : 128;
  const int64_t n_stages = (job->f.n_words + WPS - 1) / WPS;
  job->n_stages = static_cast<int32_t>((n_stages + kPrepStages - 1) / kPrepStages);    // tasks per column tile
  job->tiles_n = static_cast<int32_t>((job->f.N + job->tn - 1) / job->tn);
  job->out_down = reinterpret_cast<float*>(job->out + (job->tn == 64 ? stage_bytes<64>(job->f) : stage_bytes<128>(job->f)));
  if (job->tn == 64) set_balanced_area<64>(job->f, workspace); else set_balanced_area<128>(job->f, workspace);
}

cudaError_t launch_wait_expiry_selftest(cudaStream_t stream) {
  wait_expiry_selftest_kernel<<<1, 32, 0, stream>>>(nullptr);
  return cudaGetLastError();
}

cudaError_t gemm_fold_health(int op, int* value) {
  switch (op) {
    case kHealthRead: return umma::read_error_word(value);
    case kHealthClear: return umma::clear_error_word();
    case kHealthSetSpinLimit: return umma::set_spin_limit(static_cast<uint32_t>(*value));
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace hbmm
