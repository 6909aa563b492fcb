// HBWN contraction on the 5th-generation tensor cores: bf16 activations x Hadamard-binary weights,
//   C[m,n] = sum_k A[m,k] * (deltaW[n, k/beta] * s(W[n,k])).
// The binarized weight W~ = deltaW (.) Sign(W) (Eq. 2) is written as the sum of three bf16 matrices:
// each fp32 group scale is split as delta = d1 + d2 + d3 (bf16 pieces, 24 significant bits together,
// every remainder exact in fp32) and piece i of W~ is +-d_i.  A bf16 activation times a bf16 piece
// is exact in fp32, so C = A W1^T + A W2^T + A W3^T accumulated in fp32 tensor memory reproduces the
// per-group full-precision scaling to 2^-26 of each weight -- with no per-group epilogue at all: the
// whole K walk of a tile is one accumulation in TMEM and the epilogue runs once per tile.
// The three pieces of a 64-column tile are stacked along N, so one 128 x 192 x 16 MMA per K-step
// forms all three products; the epilogue adds the three column blocks.
// The default variant keeps two pieces (delta = d1 + d2 to 2^-17, still far finer than the 2^-9 of a bf16
// activation) and 128-column tiles: one 128 x 256 x 16 MMA per K-step.  The kernel is bound by
// shared-memory traffic (operand reads of the tensor core plus the copies that fill the stages), and that
// variant moves 24 KB instead of 40 KB per 128 x 128 outputs and K-step.
//
// One persistent CTA per SM.  Stage = 64 K-elements: the A tile (128 rows x 128 bytes) arrives by
// one tiled tensor copy (TMA, 128-byte swizzle, zeros past M and K), the three weight pieces of the
// stage (192 rows) by one bulk copy from the workspace, where a small kernel has laid them out once
// per call.  All operand tiles use the 128-byte-swizzled K-major layout.
//   warps 0-3 : epilogue (TMEM lanes 32*w.., one block of TN columns per piece, once per tile)
//   warp  4   : one thread issues both copies of every stage
//   warp  5   : TMEM allocation and the MMA-issuing thread
// Waits are bounded as in the packed kernel (error word, CTA-wide abort flag, orderly teardown).
#include <cuda_bf16.h>
#include "kernels.h"
#include "tensor_map.h"
#include "nhwc.cuh"
#include "umma_common.cuh"
#include "epilogue.cuh"
#include "pdl.cuh"

namespace hbmm {
namespace {

using namespace umma;

constexpr int kThreads = 6 * 32;
constexpr int kLoaderWarp = 4, kMmaWarp = 5;
constexpr int KB = 64;            // K elements per stage (128 bytes of bf16 per row)

struct Args {
  const __nv_bfloat16* a; int64_t lda;
  const uint32_t* w_bits; const void* w_scales; int64_t ldw_w, ldw_s; int32_t w_bf16;
  float* C; int64_t ldc; int32_t c_vec;   // c_vec: rows of C allow 16-byte stores
  int64_t M, N, K, Gw;
  int64_t beta;                   // weight group length (>= K: one group per row)
  const unsigned char* w_prep;    // [n tile][k block][3 pieces][TN rows x 128 bytes]
  int64_t n_kb;                   // stages (K blocks of 64) per tile
  // Convolution mode (conv != 0): A is the implicit im2col matrix of an NHWC bf16 image; K block
  // kb = (filter tap, block of 64 channels), i.e. the K axis is walked tap-major.  Any one-to-one
  // reordering of K leaves the product unchanged as long as both operands use it: the weight pieces
  // are laid out in the same order, each element still scaled by the group of its original index
  // k = c * taps + tap (channel slowest, Section 3.1.1).
  int32_t conv, taps, kw, cblocks, Cin;
  int32_t HoWo, Wo, sh, sw, ph, pw;
  EpiArgs ep;                     // what the epilogue does with a finished tile (plain: store C as fp32)
};

__device__ __forceinline__ float load_scale(const void* s, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(s) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(s) + idx);
}

// TN: columns of the CTA tile.  NP: bf16 pieces per weight -- 3 carry the fp32 group scale to 2^-26 (64-column
// tiles: 192 stacked rows per MMA), 2 carry it to 2^-17 (128-column tiles: 256 stacked rows per MMA, which
// moves 40 % fewer shared-memory bytes per output, the resource that bounds this kernel).
template <int TN, int NP>
struct Smem {
  static constexpr int A_STAGE = TM * 128;
  static constexpr int B_PIECE = TN * 128;
  static constexpr int B_STAGE = NP * B_PIECE;
  static constexpr int STAGES = (200 * 1024) / (A_STAGE + B_STAGE);
  static constexpr int OFF_A = 0;
  static constexpr int OFF_B = OFF_A + STAGES * A_STAGE;
  static constexpr int OFF_BAR = OFF_B + STAGES * B_STAGE;
  static constexpr int NBAR = 2 * STAGES + 4 + 2;      // full, empty, tfull[2], tempty[2], drain, wfull
  static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
  static constexpr int USED = OFF_MISC + 16;
  static constexpr int BYTES = USED > 120 * 1024 ? USED : 120 * 1024;   // one CTA per SM
  static constexpr int NST = NP * TN;                  // MMA N: the pieces side by side
  static constexpr int TMEM_COLS = 512;                // two accumulator buffers of NST columns
  // Resident mode (one column tile whose weight pieces fit beside the activation ring): the pieces of all
  // K blocks are copied into shared memory once per CTA and only activation tiles stream afterwards.
  static constexpr int RES_STAGES = 4;
  static constexpr int RES_OFF_B = RES_STAGES * A_STAGE;
  static constexpr int RES_MAX_B = 225 * 1024 - RES_OFF_B - 512;        // bytes of weight pieces that fit
  static_assert(NST <= 256 && NST % 16 == 0 && 2 * NST <= TMEM_COLS, "one MMA covers the stacked pieces");
};

// Writes the NP bf16 pieces of W~ for one (column tile, k block): thread = (row, 16-byte piece of
// 8 consecutive stage columns).  Stage column q of block kb is element k = kb * 64 + q of the weight
// row (plain mode) or channel c = cb * 64 + q at filter tap t, k = c * taps + t (convolution mode,
// kb = t * cblocks + cb).  The element is +-piece_i(deltaW[n, k / beta]); zero past K / C and past N.
template <int TN, int NP>
__device__ __forceinline__ void prepare_w_pieces_block(const Args& g, unsigned char* __restrict__ out, int64_t kb, int64_t tile_n) {
  using S = Smem<TN, NP>;
  unsigned char* base = out + (tile_n * g.n_kb + kb) * S::B_STAGE;
  const int64_t tap = g.conv ? kb / g.cblocks : 0;
  const int64_t q0 = (g.conv ? kb - tap * g.cblocks : kb) * KB;     // first channel / element of the block
  const int64_t q_end = g.conv ? g.Cin : g.K, k_mul = g.conv ? g.taps : 1;
  for (int item = threadIdx.x; item < TN * 8; item += 256) {
    const int row = item >> 3, piece = item & 7;
    const int64_t n = tile_n * TN + row;
    uint32_t o[3][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}, {0, 0, 0, 0}};
    if (n < g.N) {
      // all sixteen loads of the piece are issued before the first use
      uint32_t word[8];
      float d[8];
      bool valid[8];
#pragma unroll
      for (int e = 0; e < 8; e++) {
        const int64_t q = q0 + piece * 8 + e;
        valid[e] = q < q_end;
        const int64_t k = valid[e] ? q * k_mul + tap : 0;
        word[e] = __ldg(g.w_bits + n * g.ldw_w + (k >> 5)) >> (k & 31);
        d[e] = load_scale(g.w_scales, g.w_bf16, n * g.ldw_s + (g.beta >= g.K ? 0 : k / g.beta));
      }
#pragma unroll
      for (int e = 0; e < 8; e++) {
        if (valid[e]) {
          const __nv_bfloat16 b1 = __float2bfloat16_rn(d[e]);
          const float r1 = d[e] - __bfloat162float(b1);
          const __nv_bfloat16 b2 = __float2bfloat16_rn(r1);
          const __nv_bfloat16 b3 = __float2bfloat16_rn(r1 - __bfloat162float(b2));
          const uint32_t neg = (word[e] & 1u) ? 0u : 0x8000u;   // bit 0 <=> Sign = -1
          const uint32_t h[3] = {__bfloat16_as_ushort(b1) ^ neg, __bfloat16_as_ushort(b2) ^ neg, __bfloat16_as_ushort(b3) ^ neg};
#pragma unroll
          for (int i = 0; i < NP; i++) o[i][e >> 1] |= h[i] << ((e & 1) * 16);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < NP; i++)
      *reinterpret_cast<uint4*>(swz(base + i * S::B_PIECE, row, piece)) = make_uint4(o[i][0], o[i][1], o[i][2], o[i][3]);
  }
}

template <int TN, int NP>
__global__ void __launch_bounds__(256)
prepare_w_pieces_kernel(const Args g, unsigned char* __restrict__ out) {
  prepare_w_pieces_block<TN, NP>(g, out, blockIdx.x, blockIdx.y);
}

// Convolution front end in one launch: the first `n_copy` blocks transpose the input to NHWC bf16, the
// rest lay out the weight pieces.  The two jobs are independent, so the small weight job hides behind
// the copy instead of costing a launch of its own.
struct CopyArgs {
  const void* x; int32_t x_bf16, C, Cp; int64_t HW; unsigned short* out;
  int32_t gx, gy;          // pixel blocks and channel blocks per image
  int32_t pb;              // pixels per block
  int64_t n_copy;
};
template <int TN, int NP, int PB>
__global__ void __launch_bounds__(256)
nhwc_and_pieces_kernel(const CopyArgs c, const Args g, unsigned char* __restrict__ w_out) {
  __shared__ unsigned short tile[kNhwcCB][nhwc_pitch(PB)];
  const int64_t blk = blockIdx.x;
  pdl_launch_dependents();
  pdl_wait();                   // the workspace may still be in use by the kernel before this one
  if (blk < c.n_copy) {
    const int64_t per_image = static_cast<int64_t>(c.gx) * c.gy;
    const int64_t b = blk / per_image, r = blk - b * per_image;
    const int cblock = static_cast<int>(r / c.gx);
    nchw_to_nhwc_block<PB>(c.x, c.x_bf16, c.C, c.HW, c.Cp, c.out, b, cblock, r - static_cast<int64_t>(cblock) * c.gx, tile);
  } else {
    const int64_t j = blk - c.n_copy;
    const int64_t tile_n = j / g.n_kb;
    prepare_w_pieces_block<TN, NP>(g, w_out, j - tile_n * g.n_kb, tile_n);
  }
}

template <int TN, int NP, bool RES>
__global__ void __launch_bounds__(kThreads, 1)
hbwn_umma_kernel(const Args g, const __grid_constant__ CUtensorMap a_map) {
  using S = Smem<TN, NP>;
  constexpr int STAGES = RES ? S::RES_STAGES : S::STAGES;
  extern __shared__ __align__(1024) unsigned char smem[];
  // resident mode: [activation ring][all weight pieces][barriers]; streaming mode: the static layout of Smem
  const int off_b = RES ? S::RES_OFF_B : S::OFF_B;
  const int off_bar = RES ? S::RES_OFF_B + static_cast<int>(g.n_kb) * S::B_STAGE : S::OFF_BAR;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + off_bar);
  uint64_t* empty = full + STAGES;
  uint64_t* tfull = empty + STAGES;
  uint64_t* tempty = tfull + 2;
  uint64_t* drain = tempty + 2;
  uint64_t* wfull = drain + 1;                            // resident mode: all weight pieces have arrived
  uint32_t* tmem_base_ptr = reinterpret_cast<uint32_t*>(wfull + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_ptr + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t tiles_n = (g.N + TN - 1) / TN, tiles_m = (g.M + TM - 1) / TM;
  const int64_t n_tiles = tiles_m * tiles_n;
  const int64_t n_kb = g.n_kb;                              // stages per tile
  const int64_t my_tiles = blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

  pdl_launch_dependents();      // the next kernel of the stream may start its own set-up
  if (tid == 0) {
    for (int s = 0; s < STAGES; s++) {
      mbar_init(&full[s], 1);           // the loader's expect_tx arrival; the copies complete the bytes
      mbar_init(&empty[s], 1);          // MMA commit
    }
    for (int b = 0; b < 2; b++) { mbar_init(&tfull[b], 1); mbar_init(&tempty[b], 4); }
    mbar_init(drain, 1);
    mbar_init(wfull, 1);
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

  if (warp == kLoaderWarp) {
    // =========================== loader ===========================
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&a_map) : "memory");
      // One thread feeds the whole CTA, so the loop carries its indices along instead of dividing:
      // ring slot and round, K block -> (filter tap row, column, channel block).
      int s = 0;
      uint32_t round = 0;
      int64_t issued = 0;                                       // stages handed to the copy engine so far
      bool ok = true;
      if (RES && my_tiles > 0) {
        // one column tile: its weight pieces are the same for every row tile of this CTA
        mbar_arrive_expect_tx(wfull, static_cast<uint32_t>(n_kb) * S::B_STAGE);
        for (int64_t kb = 0; kb < n_kb; kb++)
          bulk_copy_g2s(smem + off_b + kb * S::B_STAGE, g.w_prep + kb * S::B_STAGE, S::B_STAGE, wfull);
      }
      for (int64_t ti = 0; ti < my_tiles && ok; ti++) {
        const int64_t tile = blockIdx.x + ti * gridDim.x;
        const int64_t tile_m = tile / tiles_n, tile_n = tile - tile_m * tiles_n;
        const int64_t m0 = tile_m * TM;
        const unsigned char* src = g.w_prep + tile_n * n_kb * S::B_STAGE;
        int32_t b = 0, h0 = 0, w0 = 0;
        if (g.conv) {
          // 128 consecutive output pixels from (b, yo, xo); the halo and everything past the image are zeros
          b = static_cast<int32_t>(m0 / g.HoWo);
          const int32_t rem = static_cast<int32_t>(m0 - static_cast<int64_t>(b) * g.HoWo);
          const int32_t yo = rem / g.Wo, xo = rem - yo * g.Wo;
          h0 = yo * g.sh - g.ph;
          w0 = xo * g.sw - g.pw;
        }
        int32_t cb = 0, fi = 0, fj = 0;
        for (int32_t kb = 0; kb < static_cast<int32_t>(n_kb); kb++) {
          if (round > 0 && !mbar_wait(&empty[s], (round & 1) ^ 1, abort_flag, 1)) { ok = false; break; }
          mbar_arrive_expect_tx(&full[s], RES ? S::A_STAGE : S::A_STAGE + S::B_STAGE);
          // the innermost coordinate (a channel or K offset, a multiple of 64 elements) is 128-byte aligned
          if (g.conv)
            tma_load_im2col_4d(smem + S::OFF_A + s * S::A_STAGE, &a_map, cb * KB, w0, h0, b, static_cast<uint16_t>(fj),
                               static_cast<uint16_t>(fi), &full[s]);
          else
            tma_load_2d(smem + S::OFF_A + s * S::A_STAGE, &a_map, kb * KB, static_cast<int32_t>(m0), &full[s]);
          if (!RES) bulk_copy_g2s(smem + off_b + s * S::B_STAGE, src, S::B_STAGE, &full[s]);
          src += S::B_STAGE;
          issued++;
          if (++cb == g.cblocks) { cb = 0; if (++fj == g.kw) { fj = 0; fi++; } }
          if (++s == STAGES) { s = 0; round++; }
        }
      }
      if (!ok || *abort_flag) {
        // aborted: the copies already issued must land before the CTA's shared memory goes away (their
        // barriers count nothing but this thread's arrival and the bytes, so each wait ends with its copy)
        if (RES && my_tiles > 0) mbar_wait_quiet(wfull, 0, kDrainPolls);
        const int64_t pending = issued < STAGES ? issued : STAGES;
        for (int64_t q = 1; q <= pending; q++) {
          const int64_t idx = issued - q;
          mbar_wait_quiet(&full[idx % STAGES], static_cast<uint32_t>((idx / STAGES) & 1), kDrainPolls);
        }
      }
    }
    __syncwarp();
  } else if (warp == kMmaWarp) {
    // =========================== MMA issuer ===========================
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(S::NST, kFmtBF16);
      const uint64_t da0 = smem_desc(smem_u32(smem + S::OFF_A)), db0 = smem_desc(smem_u32(smem + off_b));
      const uint64_t da_hi = da0 & 0xFFFFFFFF00000000ull, db_hi = db0 & 0xFFFFFFFF00000000ull;
      const uint32_t da_lo = static_cast<uint32_t>(da0), db_lo = static_cast<uint32_t>(db0);
      const uint32_t full_a = smem_u32(full), empty_a = smem_u32(empty), tfull_a = smem_u32(tfull), tempty_a = smem_u32(tempty);
      uint32_t s = 0, full_par = 0;
      bool ok = true;
      if (RES && my_tiles > 0) ok = mbar_wait(wfull, 0, abort_flag, 6);
      for (int64_t ti = 0; ti < my_tiles && ok; ti++) {
        const uint32_t buf = static_cast<uint32_t>(ti & 1);
        if (ti >= 2) {      // the epilogue must have drained this accumulator (used by tile ti - 2)
          if (!mbar_wait_a(tempty_a + buf * 8, static_cast<uint32_t>(((ti >> 1) & 1) ^ 1), abort_flag, 3)) { ok = false; break; }
          tc_fence_after();
        }
        const uint32_t d_tmem = tmem_base + buf * S::NST;
        for (int64_t kb = 0; kb < n_kb; kb++) {
          if (!mbar_wait_a(full_a + s * 8, full_par, abort_flag, 2)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_lo = da_lo + s * (S::A_STAGE >> 4);
          const uint32_t b_lo = db_lo + (RES ? static_cast<uint32_t>(kb) : s) * (S::B_STAGE >> 4);
#pragma unroll
          for (int ks = 0; ks < KB / 16; ks++)          // 16 K-elements = 32 bytes along the swizzled rows
            umma_bf16(d_tmem, da_hi | (a_lo + ks * 2), db_hi | (b_lo + ks * 2), idesc, (kb | ks) != 0 ? 1u : 0u);
          umma_commit_a(empty_a + s * 8);
          if (++s == STAGES) { s = 0; full_par ^= 1; }
        }
        if (ok) umma_commit_a(tfull_a + buf * 8);
      }
      // every MMA issued so far has retired before TMEM is released -- also after an abort, so this wait does
      // not look at the abort flag
      umma_commit(drain);
      if (!mbar_wait_quiet(drain, 0, g_spin_limit < kDrainPolls ? kDrainPolls : g_spin_limit)) {
        atomicCAS(&g_error_word, 0, 4);
        *abort_flag = 1;
      }
    }
    __syncwarp();
  } else if (warp < 4) {
    // =========================== epilogue ===========================
    const int row = warp * 32 + lane;
    const uint32_t t_lane = static_cast<uint32_t>(warp * 32) << 16;
    for (int64_t ti = 0; ti < my_tiles; ti++) {
      const uint32_t buf = static_cast<uint32_t>(ti & 1);
      if (!mbar_wait(&tfull[buf], static_cast<uint32_t>((ti >> 1) & 1), abort_flag, 5)) break;
      tc_fence_after();
      const int64_t tile = blockIdx.x + ti * gridDim.x;
      const int64_t m = (tile / tiles_n) * TM + row, nb = (tile % tiles_n) * TN;
      float* dst = g.C + m * g.ldc + nb;
      float carry = 0.0f;                                   // |z| sum of a next-layer group wider than a 32-column chunk
#pragma unroll
      for (int c = 0; c < TN / 32; c++) {
        uint32_t v[NP][32];
        const uint32_t t_addr = tmem_base + t_lane + buf * S::NST + c * 32;
#pragma unroll
        for (int i = 0; i < NP; i++) tmem_ld32(t_addr + i * TN, v[i]);
        tmem_ld_wait();
        if (m < g.M && g.ep.mode != kEpiPlain) {
          // activation, affine map, then a dense (fp32 / bf16) or binarized row instead of the fp32 product
          float cv[32], fs[32], fh[32];
#pragma unroll
          for (int e = 0; e < 32; e++) {
            float acc = __uint_as_float(v[NP - 1][e]);
#pragma unroll
            for (int i = NP - 2; i >= 0; i--) acc += __uint_as_float(v[i][e]);
            cv[e] = acc;
            const int64_t n = nb + c * 32 + e;
            fs[e] = (g.ep.bn_scale && n < g.N) ? __ldg(g.ep.bn_scale + n) : 1.0f;
            fh[e] = (g.ep.bn_shift && n < g.N) ? __ldg(g.ep.bn_shift + n) : 0.0f;
          }
          epi::finish_chunk(g.ep, cv, fs, fh, m, nb + c * 32, g.N, c == TN / 32 - 1, nb + TN, carry);
        } else if (m < g.M) {
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            float o[4];
#pragma unroll
            for (int e = 0; e < 4; e++) {    // smallest pieces first
              float acc = __uint_as_float(v[NP - 1][j + e]);
#pragma unroll
              for (int i = NP - 2; i >= 0; i--) acc += __uint_as_float(v[i][j + e]);
              o[e] = acc;
            }
            const int64_t n = nb + c * 32 + j;
            if (g.c_vec && n + 3 < g.N)
              *reinterpret_cast<float4*>(dst + c * 32 + j) = make_float4(o[0], o[1], o[2], o[3]);
            else
              for (int e = 0; e < 4; e++)
                if (n + e < g.N) dst[c * 32 + j + e] = o[e];
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty[buf]);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, S::TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------------------------
// The same contraction on CTA pairs.  The single-CTA kernel above is bound by shared-memory traffic: per
// 64-element stage of a 128 x 128 tile it writes 48 KB (16 KB of activations, 32 KB of stacked weight pieces)
// and the tensor core reads them back, 96 KB against 512 clocks of MMA issue.  Two CTAs on neighbouring SMs
// that work on vertically adjacent row tiles need the SAME weight stage, so they run as a cluster of two and
// issue one 256 x 256 x 16 MMA (tcgen05 cta_group::2): each CTA stages its own 128 activation rows and only
// ONE of the two weight pieces (the MMA reads the second operand's halves from both CTAs' shared memories), 32 KB
// per stage and CTA, and the ring holds six stages instead of four.  Each CTA's tensor memory receives its own
// 128 rows of the 256 stacked columns, so the epilogue is unchanged.
//   rank 0: its loader thread posts the expected bytes of BOTH CTAs' copies on its `full` barrier, its MMA
//           thread issues every MMA of the pair and commits to the `empty` / `tfull` barriers of both CTAs;
//   rank 1: its loader thread fetches its tiles with copies that complete on rank 0's `full` barrier (no
//           multicast: every CTA fetches what it stages itself); its MMA warp only owns the TMEM allocation;
//   both  : the epilogue warps drain their CTA's accumulator and arrive on rank 0's `tempty` barrier.
template <int TN, int NP>
struct PairSmem {
  static constexpr int NST = NP * TN;                      // stacked weight rows = MMA N
  static constexpr int A_STAGE = TM * 128;                 // this CTA's 128 activation rows
  static constexpr int B_HALF = (NST / 2) * 128;           // this CTA's half of the stacked weight rows
  static constexpr int STAGE = A_STAGE + B_HALF;
  static constexpr int STAGES = (200 * 1024) / STAGE;
  static constexpr int OFF_A = 0;
  static constexpr int OFF_B = STAGES * A_STAGE;
  static constexpr int OFF_BAR = STAGES * STAGE;
  static constexpr int NBAR = 2 * STAGES + 4 + 1;          // full, empty, tfull[2], tempty[2], drain
  static constexpr int BYTES = OFF_BAR + NBAR * 8 + 16;
  static constexpr int TMEM_COLS = 512;
  static_assert(NST == 256 && B_HALF == Smem<TN, NP>::B_PIECE, "each CTA of the pair stages exactly one weight piece");
};

template <int TN, int NP>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
hbwn_pair_kernel(const Args g, const __grid_constant__ CUtensorMap a_map, const __grid_constant__ CUtensorMap b_map) {
  using S = PairSmem<TN, NP>;
  constexpr int STAGES = S::STAGES;
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + S::OFF_BAR);
  uint64_t* empty = full + STAGES;
  uint64_t* tfull = empty + STAGES;
  uint64_t* tempty = tfull + 2;
  uint64_t* drain = tempty + 2;
  uint32_t* tmem_base_ptr = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_ptr + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const int64_t pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int64_t tiles_n = (g.N + TN - 1) / TN, tiles_m = (g.M + 2 * TM - 1) / (2 * TM);     // tiles of 256 rows
  const int64_t n_tiles = tiles_m * tiles_n;
  const int64_t n_kb = g.n_kb;
  const int64_t my_tiles = pair < n_tiles ? (n_tiles - pair + n_pairs - 1) / n_pairs : 0;

  pdl_launch_dependents();
  if (tid == 0) {
    for (int s = 0; s < STAGES; s++) {
      mbar_init(&full[s], 1);           // rank 0: its loader's expect_tx arrival; the copies of both CTAs complete the bytes
      mbar_init(&empty[s], 1);          // MMA commit (to both CTAs)
    }
    for (int b = 0; b < 2; b++) { mbar_init(&tfull[b], 1); mbar_init(&tempty[b], 8); }     // 4 epilogue warps x 2 CTAs
    mbar_init(drain, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    tmem_alloc_pair(tmem_base_ptr, S::TMEM_COLS);
    tmem_relinquish_pair();
  }
  pdl_wait();
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                  // both CTAs' barriers exist before either signals the other
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_ptr;

  if (warp == kLoaderWarp) {
    // =========================== loader (both CTAs) ===========================
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&a_map) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&b_map) : "memory");
      const uint32_t full0 = mapa_rank(smem_u32(full), 0);          // rank 0's `full` barriers
      int s = 0;
      uint32_t round = 0;
      int64_t issued = 0;
      bool ok = true;
      for (int64_t ti = 0; ti < my_tiles && ok; ti++) {
        const int64_t tile = pair + ti * n_pairs;
        const int64_t tile_m = tile / tiles_n, tile_n = tile - tile_m * tiles_n;
        const int64_t m0 = tile_m * (2 * TM) + rank * TM;
        // rows of the weight-piece matrix: [column tile][k block][piece][TN rows]; this CTA stages piece `rank`
        int32_t b_row = static_cast<int32_t>((tile_n * n_kb * NP + rank) * TN);
        int32_t b = 0, h0 = 0, w0 = 0;
        if (g.conv) {
          b = static_cast<int32_t>(m0 / g.HoWo);
          const int32_t rem = static_cast<int32_t>(m0 - static_cast<int64_t>(b) * g.HoWo);
          const int32_t yo = rem / g.Wo, xo = rem - yo * g.Wo;
          h0 = yo * g.sh - g.ph;
          w0 = xo * g.sw - g.pw;
        }
        int32_t cb = 0, fi = 0, fj = 0;
        for (int32_t kb = 0; kb < static_cast<int32_t>(n_kb); kb++) {
          if (round > 0 && !mbar_wait(&empty[s], (round & 1) ^ 1, abort_flag, 1)) { ok = false; break; }
          if (rank == 0) mbar_arrive_expect_tx(&full[s], 2 * S::STAGE);
          const uint32_t bar = full0 + s * 8;
          if (g.conv)
            tma_load_im2col_4d_pair(smem + S::OFF_A + s * S::A_STAGE, &a_map, cb * KB, w0, h0, b, static_cast<uint16_t>(fj),
                                    static_cast<uint16_t>(fi), bar);
          else
            tma_load_2d_pair(smem + S::OFF_A + s * S::A_STAGE, &a_map, kb * KB, static_cast<int32_t>(m0), bar);
          tma_load_2d_pair(smem + S::OFF_B + s * S::B_HALF, &b_map, 0, b_row, bar);
          b_row += NP * TN;
          issued++;
          if (++cb == g.cblocks) { cb = 0; if (++fj == g.kw) { fj = 0; fi++; } }
          if (++s == STAGES) { s = 0; round++; }
        }
      }
      if (!ok || *abort_flag) {
        // aborted: copies already issued must land before this CTA's shared memory goes away.  Rank 0 can watch
        // its barriers; rank 1 cannot see them and gives its own copies a fixed time that is far longer than a copy.
        if (rank == 0) {
          const int64_t pending = issued < STAGES ? issued : STAGES;
          for (int64_t q = 1; q <= pending; q++) {
            const int64_t idx = issued - q;
            mbar_wait_quiet(&full[idx % STAGES], static_cast<uint32_t>((idx / STAGES) & 1), kDrainPolls);
          }
        } else {
          for (int q = 0; q < 64; q++) __nanosleep(1000);
        }
      }
    }
    __syncwarp();
  } else if (warp == kMmaWarp) {
    // =========================== MMA issuer (rank 0) ===========================
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = instr_desc_pair(S::NST, kFmtBF16);
      const uint64_t da0 = smem_desc(smem_u32(smem + S::OFF_A)), db0 = smem_desc(smem_u32(smem + S::OFF_B));
      const uint64_t da_hi = da0 & 0xFFFFFFFF00000000ull, db_hi = db0 & 0xFFFFFFFF00000000ull;
      const uint32_t da_lo = static_cast<uint32_t>(da0), db_lo = static_cast<uint32_t>(db0);
      const uint32_t full_a = smem_u32(full), empty_a = smem_u32(empty), tfull_a = smem_u32(tfull), tempty_a = smem_u32(tempty);
      uint32_t s = 0, full_par = 0;
      bool ok = true;
      for (int64_t ti = 0; ti < my_tiles && ok; ti++) {
        const uint32_t buf = static_cast<uint32_t>(ti & 1);
        if (ti >= 2) {      // the epilogues of both CTAs must have drained this accumulator (used by tile ti - 2)
          if (!mbar_wait_a(tempty_a + buf * 8, static_cast<uint32_t>(((ti >> 1) & 1) ^ 1), abort_flag, 3)) { ok = false; break; }
          tc_fence_after();
        }
        const uint32_t d_tmem = tmem_base + buf * S::NST;
        for (int64_t kb = 0; kb < n_kb; kb++) {
          if (!mbar_wait_a(full_a + s * 8, full_par, abort_flag, 2)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_lo = da_lo + s * (S::A_STAGE >> 4);
          const uint32_t b_lo = db_lo + s * (S::B_HALF >> 4);
#pragma unroll
          for (int ks = 0; ks < KB / 16; ks++)
            umma_bf16_pair(d_tmem, da_hi | (a_lo + ks * 2), db_hi | (b_lo + ks * 2), idesc, (kb | ks) != 0 ? 1u : 0u);
          umma_commit_pair_mc(empty_a + s * 8, 3);
          if (++s == STAGES) { s = 0; full_par ^= 1; }
        }
        if (ok) umma_commit_pair_mc(tfull_a + buf * 8, 3);
      }
      // every MMA issued so far has retired (in both CTAs) before tensor memory is released -- also after an abort
      umma_commit_pair(smem_u32(drain));
      if (!mbar_wait_quiet(drain, 0, g_spin_limit < kDrainPolls ? kDrainPolls : g_spin_limit)) {
        atomicCAS(&g_error_word, 0, 4);
        *abort_flag = 1;
      }
    }
    __syncwarp();
  } else if (warp < 4) {
    // =========================== epilogue (both CTAs) ===========================
    const int row = warp * 32 + lane;
    const uint32_t t_lane = static_cast<uint32_t>(warp * 32) << 16;
    const uint32_t tempty0 = mapa_rank(smem_u32(tempty), 0);        // rank 0's `tempty` barriers
    for (int64_t ti = 0; ti < my_tiles; ti++) {
      const uint32_t buf = static_cast<uint32_t>(ti & 1);
      if (!mbar_wait(&tfull[buf], static_cast<uint32_t>((ti >> 1) & 1), abort_flag, 5)) break;
      tc_fence_after();
      const int64_t tile = pair + ti * n_pairs;
      const int64_t m = (tile / tiles_n) * (2 * TM) + rank * TM + row, nb = (tile % tiles_n) * TN;
      float* dst = g.C + m * g.ldc + nb;
      float carry = 0.0f;
#pragma unroll
      for (int c = 0; c < TN / 32; c++) {
        uint32_t v[NP][32];
        const uint32_t t_addr = tmem_base + t_lane + buf * S::NST + c * 32;
#pragma unroll
        for (int i = 0; i < NP; i++) tmem_ld32(t_addr + i * TN, v[i]);
        tmem_ld_wait();
        if (m < g.M && g.ep.mode != kEpiPlain) {
          float cv[32], fs[32], fh[32];
#pragma unroll
          for (int e = 0; e < 32; e++) {
            float acc = __uint_as_float(v[NP - 1][e]);
#pragma unroll
            for (int i = NP - 2; i >= 0; i--) acc += __uint_as_float(v[i][e]);
            cv[e] = acc;
            const int64_t n = nb + c * 32 + e;
            fs[e] = (g.ep.bn_scale && n < g.N) ? __ldg(g.ep.bn_scale + n) : 1.0f;
            fh[e] = (g.ep.bn_shift && n < g.N) ? __ldg(g.ep.bn_shift + n) : 0.0f;
          }
          epi::finish_chunk(g.ep, cv, fs, fh, m, nb + c * 32, g.N, c == TN / 32 - 1, nb + TN, carry);
        } else if (m < g.M) {
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            float o[4];
#pragma unroll
            for (int e = 0; e < 4; e++) {    // smallest pieces first
              float acc = __uint_as_float(v[NP - 1][j + e]);
#pragma unroll
              for (int i = NP - 2; i >= 0; i--) acc += __uint_as_float(v[i][j + e]);
              o[e] = acc;
            }
            const int64_t n = nb + c * 32 + j;
            if (g.c_vec && n + 3 < g.N)
              *reinterpret_cast<float4*>(dst + c * 32 + j) = make_float4(o[0], o[1], o[2], o[3]);
            else
              for (int e = 0; e < 4; e++)
                if (n + e < g.N) dst[c * 32 + j + e] = o[e];
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(tempty0 + buf * 8);
    }
  }

  // Neither CTA may leave while the other can still reach into it (rank 0's MMAs read rank 1's shared memory and
  // write its tensor memory; rank 1's copies and epilogue warps signal rank 0's barriers): rank 0 arrives here
  // only after its drain wait.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, S::TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------------------------
// Stride-1 convolution of a 64-channel image with at most 64 filters (the first residual stage of the
// ResNet workload): every filter tap reads the SAME staged input rows.
//
// Output positions are numbered over the zero-padded image, P = (b * Hp + y) * Wp + x with Hp = H + 2 ph and
// Wp = W + 2 pw, so that the input pixel of tap (i, j) of position P is position P + i Wp + j whatever P is.
// A tile is 128 consecutive positions; its inputs are the 128 + (kh - 1) Wp + (kw - 1) <= 256 consecutive
// positions from P0.  Positions are staged in blocks of 128 (one im2col-mode tensor copy whose bounding box is
// the padded image: 128-byte rows of 64 channels, zeros outside the tensor); a CTA walks a contiguous run of
// tiles, so block t + 1 is both the halo of tile t and the body of tile t + 1 and every block is fetched once.
// The MMA of tap (i, j) reads its 128 x 64 activation tile at a start address shifted by (i Wp + j) rows: the
// 128-byte swizzle is a function of the shared-memory address alone, so a start on any row boundary reads the
// rows as they were written.  Blocks live in a ring of four slots; a fifth slot behind the last one mirrors
// slot 0, so that the window of a tile in slot 3 continues in contiguous memory.  The input is read once
// instead of once per tap (a 3 x 3 filter: 16 KB instead of 144 KB per tile) and the copies run up to three
// tiles ahead of the MMAs; the weight pieces of all taps stay resident in shared memory.  Positions in the
// padding columns and rows (x >= Wo or y >= Ho) are computed like the others and dropped by the epilogue.
constexpr int kRing = 4;                // ring slots; slot kRing mirrors slot 0
constexpr int kBlockBytes = TM * 128;   // one block of 128 positions x 64 channels
struct HaloArgs {
  int32_t Wp, Hp, HpWp, Ho, Wo, B;
  int32_t kh, kw, ph, pw;
  int64_t positions;                    // B * Hp * Wp
  int64_t tiles_per_cta;
};

template <int NP>
__global__ void __launch_bounds__(kThreads, 1)
hbwn_halo_kernel(const Args g, const HaloArgs h, const __grid_constant__ CUtensorMap a_map) {
  constexpr int TN = 64;
  using S = Smem<TN, NP>;
  extern __shared__ __align__(1024) unsigned char smem[];
  // [ring slots 0..3][mirror of slot 0][weight pieces of every tap][barriers]
  constexpr int off_b = (kRing + 1) * kBlockBytes;
  const int off_bar = off_b + g.taps * S::B_STAGE;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + off_bar);
  uint64_t* empty = full + kRing;
  uint64_t* tfull = empty + kRing;
  uint64_t* tempty = tfull + 2;
  uint64_t* drain = tempty + 2;
  uint64_t* wfull = drain + 1;
  uint32_t* tmem_base_ptr = reinterpret_cast<uint32_t*>(wfull + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_ptr + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t n_tiles = (h.positions + TM - 1) / TM;
  const int64_t tile0 = blockIdx.x * h.tiles_per_cta;
  const int64_t my_tiles = tile0 < n_tiles ? (n_tiles - tile0 < h.tiles_per_cta ? n_tiles - tile0 : h.tiles_per_cta) : 0;

  pdl_launch_dependents();
  if (tid == 0) {
    for (int s = 0; s < kRing; s++) {
      mbar_init(&full[s], 1);           // the loader's expect_tx arrival; the copies complete the bytes
      mbar_init(&empty[s], 1);          // MMA commit
    }
    for (int b = 0; b < 2; b++) { mbar_init(&tfull[b], 1); mbar_init(&tempty[b], 4); }
    mbar_init(drain, 1);
    mbar_init(wfull, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    tmem_alloc(tmem_base_ptr, S::TMEM_COLS);
    tmem_relinquish();
  }
  pdl_wait();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_ptr;

  if (warp == kLoaderWarp) {
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&a_map) : "memory");
      int64_t issued = 0;
      bool ok = true;
      if (my_tiles > 0) {
        mbar_arrive_expect_tx(wfull, static_cast<uint32_t>(g.taps) * S::B_STAGE);
        for (int t = 0; t < g.taps; t++)
          bulk_copy_g2s(smem + off_b + t * S::B_STAGE, g.w_prep + static_cast<int64_t>(t) * S::B_STAGE, S::B_STAGE, wfull);
      }
      // block k of this CTA = positions (tile0 + k) * 128 ...; one more block than tiles (the last tile's halo)
      const int64_t n_blocks = my_tiles > 0 ? my_tiles + 1 : 0;
      const int64_t p_first = tile0 * TM;
      int32_t b = static_cast<int32_t>(p_first / h.HpWp);
      const int32_t rem = static_cast<int32_t>(p_first - static_cast<int64_t>(b) * h.HpWp);
      int32_t y = rem / h.Wp, x = rem - y * h.Wp;
      for (int64_t k = 0; k < n_blocks; k++) {
        const int s = static_cast<int>(k & (kRing - 1));
        if (k >= kRing && !mbar_wait(&empty[s], static_cast<uint32_t>(((k / kRing) & 1) ^ 1), abort_flag, 1)) { ok = false; break; }
        const bool mirror = s == 0 && k > 0;                  // also the continuation of the tile in the last slot
        mbar_arrive_expect_tx(&full[s], mirror ? 2u * kBlockBytes : 1u * kBlockBytes);
        tma_load_im2col_4d(smem + s * kBlockBytes, &a_map, 0, x - h.pw, y - h.ph, b, 0, 0, &full[s]);
        if (mirror) tma_load_im2col_4d(smem + kRing * kBlockBytes, &a_map, 0, x - h.pw, y - h.ph, b, 0, 0, &full[s]);
        issued++;
        x += TM;
        while (x >= h.Wp) { x -= h.Wp; if (++y == h.Hp) { y = 0; b++; } }
      }
      if (!ok || *abort_flag) {
        // aborted: the copies already issued must land before the CTA's shared memory goes away
        if (my_tiles > 0) mbar_wait_quiet(wfull, 0, kDrainPolls);
        const int64_t pending = issued < kRing ? issued : kRing;
        for (int64_t q = 1; q <= pending; q++) {
          const int64_t idx = issued - q;
          mbar_wait_quiet(&full[idx & (kRing - 1)], static_cast<uint32_t>((idx / kRing) & 1), kDrainPolls);
        }
      }
    }
    __syncwarp();
  } else if (warp == kMmaWarp) {
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(S::NST, kFmtBF16);
      const uint64_t da0 = smem_desc(smem_u32(smem)), db0 = smem_desc(smem_u32(smem + off_b));
      const uint64_t da_hi = da0 & 0xFFFFFFFF00000000ull, db_hi = db0 & 0xFFFFFFFF00000000ull;
      const uint32_t da_lo = static_cast<uint32_t>(da0), db_lo = static_cast<uint32_t>(db0);
      bool ok = true;
      if (my_tiles > 0) ok = mbar_wait(wfull, 0, abort_flag, 6) && mbar_wait(&full[0], 0, abort_flag, 2);
      for (int64_t ti = 0; ti < my_tiles && ok; ti++) {
        const uint32_t buf = static_cast<uint32_t>(ti & 1);
        if (ti >= 2) {      // the epilogue must have drained this accumulator (used by tile ti - 2)
          if (!mbar_wait(&tempty[buf], static_cast<uint32_t>(((ti >> 1) & 1) ^ 1), abort_flag, 3)) { ok = false; break; }
        }
        // the tile's own block arrived for the tile before (or above); its halo is block ti + 1
        const uint32_t s = static_cast<uint32_t>(ti & (kRing - 1));
        const int64_t k1 = ti + 1;
        if (!mbar_wait(&full[k1 & (kRing - 1)], static_cast<uint32_t>((k1 / kRing) & 1), abort_flag, 2)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * S::NST;
        const uint32_t win_lo = da_lo + s * (kBlockBytes >> 4);       // slot 3 continues into the mirror slot
        int32_t fi = 0, fj = 0;
        for (int32_t t = 0; t < g.taps; t++) {
          const uint32_t a_lo = win_lo + static_cast<uint32_t>(fi * h.Wp + fj) * 8u;      // 128-byte rows in 16-byte units
          const uint32_t b_lo = db_lo + static_cast<uint32_t>(t) * (S::B_STAGE >> 4);
#pragma unroll
          for (int ks = 0; ks < KB / 16; ks++)
            umma_bf16(d_tmem, da_hi | (a_lo + ks * 2), db_hi | (b_lo + ks * 2), idesc, (t | ks) != 0 ? 1u : 0u);
          if (++fj == h.kw) { fj = 0; fi++; }
        }
        umma_commit(&empty[s]);
        umma_commit(&tfull[buf]);
      }
      umma_commit(drain);
      if (!mbar_wait_quiet(drain, 0, g_spin_limit < kDrainPolls ? kDrainPolls : g_spin_limit)) {
        atomicCAS(&g_error_word, 0, 4);
        *abort_flag = 1;
      }
    }
    __syncwarp();
  } else if (warp < 4) {
    const int row = warp * 32 + lane;
    const uint32_t t_lane = static_cast<uint32_t>(warp * 32) << 16;
    for (int64_t ti = 0; ti < my_tiles; ti++) {
      const uint32_t buf = static_cast<uint32_t>(ti & 1);
      // where this thread's position lies in the padded image, and whether it is an output at all
      const int64_t p = (tile0 + ti) * TM + row;
      const int32_t b = static_cast<int32_t>(p / h.HpWp);
      const int32_t rem = static_cast<int32_t>(p - static_cast<int64_t>(b) * h.HpWp);
      const int32_t y = rem / h.Wp, x = rem - y * h.Wp;
      const bool valid = b < h.B && y < h.Ho && x < h.Wo;
      const int64_t m = (static_cast<int64_t>(b) * h.Ho + y) * h.Wo + x;
      if (!mbar_wait(&tfull[buf], static_cast<uint32_t>((ti >> 1) & 1), abort_flag, 5)) break;
      tc_fence_after();
      float* dst = g.C + m * g.ldc;
      float carry = 0.0f;
#pragma unroll
      for (int c = 0; c < TN / 32; c++) {
        uint32_t v[NP][32];
        const uint32_t t_addr = tmem_base + t_lane + buf * S::NST + c * 32;
#pragma unroll
        for (int i = 0; i < NP; i++) tmem_ld32(t_addr + i * TN, v[i]);
        tmem_ld_wait();
        if (valid && g.ep.mode != kEpiPlain) {
          float cv[32], fs[32], fh[32];
#pragma unroll
          for (int e = 0; e < 32; e++) {
            float acc = __uint_as_float(v[NP - 1][e]);
#pragma unroll
            for (int i = NP - 2; i >= 0; i--) acc += __uint_as_float(v[i][e]);
            cv[e] = acc;
            const int64_t n = c * 32 + e;
            fs[e] = (g.ep.bn_scale && n < g.N) ? __ldg(g.ep.bn_scale + n) : 1.0f;
            fh[e] = (g.ep.bn_shift && n < g.N) ? __ldg(g.ep.bn_shift + n) : 0.0f;
          }
          epi::finish_chunk(g.ep, cv, fs, fh, m, c * 32, g.N, c == TN / 32 - 1, TN, carry);
        } else if (valid) {
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            float o[4];
#pragma unroll
            for (int e = 0; e < 4; e++) {    // smallest pieces first
              float acc = __uint_as_float(v[NP - 1][j + e]);
#pragma unroll
              for (int i = NP - 2; i >= 0; i--) acc += __uint_as_float(v[i][j + e]);
              o[e] = acc;
            }
            const int64_t n = c * 32 + j;
            if (g.c_vec && n + 3 < g.N)
              *reinterpret_cast<float4*>(dst + n) = make_float4(o[0], o[1], o[2], o[3]);
            else
              for (int e = 0; e < 4; e++)
                if (n + e < g.N) dst[n + e] = o[e];
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty[buf]);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, S::TMEM_COLS);
  }
}

Args make_args(const DenseView& A, const PackedView& W, float* C, int64_t ldc) {
  Args g;
  g.a = reinterpret_cast<const __nv_bfloat16*>(A.data); g.lda = A.ld;
  g.w_bits = W.bits; g.w_scales = W.scales; g.ldw_w = W.ld_words; g.ldw_s = W.ld_scales; g.w_bf16 = W.scale_bf16;
  g.C = C; g.ldc = ldc;
  g.c_vec = (reinterpret_cast<uintptr_t>(C) % 16 == 0 && ldc % 4 == 0) ? 1 : 0;
  g.M = A.rows; g.N = W.rows; g.K = A.K;
  g.Gw = num_groups(W.K, W.beta);
  g.beta = W.beta;
  g.w_prep = nullptr;
  g.n_kb = (g.K + KB - 1) / KB;
  g.conv = 0; g.taps = 1; g.kw = 1; g.cblocks = static_cast<int32_t>(g.n_kb); g.Cin = 0;
  g.HoWo = 1; g.Wo = 1; g.sh = g.sw = 1; g.ph = g.pw = 0;
  g.ep = plain_epilogue();
  return g;
}

template <int TN, int NP>
size_t prep_bytes(const Args& g) {
  return static_cast<size_t>(((g.N + TN - 1) / TN) * g.n_kb) * Smem<TN, NP>::B_STAGE;
}

// Tensor map of the activation matrix: bf16 [M, K] with row pitch lda, boxes of 64 x 128 elements
// (one 128-byte-swizzled stage tile), zeros outside the matrix.
bool make_a_map(const Args& g, CUtensorMap* map) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(g.K), static_cast<cuuint64_t>(g.M)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(g.lda) * 2};
  const cuuint32_t box[2] = {KB, TM};
  const cuuint32_t elem[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(g.a), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// im2col tensor map of an NHWC bf16 image [B, H, W, Cp]: base pixels are the top-left input positions
// of the filter windows (from -pad, stepping by the stride, Wo x Ho per image), 128 of them per copy
// with 64 channels each; the filter tap is added by the copy instruction.
bool make_conv_map(const void* x_nhwc, const ConvGeom& c, int Cp, CUtensorMap* map) {
  EncodeIm2colFn fn = encode_im2col_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(c.C), static_cast<cuuint64_t>(c.W), static_cast<cuuint64_t>(c.H),
                              static_cast<cuuint64_t>(c.B)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(Cp) * 2, static_cast<cuuint64_t>(c.W) * Cp * 2,
                                 static_cast<cuuint64_t>(c.H) * c.W * Cp * 2};
  const int lower[2] = {-c.pw, -c.ph};
  const int upper[2] = {c.pw - (c.kw - 1), c.ph - (c.kh - 1)};
  const cuuint32_t elem[4] = {1, static_cast<cuuint32_t>(c.sw), static_cast<cuuint32_t>(c.sh), 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(x_nhwc), dims, strides, lower, upper, KB, TM, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of the shared-patch kernel: the same NHWC image, but the base pixels walk the whole zero-padded
// image (Wp x Hp positions per image) and one copy brings `rows` consecutive positions.
bool make_halo_map(const void* x_nhwc, const ConvGeom& c, int Cp, int rows, CUtensorMap* map) {
  EncodeIm2colFn fn = encode_im2col_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(c.C), static_cast<cuuint64_t>(c.W), static_cast<cuuint64_t>(c.H),
                              static_cast<cuuint64_t>(c.B)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(Cp) * 2, static_cast<cuuint64_t>(c.W) * Cp * 2,
                                 static_cast<cuuint64_t>(c.H) * c.W * Cp * 2};
  const int lower[2] = {-c.pw, -c.ph};
  const int upper[2] = {c.pw, c.ph};
  const cuuint32_t elem[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(x_nhwc), dims, strides, lower, upper, KB,
            static_cast<cuuint32_t>(rows), elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of the prepared weight pieces for the CTA-pair kernel: rows of 128 bytes (64 bf16) in the order the
// preparation kernel wrote them, already swizzled, so the copy uses no swizzle of its own; one box = one piece of
// one stage (TN rows).
bool make_pieces_map(const void* w_prep, int64_t rows, int box_rows, CUtensorMap* map) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn || rows >= (int64_t{1} << 31)) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(KB), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {128};
  const cuuint32_t box[2] = {KB, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(w_prep), dims, strides, box, elem,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kHaloSmemMax = 227 * 1024;

// Whether the shared-rows kernel takes this convolution, and its geometry: stride 1, exactly one 64-channel
// block, one 64-column tile, a tile's window within two blocks of 128 positions, and the five ring slots
// beside the resident weight pieces in shared memory.
bool plan_halo(const ConvGeom& c, int64_t N, HaloArgs* h) {
  if (c.sh != 1 || c.sw != 1 || c.C != KB || N > 64 || c.ph > 127 || c.pw > 127) return false;
  const int64_t Wp = static_cast<int64_t>(c.W) + 2 * c.pw, Hp = static_cast<int64_t>(c.H) + 2 * c.ph;
  if (static_cast<int64_t>(c.kh - 1) * Wp + (c.kw - 1) > TM || Hp * Wp >= (int64_t{1} << 31)) return false;
  const int64_t smem = static_cast<int64_t>(kRing + 1) * kBlockBytes + static_cast<int64_t>(c.kh) * c.kw * Smem<64, 2>::B_STAGE + 256;
  if (smem > kHaloSmemMax) return false;
  h->Wp = static_cast<int32_t>(Wp); h->Hp = static_cast<int32_t>(Hp); h->HpWp = static_cast<int32_t>(Hp * Wp);
  h->Ho = c.Ho; h->Wo = c.Wo; h->B = c.B;
  h->kh = c.kh; h->kw = c.kw; h->ph = c.ph; h->pw = c.pw;
  h->positions = static_cast<int64_t>(c.B) * Hp * Wp;
  h->tiles_per_cta = 0;
  return true;
}

Args make_conv_args(const ConvGeom& c, const PackedView& W, float* C, int64_t ldc) {
  Args g;
  g.a = nullptr; g.lda = 0;
  g.w_bits = W.bits; g.w_scales = W.scales; g.ldw_w = W.ld_words; g.ldw_s = W.ld_scales; g.w_bf16 = W.scale_bf16;
  g.C = C; g.ldc = ldc;
  g.c_vec = (reinterpret_cast<uintptr_t>(C) % 16 == 0 && ldc % 4 == 0) ? 1 : 0;
  g.M = static_cast<int64_t>(c.B) * c.Ho * c.Wo; g.N = W.rows; g.K = W.K;
  g.Gw = num_groups(W.K, W.beta);
  g.beta = W.beta;
  g.w_prep = nullptr;
  g.conv = 1; g.taps = c.kh * c.kw; g.kw = c.kw; g.cblocks = (c.C + KB - 1) / KB; g.Cin = c.C;
  g.n_kb = static_cast<int64_t>(g.taps) * g.cblocks;
  g.HoWo = c.Ho * c.Wo; g.Wo = c.Wo; g.sh = c.sh; g.sw = c.sw; g.ph = c.ph; g.pw = c.pw;
  g.ep = plain_epilogue();
  return g;
}

template <int TN, int NP>
cudaError_t launch(Args g, const CUtensorMap& a_map, void* workspace, cudaStream_t stream, const CopyArgs* copy = nullptr,
                   bool w_prepared = false, const HaloArgs* halo = nullptr) {
  using S = Smem<TN, NP>;
  constexpr int kResBytes = 225 * 1024;
  static DeviceOnce configured;
  int dev = 0, sms = 0;
  if (current_device(&dev, &sms) != cudaSuccess) return cudaErrorInvalidDevice;
  if (configured.pending(dev)) {
    cudaError_t e = cudaFuncSetAttribute(hbwn_umma_kernel<TN, NP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(hbwn_umma_kernel<TN, NP, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kResBytes);
    if (e != cudaSuccess) return e;
    configured.mark(dev);
  }
  const int64_t tiles_n = (g.N + TN - 1) / TN, n_kb = g.n_kb;
  dim3 pgrid(static_cast<unsigned>(n_kb), static_cast<unsigned>(tiles_n));
  if (copy) {
    const int64_t blocks = copy->n_copy + (w_prepared ? 0 : n_kb * tiles_n);     // prepared weights: the copy blocks only
    if (blocks > 0x7fffffff) return cudaErrorNotSupported;
    const cudaError_t e = copy->pb == kNhwcPBLarge
        ? launch_pdl(nhwc_and_pieces_kernel<TN, NP, kNhwcPBLarge>, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, stream, *copy, g,
                     static_cast<unsigned char*>(workspace))
        : launch_pdl(nhwc_and_pieces_kernel<TN, NP, kNhwcPBSmall>, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, stream, *copy, g,
                     static_cast<unsigned char*>(workspace));
    if (e != cudaSuccess) return e;
  } else if (!w_prepared) {
    prepare_w_pieces_kernel<TN, NP><<<pgrid, 256, 0, stream>>>(g, static_cast<unsigned char*>(workspace));
  }
  g.w_prep = static_cast<const unsigned char*>(workspace);
  if constexpr (TN == 64 && NP == 2) {
    if (halo) {
      static DeviceOnce halo_configured;
      if (halo_configured.pending(dev)) {
        const cudaError_t e = cudaFuncSetAttribute(hbwn_halo_kernel<NP>, cudaFuncAttributeMaxDynamicSharedMemorySize, kHaloSmemMax);
        if (e != cudaSuccess) return e;
        halo_configured.mark(dev);
      }
      const int64_t used = static_cast<int64_t>(kRing + 1) * kBlockBytes + static_cast<int64_t>(g.taps) * S::B_STAGE + 256;
      const int bytes = static_cast<int>(used > 120 * 1024 ? used : 120 * 1024);          // one CTA per SM
      const int64_t tiles = (halo->positions + TM - 1) / TM;
      HaloArgs hh = *halo;
      hh.tiles_per_cta = (tiles + sms - 1) / sms;                                          // contiguous runs
      const int64_t ctas = (tiles + hh.tiles_per_cta - 1) / hh.tiles_per_cta;
      return launch_pdl(hbwn_halo_kernel<NP>, dim3(static_cast<unsigned>(ctas)), dim3(kThreads), bytes, stream, g, hh, a_map);
    }
  }
  if constexpr (TN == 128 && NP == 2) {
    // at least two row tiles: CTA pairs that share each weight stage
    if (g.M > TM && sms >= 2) {
      using P = PairSmem<TN, NP>;
      static DeviceOnce pair_configured;
      if (pair_configured.pending(dev)) {
        const cudaError_t e = cudaFuncSetAttribute(hbwn_pair_kernel<TN, NP>, cudaFuncAttributeMaxDynamicSharedMemorySize, P::BYTES);
        if (e != cudaSuccess) return e;
        pair_configured.mark(dev);
      }
      CUtensorMap b_map;
      if (!make_pieces_map(g.w_prep, tiles_n * n_kb * NP * TN, TN, &b_map)) return cudaErrorNotSupported;
      const int64_t pair_tiles = ((g.M + 2 * TM - 1) / (2 * TM)) * tiles_n;
      const int64_t pairs = pair_tiles < sms / 2 ? pair_tiles : sms / 2;
      return launch_pdl(hbwn_pair_kernel<TN, NP>, dim3(static_cast<unsigned>(2 * pairs)), dim3(kThreads), P::BYTES, stream, g, a_map, b_map);
    }
  }
  const int64_t tiles = ((g.M + TM - 1) / TM) * tiles_n;
  const unsigned grid = static_cast<unsigned>(tiles < sms ? tiles : sms);
  // a single column tile whose pieces fit beside the activation ring stays resident in shared memory
  if (tiles_n == 1 && n_kb * S::B_STAGE <= S::RES_MAX_B && tiles > sms)
    return launch_pdl(hbwn_umma_kernel<TN, NP, true>, dim3(grid), dim3(kThreads), kResBytes, stream, g, a_map);
  return launch_pdl(hbwn_umma_kernel<TN, NP, false>, dim3(grid), dim3(kThreads), S::BYTES, stream, g, a_map);
}

// exact: three pieces, 64-column tiles.  Otherwise two pieces: 128-column tiles when there are more than 64 columns.
cudaError_t launch_any(const Args& g, const CUtensorMap& a_map, void* workspace, cudaStream_t stream, const CopyArgs* copy, bool w_prepared,
                       bool exact, const HaloArgs* halo = nullptr) {
  if (exact) return launch<64, 3>(g, a_map, workspace, stream, copy, w_prepared);
  if (g.N <= 64) return launch<64, 2>(g, a_map, workspace, stream, copy, w_prepared, halo);
  return launch<128, 2>(g, a_map, workspace, stream, copy, w_prepared);
}

}  // namespace

// bf16 activations whose rows start on 16-byte boundaries (what a tensor map can describe: extents
// below 2^32, pitch below 2^40 bytes); any weight group size.
bool hbwn_umma_supported(const DenseView& A, const PackedView& W) {
  (void)W;
  return A.bf16 && reinterpret_cast<uintptr_t>(A.data) % 16 == 0 && (A.ld * 2) % 16 == 0 &&
         A.rows < (int64_t{1} << 31) && A.K < (int64_t{1} << 31) && A.ld * 2 < (int64_t{1} << 40) &&
         encode_tiled_fn() != nullptr;
}

// enough for either piece count (the three-piece layout is the larger one)
size_t hbwn_umma_workspace_bytes(const DenseView& A, const PackedView& W) {
  const Args g = make_args(A, W, nullptr, 0);
  const size_t a = prep_bytes<64, 3>(g), b = prep_bytes<128, 2>(g);
  return a > b ? a : b;
}

cudaError_t launch_hbwn_umma(const DenseView& A, const PackedView& W, float* C, int64_t ldc, void* workspace,
                             cudaStream_t stream, bool w_prepared, bool exact, const EpiArgs* ep) {
  Args g = make_args(A, W, C, ldc);
  if (ep) g.ep = *ep;
  CUtensorMap a_map;
  if (!make_a_map(g, &a_map)) return cudaErrorNotSupported;
  return launch_any(g, a_map, workspace, stream, nullptr, w_prepared, exact);
}

// Implicit-GEMM convolution: whole 64-channel blocks (every tile row is then 128 bytes of real
// channels), image extents and filter offsets inside what an im2col tensor map can describe.
bool hbwn_umma_conv_supported(const ConvGeom& c, const PackedView& W) {
  (void)W;
  return c.C % KB == 0 && c.kh <= 16 && c.kw <= 16 && c.ph < 16 && c.pw < 16 && c.sh <= 8 && c.sw <= 8 &&
         static_cast<int64_t>(c.Ho) * c.Wo < (int64_t{1} << 31) && encode_im2col_fn() != nullptr;
}

size_t hbwn_umma_conv_workspace_bytes(const ConvGeom& c, const PackedView& W) {
  const Args g = make_conv_args(c, W, nullptr, 0);
  const size_t a = prep_bytes<64, 2>(g), b = prep_bytes<128, 2>(g);
  return a > b ? a : b;
}

cudaError_t launch_hbwn_umma_conv(const void* x, int x_bf16, void* x_nhwc, int Cp, const ConvGeom& c, const PackedView& W, float* C,
                                  int64_t ldc, void* workspace, cudaStream_t stream, bool w_prepared, const EpiArgs* ep,
                                  bool input_is_nhwc) {
  Args g = make_conv_args(c, W, C, ldc);
  if (ep) g.ep = *ep;
  CUtensorMap a_map;
  // more row tiles than SMs on a stride-1, 64-channel, 64-filter layer: the kernel that stages one patch per tile
  HaloArgs halo;
  int dev = 0, sms = 0;
  if (current_device(&dev, &sms) != cudaSuccess) return cudaErrorInvalidDevice;
  const bool use_halo = plan_halo(c, g.N, &halo) && (g.M + TM - 1) / TM > sms;
  const void* image = input_is_nhwc ? x : x_nhwc;
  if (use_halo ? !make_halo_map(image, c, Cp, TM, &a_map) : !make_conv_map(image, c, Cp, &a_map)) return cudaErrorNotSupported;
  // input_is_nhwc: the caller's tensor already is the NHWC bf16 image the tensor copies read (channel pitch Cp)
  if (input_is_nhwc) return launch_any(g, a_map, workspace, stream, nullptr, w_prepared, false, use_halo ? &halo : nullptr);
  CopyArgs cp;
  cp.x = x; cp.x_bf16 = x_bf16; cp.C = c.C; cp.Cp = Cp; cp.HW = static_cast<int64_t>(c.H) * c.W;
  cp.out = static_cast<unsigned short*>(x_nhwc);
  cp.pb = nhwc_pixels_per_block(cp.HW);
  cp.gx = static_cast<int32_t>((cp.HW + cp.pb - 1) / cp.pb);
  cp.gy = (Cp + kNhwcCB - 1) / kNhwcCB;
  cp.n_copy = static_cast<int64_t>(cp.gx) * cp.gy * c.B;
  return launch_any(g, a_map, workspace, stream, &cp, w_prepared, false, use_halo ? &halo : nullptr);
}

cudaError_t hbwn_umma_health(int op, int* value) {
  switch (op) {
    case kHealthRead: return umma::read_error_word(value);
    case kHealthClear: return umma::clear_error_word();
    case kHealthSetSpinLimit: return umma::set_spin_limit(static_cast<uint32_t>(*value));
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace hbmm
