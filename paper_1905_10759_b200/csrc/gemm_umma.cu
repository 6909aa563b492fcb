// HBMM contraction of two packed operands on the 5th-generation tensor cores (tcgen05 / TMEM).
//
// Section 4.2, Eq. 7: per K-segment one signed +-1 dot product D and two full-precision multiplies,
//   C[m,n] += (deltaA[m,seg] * deltaW[n,seg]) * D[m,n].
// Both factors of every term are produced by the tensor cores:
//   * D: the sign bits of both operands are expanded to +-1.0 in e4m3 (one byte per element; sums of
//     a few thousand +-1 products are exact in the fp32 accumulator) and one tcgen05.mma
//     (kind::f8f6f4, K = 32) per 32-bit K-word accumulates the segment's dot of a 128 x TN tile in
//     tensor memory.
//   * S = deltaA (x) deltaW: each fp32 scale is split into three bf16 pieces a = a1 + a2 + a3
//     (24 significant bits), and one small tcgen05.mma (kind::f16, K = 16, six non-zero columns)
//     forms a1w1 + a1w2 + a2w1 + a2w2 + a1w3 + a3w1 -- every bf16 x bf16 product is exact in fp32
//     and the omitted cross terms are below 2^-26 of the product -- so the scale product of the
//     whole tile arrives in tensor memory at fp32 accuracy without touching the FMA pipe.
// The epilogue warps then read D and S from TMEM and do one fp32 FMA per output and segment,
// C += S * D, two outputs per instruction (fma.rn.f32x2).  Every group keeps its own full-precision
// scale exactly as in the popcount path.
//
// CTA tile = 128 rows x TN columns; one persistent CTA per SM (it owns all 512 TMEM columns)
// walks the tiles of the output.
//   warps 0-7   : epilogue (warp w reads TMEM lanes 32*(w%4).., warps 0-3 the left half of the
//                 columns, warps 4-7 the right half); they take most of the register file
//   warps 8-11  : A producers: packed words -> e4m3 bytes and scales -> bf16 pieces, both in the UMMA
//                 K-major core-matrix layout (8 rows x 16 bytes contiguous)
//   warp  12    : TMEM allocation and the single MMA-issuing thread
//   warp  13    : one thread streams the W operand: a small kernel has expanded W once per call into
//                 the same stage layout in the workspace, so a stage of W is one contiguous bulk copy
//                 (cp.async.bulk, completion counted on the stage's mbarrier) instead of per-tile work
// A stage holds four K-words; stages and TMEM accumulator buffers are rings guarded by
// mbarriers.  Every wait is bounded: when a limit expires the thread records an error code in
// global memory, raises a CTA-wide abort flag that all other waits observe, and the kernel
// drains and frees its TMEM before returning.
#include <cuda_bf16.h>
#include "kernels.h"
#include "umma_common.cuh"
#include "gemm_umma_prep.cuh"

namespace hbmm {
namespace {

using namespace umma;
using namespace umma_prep;

constexpr int kEpilogueWarps = 8;                         // warpgroups 0 and 1
constexpr int kProducerWarps = 4;                         // warpgroup 2: one A row per thread
constexpr int kFirstProducerWarp = kEpilogueWarps;        // warps 8..11
constexpr int kMmaWarp = kEpilogueWarps + kProducerWarps; // warp 12: TMEM allocation, MMA issue
constexpr int kLoaderWarp = kMmaWarp + 1;                 // warp 13: bulk copies of the prepared W stages
constexpr int kThreads = 16 * 32;                         // 512: four warpgroups (warps 14, 15 only hand registers over)
constexpr int kRegsEpilogue = 208;                        // 256 x 208 + 128 x 64 + 128 x 32 = 64 K registers
constexpr int kRegsProducer = 64;
constexpr int kRegsIssuer = 32;
// Expands the weight operand once per call (one block per (stage, tile), one thread per row).
template <int TN>
__global__ void __launch_bounds__(TN)
prepare_w_kernel(const Args g, unsigned char* __restrict__ out) {
  prepare_w_task<TN>(g, out, blockIdx.x, blockIdx.y, threadIdx.x);
}

template <int TN>
__global__ void __launch_bounds__(kThreads, 1)
hbmm_umma_kernel(const Args g) {
  using S = Smem<TN>;
  constexpr int NBUF = S::NBUF;
  constexpr int HALF = TN / 2;                  // columns per epilogue warpgroup
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + S::OFF_BAR);
  uint64_t* empty = full + STAGES;
  uint64_t* tfull = empty + STAGES;
  uint64_t* tempty = tfull + NBUF;
  uint64_t* drain = tempty + NBUF;
  uint32_t* tmem_base_ptr = reinterpret_cast<uint32_t*>(smem + S::OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + S::OFF_MISC + 4);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t tiles_n = (g.N + TN - 1) / TN, tiles_m = (g.M + TM - 1) / TM;
  const int64_t n_tiles = tiles_m * tiles_n;
  const int64_t n_stages = (g.n_words + WPS - 1) / WPS;                 // per tile
  const int64_t n_segs = (g.n_words + g.seg_words - 1) / g.seg_words;   // per tile

  // ---- set-up
  // the zero halves of the A scale rows never change: written once for every stage
  if (tid < TM)
    for (int s = 0; s < STAGES; s++)
      for (int q = 0; q < WPS; q++) *reinterpret_cast<uint4*>(swz(smem + S::OFF_SA + s * S::SA_STAGE, tid, 2 * q + 1)) = make_uint4(0, 0, 0, 0);
  if (tid == 0) {
    for (int s = 0; s < STAGES; s++) {
      mbar_init(&full[s], kProducerWarps + 1);        // the A producer warps + the loader's expect_tx arrival
      mbar_init(&empty[s], 1);                        // MMA commit: the stage's bytes have been read
    }
    for (int b = 0; b < NBUF; b++) {
      mbar_init(&tfull[b], 1);                        // MMA commit
      mbar_init(&tempty[b], kEpilogueWarps);
    }
    mbar_init(drain, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  fence_async_proxy();                                // those zeros are read by the tensor core
  if (warp == kMmaWarp) {
    tmem_alloc(tmem_base_ptr, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_ptr;

  // The CTA is persistent: it walks tiles blockIdx.x, blockIdx.x + gridDim.x, ... and the stage and
  // accumulator rings simply continue across tiles (gst / gseg count stages / segments since launch).
  if (warp >= kFirstProducerWarp && warp < kMmaWarp) {
    // =========================== A producers ===========================
    reg_dec<kRegsProducer>();
    const int p = tid - kFirstProducerWarp * 32;             // tile row of this thread
    // fp32 scales with one group per segment: the four scales of a stage are one 16-byte vector
    const bool vec_scales = !g.a_bf16 && g.ra == 1 && g.seg_words == 1;
    int64_t gst = 0;
    bool ok = true;
    for (int64_t tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
      const int64_t m = (tile / tiles_n) * TM + p;
      const bool in = m < g.M;
      const uint32_t* bptr = g.a_bits + (in ? m : 0) * g.lda_w;
      const int64_t srow = (in ? m : 0) * g.lda_s;
      int in_seg = 0, in_g = 0;      // position of the next word to fetch inside its segment / group
      int64_t grp = 0;
      auto fetch = [&](int64_t st, uint4& w, float (&f)[WPS]) {
        const int64_t kw = st * WPS;
        w = make_uint4(0, 0, 0, 0);
        if (in && kw < g.lda_w) w = __ldg(reinterpret_cast<const uint4*>(bptr + kw));
        if (vec_scales) {
          float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
          if (in && kw < g.lda_s) v = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(g.a_scales) + srow + kw));
          f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;    // entries past the last group are stored zeros
        } else {
          // first decide which scale every word needs (no loaded value is touched here) ...
          int64_t idx[WPS];
#pragma unroll
          for (int q = 0; q < WPS; q++) {
            idx[q] = (in && kw + q < g.n_words && grp < g.Ga) ? srow + grp : -1;
            if (++in_seg == g.seg_words) { in_seg = 0; if (++in_g == g.ra) { in_g = 0; grp++; } }
          }
          // ... then issue the loads back to back
#pragma unroll
          for (int q = 0; q < WPS; q++) { f[q] = 0.0f; if (idx[q] >= 0) f[q] = load_scale(g.a_scales, g.a_bf16, idx[q]); }
        }
      };
      uint4 w, nw;
      float f[WPS], nf[WPS];
      fetch(0, w, f);
      for (int64_t st = 0; st < n_stages; st++, gst++) {
        if (st + 1 < n_stages) fetch(st + 1, nw, nf);     // in flight while this stage is expanded
        const int s = static_cast<int>(gst % STAGES);
        if (gst >= STAGES && !mbar_wait(&empty[s], static_cast<uint32_t>(((gst / STAGES) & 1) ^ 1), abort_flag, 1)) { ok = false; break; }
        expand_words(smem + S::OFF_A + s * S::A_STAGE, p, w);
#pragma unroll
        for (int q = 0; q < WPS; q++)
          *reinterpret_cast<uint4*>(swz(smem + S::OFF_SA + s * S::SA_STAGE, p, 2 * q)) = scale_row<false>(f[q]);
        fence_async_proxy();          // make the generic-proxy stores visible to the tensor core
        __syncwarp();
        if (lane == 0) mbar_arrive(&full[s]);
        w = nw;
#pragma unroll
        for (int q = 0; q < WPS; q++) f[q] = nf[q];
      }
    }
  } else if (warp == kLoaderWarp) {
    // =========================== W loader ===========================
    reg_dec<kRegsIssuer>();
    if (lane == 0) {
      int64_t gst = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const unsigned char* src = g.w_prep + (tile % tiles_n) * n_stages * S::B_STAGE;
        for (int64_t st = 0; st < n_stages; st++, gst++) {
          const int s = static_cast<int>(gst % STAGES);
          if (gst >= STAGES && !mbar_wait(&empty[s], static_cast<uint32_t>(((gst / STAGES) & 1) ^ 1), abort_flag, 6)) { ok = false; break; }
          mbar_arrive_expect_tx(&full[s], S::B_STAGE);
          bulk_copy_g2s(smem + S::OFF_B + s * S::B_STAGE, src + st * S::B_STAGE, S::B_STAGE, &full[s]);
        }
      }
      if (!ok || *abort_flag) {
        // aborted: the copies already issued (at most one per stage) must land before the CTA's shared memory
        // goes away.  Their barriers also count producer arrivals that may never come, so each wait is a
        // short bounded one that ignores the abort flag.
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
    reg_dec<kRegsIssuer>();
    if (lane == 0) {
      constexpr uint32_t idesc_sign = instr_desc(TN, kFmtE4M3), idesc_scale = instr_desc(TN, kFmtBF16);
      // Descriptors of stage 0 / word slot 0; every other slot differs only by its start address, so
      // the low descriptor word is stepped by bytes/16.
      const uint64_t da0 = smem_desc(smem_u32(smem + S::OFF_A)), db0 = smem_desc(smem_u32(smem + S::OFF_B));
      const uint64_t dsa0 = smem_desc(smem_u32(smem + S::OFF_SA)), dsb0 = smem_desc(smem_u32(smem + S::OFF_B + S::B_SIGNS));
      constexpr uint32_t kWord = 32 >> 4;                                   // next word slot: 32 bytes along the rows
      constexpr uint32_t kStageA = S::A_STAGE >> 4, kStageSA = S::SA_STAGE >> 4, kStageB = S::B_STAGE >> 4;
      const uint32_t n_words = static_cast<uint32_t>(g.n_words), seg_words = static_cast<uint32_t>(g.seg_words);
      const uint32_t full_a = smem_u32(full), empty_a = smem_u32(empty), tfull_a = smem_u32(tfull), tempty_a = smem_u32(tempty);
      const uint32_t da_lo = static_cast<uint32_t>(da0), db_lo = static_cast<uint32_t>(db0);
      const uint32_t dsa_lo = static_cast<uint32_t>(dsa0), dsb_lo = static_cast<uint32_t>(dsb0);
      const uint64_t da_hi = da0 & 0xFFFFFFFF00000000ull, db_hi = db0 & 0xFFFFFFFF00000000ull;
      const uint64_t dsa_hi = dsa0 & 0xFFFFFFFF00000000ull, dsb_hi = dsb0 & 0xFFFFFFFF00000000ull;
      uint32_t s = 0, full_par = 0;          // stage slot and the parity its "full" barrier completes with next
      uint32_t buf = 0, tempty_par = 0;      // accumulator buffer; the first pass over the ring needs no wait
      bool first_ring = true;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        uint32_t in_seg = 0;
        for (uint32_t kw0 = 0; kw0 < n_words && ok; kw0 += WPS) {
          if (!mbar_wait_a(full_a + s * 8, full_par, abort_flag, 2)) { ok = false; break; }
          tc_fence_after();
          const uint32_t nq = n_words - kw0 < WPS ? n_words - kw0 : WPS;
          // low descriptor words of word slot 0 of this stage; the slots step by constants
          uint32_t a_lo = da_lo + s * kStageA, b_lo = db_lo + s * kStageB;
          uint32_t sa_lo = dsa_lo + s * kStageSA, sb_lo = dsb_lo + s * kStageB;
          for (uint32_t q = 0; q < nq; q++) {
            const uint32_t d_tmem = tmem_base + buf * (2 * TN);
            if (in_seg == 0 && !first_ring) {
              if (!mbar_wait_a(tempty_a + buf * 8, tempty_par, abort_flag, 3)) { ok = false; break; }
              tc_fence_after();
            }
            umma_f8(d_tmem, da_hi | a_lo, db_hi | b_lo, idesc_sign, in_seg);
            if (++in_seg == seg_words || kw0 + q == n_words - 1) {
              // scale product of the segment (K columns 0..7 hold the pieces of this word slot, 8..15 zeros)
              umma_bf16_overwrite(d_tmem + TN, dsa_hi | sa_lo, dsb_hi | sb_lo, idesc_scale);
              umma_commit_a(tfull_a + buf * 8);   // segment complete: hand D and S to the epilogue
              in_seg = 0;
              if (++buf == NBUF) { buf = 0; if (first_ring) first_ring = false; else tempty_par ^= 1; }
            }
            a_lo += kWord; b_lo += kWord; sa_lo += kWord; sb_lo += kWord;
          }
          umma_commit_a(empty_a + s * 8);     // stage's bytes are free once these MMAs have read them
          if (++s == STAGES) { s = 0; full_par ^= 1; }
        }
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
  } else if (warp < kEpilogueWarps) {
    // =========================== epilogue ===========================
    reg_inc<kRegsEpilogue>();
    const int wg = warp >> 2;                       // column half
    const int row = (warp & 3) * 32 + lane;         // TMEM lane = tile row
    const uint32_t t_lane = static_cast<uint32_t>((warp & 3) * 32) << 16;
    // The warp's columns of a segment are read in two pieces (D and S of each), double buffered: while the
    // FMAs of one piece run, the loads of the next piece -- of the next segment when this was the
    // last one -- are in flight.  (tcgen05.wait::ld waits for every outstanding load, so two pieces
    // are as deep as the pipeline can usefully go.)
    constexpr int PIECES = 2, PW = HALF / 2;        // piece width: 32 columns for TN = 128, 16 for TN = 64
    const int64_t my_tiles = blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const int64_t total_segs = my_tiles * n_segs;
    uint32_t d[2][PW], sc[2][PW];
    uint64_t acc[HALF / 2];                         // two fp32 outputs per register pair
    bool ok = true;
    auto tmem_of = [&](int64_t gseg) { return tmem_base + t_lane + static_cast<uint32_t>(gseg % NBUF) * 2 * TN + wg * HALF; };
    if (total_segs > 0) {
      ok = mbar_wait(&tfull[0], 0, abort_flag, 5);
      tc_fence_after();
      if (ok) { tmem_ld_piece(tmem_of(0), d[0]); tmem_ld_piece(tmem_of(0) + TN, sc[0]); tmem_ld_wait(); }
    }
    int64_t tile = blockIdx.x, seg = 0;
    for (int64_t gseg = 0; gseg < total_segs && ok; gseg++) {
      if (seg == 0) {
#pragma unroll
        for (int j = 0; j < HALF / 2; j++) acc[j] = 0ull;
      }
#pragma unroll
      for (int c = 0; c < PIECES; c++) {
        // piece c of this segment is in d[c & 1] / sc[c & 1]; start the loads of what comes next
        if (c + 1 < PIECES) {
          tmem_ld_piece(tmem_of(gseg) + (c + 1) * PW, d[(c + 1) & 1]);
          tmem_ld_piece(tmem_of(gseg) + TN + (c + 1) * PW, sc[(c + 1) & 1]);
        } else {
          // every column of this segment is in registers: the buffer can be refilled
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tempty[gseg % NBUF]);
          if (gseg + 1 < total_segs) {
            if (!mbar_wait(&tfull[(gseg + 1) % NBUF], static_cast<uint32_t>(((gseg + 1) / NBUF) & 1), abort_flag, 5)) { ok = false; break; }
            tc_fence_after();
            tmem_ld_piece(tmem_of(gseg + 1), d[(c + 1) & 1]);
            tmem_ld_piece(tmem_of(gseg + 1) + TN, sc[(c + 1) & 1]);
          }
        }
#pragma unroll
        for (int j = 0; j < PW; j += 2)
          acc[(c * PW + j) / 2] = fma2(pack2(sc[c & 1][j], sc[c & 1][j + 1]), pack2(d[c & 1][j], d[c & 1][j + 1]), acc[(c * PW + j) / 2]);
        tmem_ld_wait();
      }
      if (!ok) break;
      if (++seg == n_segs) {
        seg = 0;
        const int64_t m = (tile / tiles_n) * TM + row, nb = (tile % tiles_n) * TN + wg * HALF;
        if (m < g.M) {
          float* dst = g.C + m * g.ldc + nb;
#pragma unroll
          for (int j = 0; j < HALF; j += 4) {
            float v[4];
            unpack2(acc[j / 2], v[0], v[1]);
            unpack2(acc[j / 2 + 1], v[2], v[3]);
            if (nb + j + 3 < g.N) *reinterpret_cast<float4*>(dst + j) = make_float4(v[0], v[1], v[2], v[3]);
            else
              for (int e = 0; e < 4; e++)
                if (nb + j + e < g.N) dst[j + e] = v[e];
          }
        }
        tile += gridDim.x;
      }
    }
  } else {
    reg_dec<kRegsIssuer>();   // warps 14, 15: nothing to do but hand their registers over
  }

  // ---- teardown: everyone meets here (aborted threads too), then the allocating warp frees TMEM
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

template <int TN>
size_t prep_bytes(const Args& g) {
  const int64_t tiles_n = (g.N + TN - 1) / TN, n_stages = (g.n_words + WPS - 1) / WPS;
  return static_cast<size_t>(tiles_n * n_stages) * Smem<TN>::B_STAGE;
}

template <int TN>
cudaError_t launch_umma(Args g, void* workspace, cudaStream_t stream, bool w_prepared) {
  using S = Smem<TN>;
  static DeviceOnce configured;
  int dev = 0, sms = 0;
  if (current_device(&dev, &sms) != cudaSuccess) return cudaErrorInvalidDevice;
  if (configured.pending(dev)) {
    cudaError_t e = cudaFuncSetAttribute(hbmm_umma_kernel<TN>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::BYTES);
    if (e != cudaSuccess) return e;
    configured.mark(dev);
  }
  const int64_t tiles_n = (g.N + TN - 1) / TN, n_stages = (g.n_words + WPS - 1) / WPS;
  dim3 pgrid(static_cast<unsigned>(n_stages), static_cast<unsigned>(tiles_n));
  if (!w_prepared) prepare_w_kernel<TN><<<pgrid, TN, 0, stream>>>(g, static_cast<unsigned char*>(workspace));
  g.w_prep = static_cast<const unsigned char*>(workspace);
  const int64_t tiles = ((g.M + TM - 1) / TM) * tiles_n;
  const unsigned grid = static_cast<unsigned>(tiles < sms ? tiles : sms);   // one persistent CTA per SM
  hbmm_umma_kernel<TN><<<grid, kThreads, S::BYTES, stream>>>(g);
  return cudaGetLastError();
}

Args make_args(const PackedView& A, const PackedView& W, float* C, int64_t ldc) {
  Args g;
  g.a_bits = A.bits; g.a_scales = A.scales; g.w_bits = W.bits; g.w_scales = W.scales; g.C = C;
  g.M = A.rows; g.N = W.rows; g.lda_w = A.ld_words; g.ldw_w = W.ld_words; g.lda_s = A.ld_scales; g.ldw_s = W.ld_scales;
  g.ldc = ldc; g.a_bf16 = A.scale_bf16; g.w_bf16 = W.scale_bf16;
  g.n_words = A.K / 32;
  const bool a_one = A.beta >= A.K, w_one = W.beta >= W.K;
  int64_t seg;
  if (a_one && w_one) seg = A.K;
  else if (a_one) seg = W.beta;
  else if (w_one) seg = A.beta;
  else seg = A.beta < W.beta ? A.beta : W.beta;
  g.seg_words = seg / 32;
  const int64_t T = (g.n_words + g.seg_words - 1) / g.seg_words;
  g.ra = static_cast<int32_t>(a_one ? T : A.beta / seg);
  g.rw = static_cast<int32_t>(w_one ? T : W.beta / seg);
  g.Ga = num_groups(A.K, A.beta);
  g.Gw = num_groups(W.K, W.beta);
  g.w_prep = nullptr;
  return g;
}

}  // namespace

// K a multiple of 32 and segments of whole words (any number of them).
bool gemm_tensor_supported(const PackedView& A, const PackedView& W) {
  if (A.K % 32 != 0) return false;
  const bool a_one = A.beta >= A.K, w_one = W.beta >= W.K;
  if (!a_one && A.beta % 32 != 0) return false;
  if (!w_one && W.beta % 32 != 0) return false;
  return true;
}

// Bytes of workspace the tensor path needs: the weight operand expanded into its stage layout.
size_t gemm_tensor_workspace_bytes(const PackedView& A, const PackedView& W) {
  const Args g = make_args(A, W, nullptr, 0);
  return g.N <= 64 ? prep_bytes<64>(g) : prep_bytes<128>(g);
}

// workspace: device, 16-byte aligned, at least gemm_tensor_workspace_bytes.
cudaError_t launch_gemm_tensor(const PackedView& A, const PackedView& W, float* C, int64_t ldc, void* workspace,
                               cudaStream_t stream, bool w_prepared) {
  const Args g = make_args(A, W, C, ldc);
  return g.N <= 64 ? launch_umma<64>(g, workspace, stream, w_prepared) : launch_umma<128>(g, workspace, stream, w_prepared);
}

// The weight expansion of launch_gemm_tensor(A, W, ..., workspace) as a job for another kernel.
void gemm_tensor_prep_job(const PackedView& A, const PackedView& W, void* workspace, UmmaPrepJob* job) {
  job->g = make_args(A, W, nullptr, 0);
  job->folded = 0;
  job->out_down = nullptr;
  job->out = static_cast<unsigned char*>(workspace);
  job->tn = job->g.N <= 64 ? 64 : 128;
  job->n_stages = static_cast<int32_t>((job->g.n_words + WPS - 1) / WPS);
  job->tiles_n = static_cast<int32_t>((job->g.N + job->tn - 1) / job->tn);
}

cudaError_t gemm_umma_health(int op, int* value) {
  switch (op) {
    case kHealthRead: return umma::read_error_word(value);
    case kHealthClear: return umma::clear_error_word();
    case kHealthSetSpinLimit: return umma::set_spin_limit(static_cast<uint32_t>(*value));
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace hbmm
