// HBMM contraction of two packed operands on the 5th-generation tensor cores (tcgen05 / TMEM).
//
// Section 4.2, Eq. 7: per K-segment one signed +-1 dot product and two full-precision multiplies.
// Here the +-1 dot of a segment is a dense contraction: the sign bits of both operands are
// expanded to +-1.0 in e4m3 (one byte per element, products and sums of at most a few thousand
// +-1 terms are exact in the fp32 accumulator), and one tcgen05.mma (kind::f8f6f4, K = 32) per
// 32-bit K-word accumulates the segment's dot for a 128 x TN tile in tensor memory.  The epilogue
// warps read each finished segment from TMEM and apply C += (deltaA * D) * deltaW in fp32
// registers, so every group keeps its own full-precision scale exactly as in the popcount path.
//
// CTA = 128 rows x TN columns, one CTA per SM (it owns all 512 TMEM columns).
//   warps 0-7   : epilogue (warp w reads TMEM lanes 32*(w%4).., warps 0-3 the left half of the
//                 columns, warps 4-7 the right half); they take most of the register file
//   warps 8-11  : producers: packed words -> e4m3 bytes in the UMMA K-major core-matrix layout
//                 (8 rows x 16 bytes contiguous), plus the segment scales of the stage
//   warp  12    : TMEM allocation and the single MMA-issuing thread
// A stage holds four K-words; stages and TMEM accumulator buffers are rings guarded by
// mbarriers.  Every wait is bounded: when a limit expires the thread records an error code in
// global memory, raises a CTA-wide abort flag that all other waits observe, and the kernel
// drains and frees its TMEM before returning.
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {

__device__ int g_umma_error = 0;  // 0 = ok; otherwise the code of the first wait that gave up

namespace {

constexpr int kEpilogueWarps = 8;                         // warpgroups 0 and 1
constexpr int kProducerWarps = 4;                         // warpgroup 2
constexpr int kFirstProducerWarp = kEpilogueWarps;        // warps 8..11
constexpr int kMmaWarp = kEpilogueWarps + kProducerWarps; // warp 12 (warps 13..15 only rebalance registers)
constexpr int kThreads = 16 * 32;                         // 512: four warpgroups
constexpr int kRegsEpilogue = 200;                        // 256 threads x 200 + 256 threads x 56 = 64 K registers
constexpr int kRegsOther = 56;
constexpr int TM = 128;
constexpr int WPS = 4;            // K-words per stage
constexpr int STAGES = 4;
constexpr uint32_t kSpinLimit = 1u << 20;   // polls of a (hardware time-limited) try_wait

struct Args {
  const uint32_t* a_bits; const void* a_scales;
  const uint32_t* w_bits; const void* w_scales;
  float* C;
  int64_t M, N, lda_w, ldw_w, lda_s, ldw_s, ldc;
  int32_t a_bf16, w_bf16;
  int32_t ra, rw;          // A group = segment / ra, W group = segment / rw
  int64_t Ga, Gw;
  int64_t n_words;         // K / 32 (K is a multiple of 32 on this path)
  int64_t seg_words;       // K-words per segment
};

__device__ __forceinline__ float load_scale(const void* s, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(s) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(s) + idx);
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

// ---- mbarrier helpers (shared::cta)
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the limit expired or another thread aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int code) {
  for (uint32_t it = 0; it < kSpinLimit; it++) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
  }
  atomicCAS(&g_umma_error, 0, code);
  *abort_flag = 1;
  return false;
}

// ---- tcgen05 helpers
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols));
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::); }
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols));
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]^T, 128 x N x 32, e4m3 operands, fp32 accumulate.
__device__ __forceinline__ void umma_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(addr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
template <int R> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(R)); }
template <int R> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(R)); }

// K-major operand without swizzle: core matrices of 8 rows x 16 bytes stored contiguously
// (128 bytes); `sbo` = byte distance between 8-row groups, `lbo` = byte distance between the two
// 16-byte K-chunks of one K = 32 instruction.  Descriptor version 1, layout type 0.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr >> 4) & 0x3FFF);
  d |= static_cast<uint64_t>((lbo >> 4) & 0x3FFF) << 16;
  d |= static_cast<uint64_t>((sbo >> 4) & 0x3FFF) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  return d;
}
// Instruction descriptor: fp32 accumulator, e4m3 x e4m3, both K-major, M = 128, N = TN.
__host__ __device__ constexpr uint32_t instr_desc_f8(int n) {
  return (1u << 4) | (0u << 7) | (0u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(TM >> 4) << 24);
}

template <int TN>
struct Smem {
  static constexpr int A_WORD_BYTES = TM * 32;            // one K-word of the A tile, expanded
  static constexpr int B_WORD_BYTES = TN * 32;
  static constexpr int A_STAGE = WPS * A_WORD_BYTES;
  static constexpr int B_STAGE = WPS * B_WORD_BYTES;
  static constexpr int OFF_A = 0;
  static constexpr int OFF_B = OFF_A + STAGES * A_STAGE;
  static constexpr int OFF_SA = OFF_B + STAGES * B_STAGE;               // [STAGES][WPS][TM] float
  static constexpr int OFF_SW = OFF_SA + STAGES * WPS * TM * 4;         // [STAGES][WPS][TN] float
  static constexpr int OFF_LUT = OFF_SW + STAGES * WPS * TN * 4;        // [256] uint2
  static constexpr int OFF_BAR = OFF_LUT + 256 * 8;
  static constexpr int NBUF = 512 / TN;                                 // TMEM accumulator buffers
  // barriers: full[STAGES], empty[STAGES], tfull[NBUF], tempty[NBUF], drain
  static constexpr int NBAR = 2 * STAGES + 2 * NBUF + 1;
  static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;                   // tmem base, abort flag
  static constexpr int USED = OFF_MISC + 16;
  // at least 120 KB so that two CTAs never share an SM (each one allocates all of TMEM)
  static constexpr int BYTES = USED > 120 * 1024 ? USED : 120 * 1024;
};

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
  uint2* lut = reinterpret_cast<uint2*>(smem + S::OFF_LUT);
  float* sA = reinterpret_cast<float*>(smem + S::OFF_SA);
  float* sW = reinterpret_cast<float*>(smem + S::OFF_SW);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * TM, n0 = static_cast<int64_t>(blockIdx.x) * TN;
  const int64_t n_stages = (g.n_words + WPS - 1) / WPS;
  const int64_t n_segs = (g.n_words + g.seg_words - 1) / g.seg_words;

  // ---- set-up
  if (tid < 256) {  // byte of sign bits -> eight e4m3 bytes: 0x38 = +1.0 for bit 1, 0xB8 = -1.0 for bit 0
    uint32_t lo = 0, hi = 0;
#pragma unroll
    for (int i = 0; i < 4; i++) {
      lo |= (((tid >> i) & 1) ? 0x38u : 0xB8u) << (8 * i);
      hi |= (((tid >> (i + 4)) & 1) ? 0x38u : 0xB8u) << (8 * i);
    }
    lut[tid] = make_uint2(lo, hi);
  }
  if (tid == 0) {
    for (int s = 0; s < STAGES; s++) {
      mbar_init(&full[s], kProducerWarps);            // one arrival per producer warp
      mbar_init(&empty[s], 1 + kEpilogueWarps);       // MMA commit + every epilogue warp (scales read)
    }
    for (int b = 0; b < NBUF; b++) {
      mbar_init(&tfull[b], 1);                        // MMA commit
      mbar_init(&tempty[b], kEpilogueWarps);
    }
    mbar_init(drain, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    tmem_alloc(tmem_base_ptr, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_ptr;

  if (warp >= kFirstProducerWarp && warp < kMmaWarp) {
    // =========================== producers ===========================
    reg_dec<kRegsOther>();
    const int p = tid - kFirstProducerWarp * 32;   // 0..127: A row p and B row p
    const bool b_row = p < TN;
    const int64_t m = m0 + p, n = n0 + p;
    const bool a_in = m < g.M, b_in = b_row && n < g.N;
    const uint32_t* a_ptr = g.a_bits + (a_in ? m : 0) * g.lda_w;
    const uint32_t* b_ptr = g.w_bits + (b_in ? n : 0) * g.ldw_w;
    const int64_t a_srow = (a_in ? m : 0) * g.lda_s, b_srow = (b_in ? n : 0) * g.ldw_s;
    // running position of the next word to fetch: segment phase and the two group indices
    int in_seg = 0, in_ga = 0, in_gw = 0;
    int64_t ga = 0, gw = 0;
    float cur_a = 0.0f, cur_w = 0.0f;
    bool need_a = true, need_w = true;
    uint4 wa, wb;
    float fa[WPS], fb[WPS];
    auto fetch = [&](int64_t st) {
      const int64_t kw = st * WPS;
      wa = make_uint4(0, 0, 0, 0);
      wb = make_uint4(0, 0, 0, 0);
      if (a_in && kw < g.lda_w) wa = __ldg(reinterpret_cast<const uint4*>(a_ptr + kw));
      if (b_in && kw < g.ldw_w) wb = __ldg(reinterpret_cast<const uint4*>(b_ptr + kw));
#pragma unroll
      for (int q = 0; q < WPS; q++) {
        const bool live = kw + q < g.n_words;
        if (need_a) { cur_a = (a_in && live && ga < g.Ga) ? load_scale(g.a_scales, g.a_bf16, a_srow + ga) : 0.0f; need_a = false; }
        if (need_w) { cur_w = (b_in && live && gw < g.Gw) ? load_scale(g.w_scales, g.w_bf16, b_srow + gw) : 0.0f; need_w = false; }
        fa[q] = live ? cur_a : 0.0f;
        fb[q] = live ? cur_w : 0.0f;
        if (++in_seg == g.seg_words) {           // next word starts a new segment
          in_seg = 0;
          if (++in_ga == g.ra) { in_ga = 0; ga++; need_a = true; }
          if (++in_gw == g.rw) { in_gw = 0; gw++; need_w = true; }
        }
      }
    };
    auto expand_row = [&](unsigned char* tile, int rows, int row, const uint4& w4) {
      const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
      for (int q = 0; q < WPS; q++) {
        unsigned char* base = tile + q * rows * 32 + (row >> 3) * 128 + (row & 7) * 16;
        const uint2 b0 = lut[w[q] & 0xFF], b1 = lut[(w[q] >> 8) & 0xFF];
        const uint2 b2 = lut[(w[q] >> 16) & 0xFF], b3 = lut[w[q] >> 24];
        *reinterpret_cast<uint4*>(base) = make_uint4(b0.x, b0.y, b1.x, b1.y);                 // K bytes 0..15
        *reinterpret_cast<uint4*>(base + rows * 16) = make_uint4(b2.x, b2.y, b3.x, b3.y);     // K bytes 16..31
      }
    };
    if (n_stages > 0) fetch(0);
    for (int64_t st = 0; st < n_stages; st++) {
      const int s = static_cast<int>(st % STAGES);
      const uint32_t par = static_cast<uint32_t>((st / STAGES) & 1);
      if (st >= STAGES && !mbar_wait(&empty[s], par ^ 1, abort_flag, 1)) break;
      expand_row(smem + S::OFF_A + s * S::A_STAGE, TM, p, wa);
#pragma unroll
      for (int q = 0; q < WPS; q++) sA[(s * WPS + q) * TM + p] = fa[q];
      if (b_row) {
        expand_row(smem + S::OFF_B + s * S::B_STAGE, TN, p, wb);
#pragma unroll
        for (int q = 0; q < WPS; q++) sW[(s * WPS + q) * TN + p] = fb[q];
      }
      if (st + 1 < n_stages) fetch(st + 1);
      fence_async_proxy();          // make the generic-proxy stores visible to the tensor core
      __syncwarp();
      if (lane == 0) mbar_arrive(&full[s]);
    }
  } else if (warp == kMmaWarp) {
    // =========================== MMA issuer ===========================
    reg_dec<kRegsOther>();
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_f8(TN);
      int64_t seg = 0;      // segment being accumulated
      bool ok = true;
      for (int64_t st = 0; st < n_stages && ok; st++) {
        const int s = static_cast<int>(st % STAGES);
        if (!mbar_wait(&full[s], static_cast<uint32_t>((st / STAGES) & 1), abort_flag, 2)) { ok = false; break; }
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + S::OFF_A + s * S::A_STAGE);
        const uint32_t b_addr = smem_u32(smem + S::OFF_B + s * S::B_STAGE);
        for (int q = 0; q < WPS; q++) {
          const int64_t kw = st * WPS + q;
          if (kw >= g.n_words) break;
          const int64_t in_seg = kw - seg * g.seg_words;
          const int buf = static_cast<int>(seg % NBUF);
          if (in_seg == 0 && seg >= NBUF) {
            if (!mbar_wait(&tempty[buf], static_cast<uint32_t>(((seg / NBUF) & 1) ^ 1), abort_flag, 3)) { ok = false; break; }
            tc_fence_after();
          }
          umma_f8(tmem_base + buf * TN,
                  smem_desc(a_addr + q * S::A_WORD_BYTES, TM * 16, 128),
                  smem_desc(b_addr + q * S::B_WORD_BYTES, TN * 16, 128), idesc, in_seg != 0 ? 1u : 0u);
          if (in_seg == g.seg_words - 1 || kw == g.n_words - 1) {
            umma_commit(&tfull[buf]);     // segment complete: hand the accumulator to the epilogue
            seg++;
          }
        }
        umma_commit(&empty[s]);           // stage's bytes are free once these MMAs have read them
      }
      umma_commit(drain);
      mbar_wait(drain, 0, abort_flag, 4); // every MMA has retired before TMEM is released
    }
    __syncwarp();
  } else if (warp < kEpilogueWarps) {
    // =========================== epilogue ===========================
    reg_inc<kRegsEpilogue>();
    const int wg = warp >> 2;                       // column half
    const int row = (warp & 3) * 32 + lane;         // TMEM lane = tile row
    const uint32_t t_lane = static_cast<uint32_t>((warp & 3) * 32) << 16;
    float acc[HALF];
#pragma unroll
    for (int j = 0; j < HALF; j++) acc[j] = 0.0f;
    bool ok = true;
    int64_t released = 0;   // stages this warp has handed back to the producers
    for (int64_t seg = 0; seg < n_segs && ok; seg++) {
      const int buf = static_cast<int>(seg % NBUF);
      if (!mbar_wait(&tfull[buf], static_cast<uint32_t>((seg / NBUF) & 1), abort_flag, 5)) { ok = false; break; }
      tc_fence_after();
      int64_t kw_last = (seg + 1) * g.seg_words - 1;        // the word that carries this segment's scales
      if (kw_last > g.n_words - 1) kw_last = g.n_words - 1;
      const int64_t st = kw_last / WPS;
      const int s = static_cast<int>(st % STAGES), q = static_cast<int>(kw_last % WPS);
      const float sa = sA[(s * WPS + q) * TM + row];
      const float* swp = sW + (s * WPS + q) * TN + wg * HALF;
      uint32_t d[HALF / 32][32];
#pragma unroll
      for (int c = 0; c < HALF / 32; c++) tmem_ld32(tmem_base + t_lane + buf * TN + wg * HALF + c * 32, d[c]);
      tmem_ld_wait();
#pragma unroll
      for (int c = 0; c < HALF / 32; c++)
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const float4 sw = *reinterpret_cast<const float4*>(swp + c * 32 + j);
          acc[c * 32 + j + 0] = fmaf(sa * __uint_as_float(d[c][j + 0]), sw.x, acc[c * 32 + j + 0]);
          acc[c * 32 + j + 1] = fmaf(sa * __uint_as_float(d[c][j + 1]), sw.y, acc[c * 32 + j + 1]);
          acc[c * 32 + j + 2] = fmaf(sa * __uint_as_float(d[c][j + 2]), sw.z, acc[c * 32 + j + 2]);
          acc[c * 32 + j + 3] = fmaf(sa * __uint_as_float(d[c][j + 3]), sw.w, acc[c * 32 + j + 3]);
        }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&tempty[buf]);
        // release every stage whose words are now all consumed (their scales will not be read again)
        int64_t done_words = (seg + 1) * g.seg_words;
        if (done_words > g.n_words) done_words = g.n_words;
        const int64_t consumed = (done_words == g.n_words) ? n_stages : done_words / WPS;
        for (; released < consumed; released++) mbar_arrive(&empty[released % STAGES]);
      }
    }
    if (ok) {
      const int64_t m = m0 + row;
      if (m < g.M) {
        float* dst = g.C + m * g.ldc + n0 + wg * HALF;
#pragma unroll
        for (int j = 0; j < HALF; j += 4) {
          const int64_t n = n0 + wg * HALF + j;
          if (n + 3 < g.N) *reinterpret_cast<float4*>(dst + j) = make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
          else
            for (int e = 0; e < 4; e++)
              if (n + e < g.N) dst[j + e] = acc[j + e];
        }
      }
    }
  } else {
    reg_dec<kRegsOther>();   // warps 13..15: nothing to do but hand their registers over
  }

  // ---- teardown: everyone meets here (aborted threads too), then the allocating warp frees TMEM
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
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

cudaError_t launch_gemm_tensor(const PackedView& A, const PackedView& W, float* C, int64_t ldc, cudaStream_t stream) {
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
  static bool configured[2] = {false, false};
  if (g.N <= 64) {
    using S = Smem<64>;
    if (!configured[0]) {
      cudaError_t e = cudaFuncSetAttribute(hbmm_umma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::BYTES);
      if (e != cudaSuccess) return e;
      configured[0] = true;
    }
    dim3 grid(static_cast<unsigned>((g.N + 63) / 64), static_cast<unsigned>((g.M + TM - 1) / TM));
    hbmm_umma_kernel<64><<<grid, kThreads, S::BYTES, stream>>>(g);
  } else {
    using S = Smem<128>;
    if (!configured[1]) {
      cudaError_t e = cudaFuncSetAttribute(hbmm_umma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::BYTES);
      if (e != cudaSuccess) return e;
      configured[1] = true;
    }
    dim3 grid(static_cast<unsigned>((g.N + 127) / 128), static_cast<unsigned>((g.M + TM - 1) / TM));
    hbmm_umma_kernel<128><<<grid, kThreads, S::BYTES, stream>>>(g);
  }
  return cudaGetLastError();
}

cudaError_t read_umma_error(int* code) {
  return cudaMemcpyFromSymbol(code, g_umma_error, sizeof(int));
}

}  // namespace hbmm
