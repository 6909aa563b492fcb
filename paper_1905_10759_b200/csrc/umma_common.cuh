// Device helpers shared by the tcgen05 / TMEM kernels: mbarriers with bounded waits, bulk copies,
// tensor-memory allocation and loads, UMMA descriptors for 128-byte-swizzled K-major operands.
// Every kernel file that includes this gets its own error word (static linkage).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace hbmm {
namespace umma {

static __device__ int g_error_word = 0;    // 0 = ok; otherwise the code of the first wait that gave up (kept until cleared)
constexpr uint32_t kSpinLimit = 1u << 20;   // polls of a (hardware time-limited) try_wait
static __device__ uint32_t g_spin_limit = kSpinLimit;   // the limit in force: the default unless a test lowered it
// Teardown waits -- for asynchronous work that has already been issued and only needs to land -- ignore the
// abort flag and use this many polls: far longer than a copy or an MMA batch takes, short next to kSpinLimit.
constexpr uint32_t kDrainPolls = 1u << 14;
constexpr int TM = 128;                     // rows of every UMMA tile (= TMEM lanes)

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
// The same on a precomputed shared-memory address (keeps the single-thread issue loops short).
__device__ __forceinline__ bool mbar_try_wait_a(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ void umma_commit_a(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Bounded wait.  Returns false when the limit expired or another thread aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint32_t limit = g_spin_limit;             // read on the slow path only
  for (uint32_t it = 0; it < limit; it++) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
  }
  atomicCAS(&g_error_word, 0, code);
  *abort_flag = 1;
  return false;
}
// Bounded wait that does not look at the abort flag and records nothing: used on the way out, where work
// already handed to the copy engine or the tensor core must finish before shared or tensor memory goes away.
__device__ __forceinline__ bool mbar_wait_quiet(uint64_t* bar, uint32_t parity, uint32_t polls) {
  for (uint32_t it = 0; it < polls; it++)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Asynchronous bulk copy global -> this CTA's shared memory (both 16-byte aligned, size a multiple of
// 16); completion is counted in bytes on the mbarrier.  The copy targets this CTA alone.
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Tiled 2-D tensor copy global -> this CTA's shared memory through a tensor map (this CTA alone).
// x (innermost coordinate) times the element size must be a multiple of 16 bytes; rows and columns
// outside the tensor arrive as zeros and still count towards the transaction bytes.
__device__ __forceinline__ void tma_load_2d(void* dst, const void* tensor_map, int32_t x, int32_t y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(smem_u32(dst)), "l"(tensor_map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
// The same for a 4-D tensor (x innermost).  Loads may start at negative or out-of-range coordinates
// (x still 16-byte aligned): whatever lies outside the tensor arrives as zeros.
__device__ __forceinline__ void tma_load_4d(void* dst, const void* tensor_map, int32_t x, int32_t y, int32_t z, int32_t w,
                                            uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
               ::"r"(smem_u32(dst)), "l"(tensor_map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(smem_u32(bar)) : "memory");
}
// im2col-mode tensor copy of an NHWC image: `pixels-per-column` consecutive base pixels starting at
// (w, h, n) (walking W, then H, then N inside the map's bounding box), each displaced by the filter
// offsets (w_off, h_off), `channels-per-pixel` channels from c.  c times the element size must be a
// multiple of 16 bytes; pixels outside the image arrive as zeros.  This CTA alone.
__device__ __forceinline__ void tma_load_im2col_4d(void* dst, const void* tensor_map, int32_t c, int32_t w, int32_t h, int32_t n,
                                                   uint16_t w_off, uint16_t h_off, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6], {%7, %8};"
               ::"r"(smem_u32(dst)), "l"(tensor_map), "r"(c), "r"(w), "r"(h), "r"(n), "r"(smem_u32(bar)), "h"(w_off), "h"(h_off)
               : "memory");
}

// ---- tcgen05 helpers
__device__ __forceinline__ bool mbar_wait_a(uint32_t bar, uint32_t parity, volatile int* abort_flag, int code) {
  if (mbar_try_wait_a(bar, parity)) return true;
  const uint32_t limit = g_spin_limit;
  for (uint32_t it = 0; it < limit; it++) {
    if (mbar_try_wait_a(bar, parity)) return true;
    if (*abort_flag) return false;
  }
  atomicCAS(&g_error_word, 0, code);
  *abort_flag = 1;
  return false;
}
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
__device__ __forceinline__ void tmem_ld16(uint32_t addr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(addr));
}
// Registers -> tensor memory: thread i of the warp writes lane (32 * (warp % 4) + i), 16 consecutive columns
// from the address's column.  Asynchronous: tmem_st_wait before anything is told that the data is there.
__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(addr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
        "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D[tmem] (+)= A[tmem] * B[smem desc]^T, 128 x N x 16, 16-bit operands (type by the instruction descriptor), fp32
// accumulate.  A: row r in lane r, the 16 K-elements in 8 consecutive 32-bit columns (two per column, the
// lower K index in the low half).
__device__ __forceinline__ void umma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld_piece(uint32_t addr, uint32_t (&v)[32]) { tmem_ld32(addr, v); }
__device__ __forceinline__ void tmem_ld_piece(uint32_t addr, uint32_t (&v)[16]) { tmem_ld16(addr, v); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
template <int R> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(R)); }
template <int R> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(R)); }

// Two fp32 lanes per instruction (halves the issue slots of the scale epilogue).
__device__ __forceinline__ uint64_t pack2(uint32_t lo, uint32_t hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
// D[tmem] (+)= A[smem desc] * B[smem desc]^T, 128 x N x 16, bf16 (or, by the instruction descriptor, fp16)
// operands, fp32 accumulate.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// 16-byte asynchronous copy global -> shared; bytes beyond src_bytes are filled with zeros.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }
// D[tmem] = A[smem desc] * B[smem desc]^T, 128 x N x 16, bf16 operands, fp32 result (overwrites).
__device__ __forceinline__ void umma_bf16_overwrite(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc) : "memory");
}

// ---- CTA pairs: a cluster of two CTAs on neighbouring SMs issues one MMA over 256 rows (128 per CTA) whose
// second operand is split between the two CTAs' shared memories, so each CTA stages and serves half of it.
// The CTA of cluster rank 0 issues the MMAs and owns the barriers the copies of both CTAs complete on.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// every thread of both CTAs
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in the CTA of the given cluster rank (shared::cluster window)
__device__ __forceinline__ uint32_t mapa_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Tensor memory of both CTAs at once: the same warp of each CTA executes these with the same arguments.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols));
}
__device__ __forceinline__ void tmem_relinquish_pair() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::); }
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols));
}
// D[tmem of both CTAs] (+)= A * B^T, 256 x N x 16: each CTA's descriptor addresses name its own 128 rows of A and
// its own N / 2 rows of B.  Issued by one thread of the rank-0 CTA.
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives, once the pair's MMAs issued so far have completed, on the barrier at this address in every CTA of the mask.
__device__ __forceinline__ void umma_commit_pair_mc(uint32_t bar, uint16_t cta_mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(cta_mask) : "memory");
}
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Tensor copies into this CTA's shared memory whose bytes complete on a barrier of either CTA of the pair
// (`bar` is a shared::cluster address).  No multicast: each CTA fetches its own tiles.
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const void* tensor_map, int32_t x, int32_t y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(smem_u32(dst)), "l"(tensor_map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_im2col_4d_pair(void* dst, const void* tensor_map, int32_t c, int32_t w, int32_t h, int32_t n,
                                                        uint16_t w_off, uint16_t h_off, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.4d.im2col.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6], {%7, %8};"
               ::"r"(smem_u32(dst)), "l"(tensor_map), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar), "h"(w_off), "h"(h_off)
               : "memory");
}

// Operand tiles in shared memory use the 128-byte-swizzled K-major layout of the tensor core: a row is
// 128 contiguous bytes (the four K-words of a stage, 32 bytes each), rows follow each other, and the
// 16-byte piece c of row r is stored at piece position c ^ (r % 8).  A tile starts on a 1024-byte
// boundary; the instruction for word slot q reads from byte offset 32*q of the rows.
__device__ __forceinline__ unsigned char* swz(unsigned char* tile, int row, int piece) {
  return tile + row * 128 + ((piece ^ (row & 7)) << 4);
}
// Shared-memory descriptor of a K-major, 128-byte-swizzled operand: start address, stride between
// 8-row groups = 1024 bytes, descriptor version 1, layout type 2 (128-byte swizzle); the leading
// offset is not used by this layout.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr >> 4) & 0x3FFF);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// Instruction descriptors: fp32 accumulator, both operands K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc(int n, uint32_t ab_format) {
  return (1u << 4) | (ab_format << 7) | (ab_format << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(TM >> 4) << 24);
}
// The same for a CTA pair: M = 256 (128 rows in each CTA).
__host__ __device__ constexpr uint32_t instr_desc_pair(int n, uint32_t ab_format) {
  return (1u << 4) | (ab_format << 7) | (ab_format << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>((2 * TM) >> 4) << 24);
}
constexpr uint32_t kFmtE4M3 = 0, kFmtBF16 = 1;   // kind::f8f6f4 / kind::f16 operand codes
constexpr uint32_t kFmtF16 = 0;                  // kind::f16 with fp16 operands

// Host side of this translation unit's health word and spin limit (each file that includes this header has
// its own copies, hence internal linkage).  All three synchronise with the device.
static inline cudaError_t read_error_word(int* code) { return cudaMemcpyFromSymbol(code, g_error_word, sizeof(int)); }
static inline cudaError_t clear_error_word() {
  const int zero = 0;
  return cudaMemcpyToSymbol(g_error_word, &zero, sizeof(int));
}
static inline cudaError_t set_spin_limit(uint32_t polls) {     // 0 restores the default
  const uint32_t v = polls == 0 ? kSpinLimit : polls;
  return cudaMemcpyToSymbol(g_spin_limit, &v, sizeof(uint32_t));
}

}  // namespace umma
}  // namespace hbmm
