// HBMM contraction on the legacy single-bit tensor instruction (mma.sync ... b1 xor.popc).
//
// One mma.sync.m16n8k128 adds popc(a ^ w) over 128 K-bits to a 16 x 8 tile of int32 counters, so a
// segment must be a whole number of 128-bit chunks (beta a multiple of 128, or one group per row).
// The signed dot of a segment is n_valid - 2 * count (Section 4.2, Eq. 7; pad bits are zero in both
// operands and never count); the fp32 scale epilogue is the same as on the integer-pipe path.
// On B200 this instruction runs far below the other two paths (it is kept for comparison): the
// kernel is a plain one, fragments are read straight from global memory through L1.
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int kThreads = 128;   // 4 warps, each 16 rows x 64 columns of a 64 x 64 CTA tile

__device__ __forceinline__ float load_scale(const void* s, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(s) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(s) + idx);
}

struct B1Args {
  const uint32_t* a_bits; const void* a_scales;
  const uint32_t* w_bits; const void* w_scales;
  float* C; int32_t* D;
  int64_t M, N, K, lda_w, ldw_w, lda_s, ldw_s, ldc;
  int32_t a_bf16, w_bf16, ra, rw;
  int64_t n_chunks;     // 128-bit chunks per row
  int64_t seg_chunks;   // chunks per segment
  int64_t T;            // segments
};

// c[0..3] += popc(A ^ B): A 16 x 128 bits (a0: row lane/4, a1: row lane/4 + 8; bits 32*(lane%4)..),
// B 128 bits x 8 columns (column lane/4, same bits).  c0,c1: row lane/4, columns 2*(lane%4), +1;
// c2,c3: row lane/4 + 8.
__device__ __forceinline__ void mma_b1(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm volatile("mma.sync.aligned.m16n8k128.row.col.s32.b1.b1.s32.xor.popc {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};\n"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a0), "r"(a1), "r"(b0));
}

template <bool PARTIALS>
__global__ void __launch_bounds__(kThreads)
gemm_b1_kernel(const B1Args g) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int grp = lane >> 2, tig = lane & 3;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * 64 + warp * 16, n0 = static_cast<int64_t>(blockIdx.x) * 64;
  const int64_t ma = m0 + grp, mb = m0 + grp + 8;
  const uint32_t* a_row0 = g.a_bits + (ma < g.M ? ma : 0) * g.lda_w + tig;
  const uint32_t* a_row1 = g.a_bits + (mb < g.M ? mb : 0) * g.lda_w + tig;
  const uint32_t* w_row[8];
#pragma unroll
  for (int j = 0; j < 8; j++) {
    const int64_t n = n0 + j * 8 + grp;
    w_row[j] = g.w_bits + (n < g.N ? n : 0) * g.ldw_w + tig;
  }
  float acc[8][4];
  int cnt[8][4];
#pragma unroll
  for (int j = 0; j < 8; j++)
#pragma unroll
    for (int e = 0; e < 4; e++) { acc[j][e] = 0.0f; cnt[j][e] = 0; }

  int64_t seg = 0, in_seg = 0;
  for (int64_t ch = 0; ch < g.n_chunks; ch++) {
    const uint32_t a0 = __ldg(a_row0 + ch * 4), a1 = __ldg(a_row1 + ch * 4);
#pragma unroll
    for (int j = 0; j < 8; j++) mma_b1(cnt[j], a0, a1, __ldg(w_row[j] + ch * 4));
    if (++in_seg == g.seg_chunks || ch == g.n_chunks - 1) {
      int64_t nv = g.K - seg * g.seg_chunks * 128;
      if (nv > g.seg_chunks * 128) nv = g.seg_chunks * 128;
      if (PARTIALS) {
#pragma unroll
        for (int j = 0; j < 8; j++)
#pragma unroll
          for (int e = 0; e < 4; e++) {
            const int64_t m = (e < 2) ? ma : mb, n = n0 + j * 8 + tig * 2 + (e & 1);
            if (m < g.M && n < g.N) g.D[(m * g.N + n) * g.T + seg] = static_cast<int32_t>(nv) - 2 * cnt[j][e];
            cnt[j][e] = 0;
          }
      } else {
        const int64_t ga = seg / g.ra, gw = seg / g.rw;
        const float sa0 = ma < g.M ? load_scale(g.a_scales, g.a_bf16, ma * g.lda_s + ga) : 0.0f;
        const float sa1 = mb < g.M ? load_scale(g.a_scales, g.a_bf16, mb * g.lda_s + ga) : 0.0f;
#pragma unroll
        for (int j = 0; j < 8; j++) {
          const int64_t n = n0 + j * 8 + tig * 2;
          const float sw0 = n < g.N ? load_scale(g.w_scales, g.w_bf16, n * g.ldw_s + gw) : 0.0f;
          const float sw1 = n + 1 < g.N ? load_scale(g.w_scales, g.w_bf16, (n + 1) * g.ldw_s + gw) : 0.0f;
#pragma unroll
          for (int e = 0; e < 4; e++) {
            const float d = static_cast<float>(static_cast<int>(nv) - 2 * cnt[j][e]);
            acc[j][e] = fmaf(d * (e < 2 ? sa0 : sa1), (e & 1) ? sw1 : sw0, acc[j][e]);
            cnt[j][e] = 0;
          }
        }
      }
      seg++;
      in_seg = 0;
    }
  }
  if (!PARTIALS) {
#pragma unroll
    for (int j = 0; j < 8; j++)
#pragma unroll
      for (int e = 0; e < 4; e++) {
        const int64_t m = (e < 2) ? ma : mb, n = n0 + j * 8 + tig * 2 + (e & 1);
        if (m < g.M && n < g.N) g.C[m * g.ldc + n] = acc[j][e];
      }
  }
}

bool make_args(const PackedView& A, const PackedView& W, B1Args& g) {
  const bool a_one = A.beta >= A.K, w_one = W.beta >= W.K;
  if ((!a_one && A.beta % 128 != 0) || (!w_one && W.beta % 128 != 0)) return false;
  g.a_bits = A.bits; g.a_scales = A.scales; g.w_bits = W.bits; g.w_scales = W.scales;
  g.C = nullptr; g.D = nullptr;
  g.M = A.rows; g.N = W.rows; g.K = A.K; g.lda_w = A.ld_words; g.ldw_w = W.ld_words;
  g.lda_s = A.ld_scales; g.ldw_s = W.ld_scales; g.ldc = 0;
  g.a_bf16 = A.scale_bf16; g.w_bf16 = W.scale_bf16;
  g.n_chunks = (A.K + 127) / 128;      // rows are padded to whole 128-bit chunks (ld_words % 4 == 0)
  int64_t seg;
  if (a_one && w_one) seg = g.n_chunks * 128;
  else if (a_one) seg = W.beta;
  else if (w_one) seg = A.beta;
  else seg = A.beta < W.beta ? A.beta : W.beta;
  g.seg_chunks = seg / 128;
  g.T = (A.K + seg - 1) / seg;
  g.ra = static_cast<int32_t>(a_one ? g.T : A.beta / seg);
  g.rw = static_cast<int32_t>(w_one ? g.T : W.beta / seg);
  return true;
}

}  // namespace

bool gemm_b1_supported(const PackedView& A, const PackedView& W) {
  B1Args g;
  return make_args(A, W, g);
}

cudaError_t launch_gemm_b1(const PackedView& A, const PackedView& W, float* C, int64_t ldc, cudaStream_t stream) {
  B1Args g;
  if (!make_args(A, W, g)) return cudaErrorNotSupported;
  g.C = C; g.ldc = ldc;
  dim3 grid(static_cast<unsigned>((g.N + 63) / 64), static_cast<unsigned>((g.M + 63) / 64));
  gemm_b1_kernel<false><<<grid, kThreads, 0, stream>>>(g);
  return cudaGetLastError();
}

cudaError_t launch_partials_b1(const PackedView& A, const PackedView& W, int32_t* D, cudaStream_t stream) {
  B1Args g;
  if (!make_args(A, W, g)) return cudaErrorNotSupported;
  g.D = D;
  dim3 grid(static_cast<unsigned>((g.N + 63) / 64), static_cast<unsigned>((g.M + 63) / 64));
  gemm_b1_kernel<true><<<grid, kThreads, 0, stream>>>(g);
  return cudaGetLastError();
}

}  // namespace hbmm
