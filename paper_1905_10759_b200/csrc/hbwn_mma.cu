// HBWN contraction on the tensor cores: bf16 activations x Hadamard-binary weights.
//   C[m,n] = sum_g deltaW[n,g] * sum_{k in g} s(W[n,k]) * A[m,k]
// The sign bits of a weight tile are expanded to +-1.0 bf16 in shared memory (a product of a bf16
// value with +-1 is exact), each weight group is contracted by mma.sync m16n8k16 into an fp32
// group partial, and the partial is folded into the accumulator with one fp32 FMA per output and
// group, so every group keeps its full-precision scale.
//
// CTA tile 128 x TN, 8 warps as 4 (M) x 2 (N), K walked in chunks of 64 elements through a
// 3-stage ring: activations arrive by 16-byte cp.async (zero-filled past M and K), the weight
// words of the chunk are expanded by the same threads one stage ahead.
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int kThreads = 256;
constexpr int TM = 128;
constexpr int KC = 64;            // K elements per stage (two 32-bit weight words)
constexpr int LDK = KC + 8;       // padded row length (bf16): 144-byte rows, conflict-free ldmatrix
constexpr int STAGES = 3;

struct Args {
  const __nv_bfloat16* a; int64_t lda;
  const uint32_t* w_bits; const void* w_scales; int64_t ldw_w, ldw_s; int32_t w_bf16;
  float* C; int64_t ldc;
  int64_t M, N, K, n_words, Gw;
  int64_t group_words;
};

__device__ __forceinline__ float load_scale(const void* s, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(s) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(s) + idx);
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16_zero(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};\n"
               : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.0f));
}

// Four sign bits -> four bf16 values (+1.0 = 0x3F80 for bit 1, -1.0 = 0xBF80 for bit 0), two per register.
__device__ __forceinline__ uint2 expand_nibble(uint32_t nib) {
  const uint32_t t = ~nib;
  uint2 r;
  r.x = 0x3F803F80u | ((t & 1u) << 15) | ((t & 2u) << 30);
  r.y = 0x3F803F80u | ((t & 4u) << 13) | ((t & 8u) << 28);
  return r;
}

// GW: weight-group length in words: 1 (beta 32), 2 (beta 64), 0 = a whole number of chunks (runtime).
template <int TN, int GW>
__global__ void __launch_bounds__(kThreads, 1)
hbwn_mma_kernel(const Args g) {
  constexpr int NT = TN / 16;   // n-tiles (8 columns) per warp
  constexpr int MT = 2;         // m-tiles (16 rows) per warp
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __nv_bfloat16* As = reinterpret_cast<__nv_bfloat16*>(smem_raw);                 // [STAGES][TM][LDK]
  __nv_bfloat16* Bs = As + STAGES * TM * LDK;                                     // [STAGES][TN][LDK]
  float* Ss = reinterpret_cast<float*>(Bs + STAGES * TN * LDK);                   // [STAGES][2][TN]
  __shared__ uint2 lut[16];

  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int wm = warp & 3, wn = warp >> 2;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * TM, n0 = static_cast<int64_t>(blockIdx.x) * TN;
  if (t < 16) lut[t] = expand_nibble(t);

  const int64_t n_chunks = (g.K + KC - 1) / KC;

  // ---- producers
  auto issue_a = [&](int64_t chunk, int stage) {
    // 128 rows x 8 sixteen-byte pieces = 1024 pieces, 4 per thread
#pragma unroll
    for (int p = 0; p < 4; p++) {
      const int piece = t + p * kThreads;
      const int row = piece >> 3, kp = (piece & 7) * 8;
      const int64_t m = m0 + row, k = chunk * KC + kp;
      int bytes = 0;
      if (m < g.M && k < g.K) bytes = (g.K - k >= 8) ? 16 : static_cast<int>(g.K - k) * 2;
      const __nv_bfloat16* src = g.a + (m < g.M ? m : 0) * g.lda + (k < g.K ? k : 0);
      cp_async16(smem_u32(As + (stage * TM + row) * LDK + kp), src, bytes);
    }
  };
  // weight words / scales of a chunk: thread -> (row = t % TN, sub-word = t / TN)
  constexpr int WORD_THREADS = TN * 2;
  const int wrow = t % TN, wsub = t / TN;
  auto fetch_w = [&](int64_t chunk, uint32_t& word, float& scale) {
    word = 0; scale = 0.0f;
    if (t < WORD_THREADS) {
      const int64_t n = n0 + wrow, kw = chunk * 2 + wsub;
      if (n < g.N) {
        if (kw < g.n_words) word = __ldg(g.w_bits + n * g.ldw_w + kw);
        // a word past the end of the row contributes zeros; it keeps the last group's scale so
        // that a flush at the end of the K walk still scales that group correctly
        int64_t grp = (kw < g.n_words ? kw : g.n_words - 1) / g.group_words;
        if (grp >= g.Gw) grp = g.Gw - 1;
        scale = load_scale(g.w_scales, g.w_bf16, n * g.ldw_s + grp);
      }
    }
  };
  auto expand_w = [&](int stage, uint32_t word, float scale) {
    if (t < WORD_THREADS) {
      uint4* dst = reinterpret_cast<uint4*>(Bs + (stage * TN + wrow) * LDK + wsub * 32);
#pragma unroll
      for (int q = 0; q < 4; q++) {
        const uint2 lo = lut[(word >> (8 * q)) & 15], hi = lut[(word >> (8 * q + 4)) & 15];
        dst[q] = make_uint4(lo.x, lo.y, hi.x, hi.y);
      }
      Ss[(stage * 2 + wsub) * TN + wrow] = scale;
    }
  };

  float acc[MT][NT][4], part[MT][NT][4];
#pragma unroll
  for (int i = 0; i < MT; i++)
#pragma unroll
    for (int j = 0; j < NT; j++)
#pragma unroll
      for (int e = 0; e < 4; e++) { acc[i][j][e] = 0.0f; part[i][j][e] = 0.0f; }

  __syncthreads();  // lut
  uint32_t wnext; float snext;
  // prologue: stages 0 and 1
  fetch_w(0, wnext, snext);
  issue_a(0, 0); cp_async_commit();
  expand_w(0, wnext, snext);
  if (n_chunks > 1) { fetch_w(1, wnext, snext); issue_a(1, 1); }
  cp_async_commit();
  if (n_chunks > 1) expand_w(1, wnext, snext);
  if (n_chunks > 2) fetch_w(2, wnext, snext);

  const int64_t chunks_per_group = (GW == 0) ? g.group_words / 2 : 1;
  for (int64_t chunk = 0; chunk < n_chunks; chunk++) {
    const int stage = static_cast<int>(chunk % STAGES);
    cp_async_wait<1>();
    __syncthreads();
    // refill the stage freed by the previous iteration
    if (chunk + 2 < n_chunks) {
      const int s2 = static_cast<int>((chunk + 2) % STAGES);
      issue_a(chunk + 2, s2);
      expand_w(s2, wnext, snext);
      if (chunk + 3 < n_chunks) fetch_w(chunk + 3, wnext, snext);
    }
    cp_async_commit();

    const __nv_bfloat16* a_st = As + stage * TM * LDK;
    const __nv_bfloat16* b_st = Bs + stage * TN * LDK;
#pragma unroll
    for (int sub = 0; sub < 2; sub++) {
#pragma unroll
      for (int ks = 0; ks < 2; ks++) {
        const int kk = sub * 32 + ks * 16;
        uint32_t af[MT][4];
#pragma unroll
        for (int i = 0; i < MT; i++)
          ldmatrix_x4(smem_u32(a_st + (wm * 32 + i * 16 + (lane & 15)) * LDK + kk + (lane >> 4) * 8),
                      af[i][0], af[i][1], af[i][2], af[i][3]);
#pragma unroll
        for (int jp = 0; jp < NT / 2; jp++) {
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(smem_u32(b_st + (wn * (TN / 2) + jp * 16 + (lane & 7) + (lane >> 4) * 8) * LDK + kk + ((lane >> 3) & 1) * 8),
                      b0, b1, b2, b3);
          const bool fresh = (GW == 1 && ks == 0) || (GW == 2 && sub == 0 && ks == 0);
#pragma unroll
          for (int i = 0; i < MT; i++) {
            if (fresh) {
              mma_bf16_zero(part[i][2 * jp], af[i], b0, b1);
              mma_bf16_zero(part[i][2 * jp + 1], af[i], b2, b3);
            } else {
              mma_bf16(part[i][2 * jp], af[i], b0, b1);
              mma_bf16(part[i][2 * jp + 1], af[i], b2, b3);
            }
          }
        }
      }
      // end of a weight group: fold the partial into the accumulator with the group's scale
      bool flush;
      if (GW == 1) flush = true;
      else if (GW == 2) flush = (sub == 1);
      else flush = (sub == 1) && (((chunk + 1) % chunks_per_group == 0) || chunk + 1 == n_chunks);
      if (flush) {
        const float* sc = Ss + (stage * 2 + sub) * TN + wn * (TN / 2) + (lane & 3) * 2;
#pragma unroll
        for (int j = 0; j < NT; j++) {
          const float2 s = *reinterpret_cast<const float2*>(sc + j * 8);
#pragma unroll
          for (int i = 0; i < MT; i++) {
            acc[i][j][0] = fmaf(s.x, part[i][j][0], acc[i][j][0]);
            acc[i][j][1] = fmaf(s.y, part[i][j][1], acc[i][j][1]);
            acc[i][j][2] = fmaf(s.x, part[i][j][2], acc[i][j][2]);
            acc[i][j][3] = fmaf(s.y, part[i][j][3], acc[i][j][3]);
            if (GW == 0) { part[i][j][0] = 0.f; part[i][j][1] = 0.f; part[i][j][2] = 0.f; part[i][j][3] = 0.f; }
          }
        }
      }
    }
  }
  cp_async_wait<0>();

  // ---- epilogue
#pragma unroll
  for (int i = 0; i < MT; i++)
#pragma unroll
    for (int h = 0; h < 2; h++) {
      const int64_t m = m0 + wm * 32 + i * 16 + (lane >> 2) + h * 8;
      if (m >= g.M) continue;
#pragma unroll
      for (int j = 0; j < NT; j++) {
        const int64_t n = n0 + wn * (TN / 2) + j * 8 + (lane & 3) * 2;
        float* dst = g.C + m * g.ldc + n;
        if (n + 1 < g.N) *reinterpret_cast<float2*>(dst) = make_float2(acc[i][j][2 * h], acc[i][j][2 * h + 1]);
        else if (n < g.N) dst[0] = acc[i][j][2 * h];
      }
    }
}

template <int TN>
constexpr size_t smem_bytes() {
  return static_cast<size_t>(STAGES) * (TM + TN) * LDK * 2 + static_cast<size_t>(STAGES) * 2 * TN * 4;
}

template <int TN, int GW>
cudaError_t launch(const Args& g, cudaStream_t stream) {
  constexpr size_t smem = smem_bytes<TN>();
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(hbwn_mma_kernel<TN, GW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid(static_cast<unsigned>((g.N + TN - 1) / TN), static_cast<unsigned>((g.M + TM - 1) / TM));
  hbwn_mma_kernel<TN, GW><<<grid, kThreads, smem, stream>>>(g);
  return cudaGetLastError();
}

}  // namespace

// bf16 activations with 16-byte aligned rows, weight groups of 32 / 64 bits or a whole number of
// 64-bit chunks (one group per row included).
bool hbwn_mma_supported(const DenseView& A, const PackedView& W) {
  if (!A.bf16) return false;
  if (reinterpret_cast<uintptr_t>(A.data) % 16 != 0 || (A.ld * 2) % 16 != 0) return false;
  if (W.beta >= W.K) return true;
  if (W.beta % 32 != 0) return false;       // sub-word groups: the tcgen05 and the sign-select kernels take them
  const int64_t gw = W.beta / 32;
  return gw == 1 || gw % 2 == 0;
}

cudaError_t launch_hbwn_mma(const DenseView& A, const PackedView& W, float* C, int64_t ldc, cudaStream_t stream) {
  Args g;
  g.a = reinterpret_cast<const __nv_bfloat16*>(A.data); g.lda = A.ld;
  g.w_bits = W.bits; g.w_scales = W.scales; g.ldw_w = W.ld_words; g.ldw_s = W.ld_scales; g.w_bf16 = W.scale_bf16;
  g.C = C; g.ldc = ldc; g.M = A.rows; g.N = W.rows; g.K = A.K;
  g.n_words = (A.K + 31) / 32;
  g.Gw = num_groups(W.K, W.beta);
  const bool one = W.beta >= W.K;
  // one group per row: a group as long as the padded K walk (even number of words)
  g.group_words = one ? ((g.n_words + 1) / 2) * 2 : W.beta / 32;
  const bool narrow = g.N <= 64;
  if (g.group_words == 1) return narrow ? launch<64, 1>(g, stream) : launch<128, 1>(g, stream);
  if (g.group_words == 2) return narrow ? launch<64, 2>(g, stream) : launch<128, 2>(g, stream);
  return narrow ? launch<64, 0>(g, stream) : launch<128, 0>(g, stream);
}

}  // namespace hbmm
