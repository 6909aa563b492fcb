// HBMM contraction on the integer pipe for sub-word segments (Section 4.2, Eq. 7 with the group sizes
// of the paper's experiments, beta = 2 .. 16): the segment min(beta_a, beta_w) is 2, 4, 8 or 16 bits, so one
// XOR word holds 32 / segment group dots, each read with a shifted, masked popcount:
//   D = n_valid - 2 * popc(((a ^ w) >> shift) & mask),   C += (deltaA * deltaW) * D.
// This is the workspace-free path for these group sizes (the tensor-core kernel needs the expanded
// weights) and the source of the integer partials; it is written for clarity, not for speed: a 16 x 16
// output tile per CTA, one output per thread, packed words and the scales of both operands (already
// looked up per segment) staged in shared memory per chunk of KC words.
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int TS = 16;     // tile side
constexpr int KC = 2;      // K-words per chunk
constexpr int MAXSEG = KC * 16;   // segments per chunk at 2 bits per segment

struct SubArgs {
  const uint32_t* a_bits; const void* a_scales;
  const uint32_t* w_bits; const void* w_scales;
  float* C;
  int64_t M, N, K, lda_w, ldw_w, lda_s, ldw_s, ldc;
  int32_t a_bf16, w_bf16;
  int32_t seg;                 // bits per segment: 2, 4, 8 or 16
  int64_t a_beta, w_beta;      // group length in elements (K when there is one group per row)
  int64_t n_words, T;          // ceil(K / 32), ceil(K / seg)
};

__device__ __forceinline__ float load_scale(const void* s, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(s) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(s) + idx);
}

__global__ void __launch_bounds__(TS * TS)
gemm_popc_sub_kernel(const SubArgs g) {
  __shared__ uint32_t As[TS][KC], Ws[TS][KC];
  __shared__ float Sa[TS][MAXSEG + 1], Sw[TS][MAXSEG + 1];
  const int tx = threadIdx.x % TS, ty = threadIdx.x / TS;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * TS, n0 = static_cast<int64_t>(blockIdx.x) * TS;
  const int spw = 32 / g.seg;                        // segments per word
  const int spc = spw * KC;                          // segments per chunk
  const uint32_t mask = (1u << g.seg) - 1u;
  float acc = 0.0f;
  for (int64_t w0 = 0; w0 < g.n_words; w0 += KC) {
    __syncthreads();
    // stage: threads 0..TS*KC-1 the words of A, the next TS*KC those of W; everyone the scales
    for (int i = threadIdx.x; i < 2 * TS * KC; i += TS * TS) {
      const int which = i / (TS * KC), r = (i % (TS * KC)) / KC, c = i % KC;
      const int64_t row = (which ? n0 : m0) + r, wi = w0 + c;
      const bool in = row < (which ? g.N : g.M) && wi < g.n_words;
      const uint32_t v = in ? __ldg((which ? g.w_bits : g.a_bits) + row * (which ? g.ldw_w : g.lda_w) + wi) : 0u;
      if (which) Ws[r][c] = v; else As[r][c] = v;
    }
    for (int i = threadIdx.x; i < 2 * TS * spc; i += TS * TS) {
      const int which = i / (TS * spc), r = (i % (TS * spc)) / spc, t = i % spc;
      const int64_t row = (which ? n0 : m0) + r;
      const int64_t k0 = (w0 * spw + t) * g.seg;     // first element of the segment
      float v = 0.0f;
      if (row < (which ? g.N : g.M) && k0 < g.K)
        v = which ? load_scale(g.w_scales, g.w_bf16, row * g.ldw_s + k0 / g.w_beta)
                  : load_scale(g.a_scales, g.a_bf16, row * g.lda_s + k0 / g.a_beta);
      if (which) Sw[r][t] = v; else Sa[r][t] = v;
    }
    __syncthreads();
    for (int c = 0; c < KC; c++) {
      const uint32_t x = As[ty][c] ^ Ws[tx][c];
      for (int s = 0; s < spw; s++) {
        const int64_t k0 = ((w0 + c) * spw + s) * g.seg;
        if (k0 >= g.K) break;
        const int64_t left = g.K - k0;
        const int nv = left < g.seg ? static_cast<int>(left) : g.seg;      // pad bits are zero in both operands
        const int d = nv - 2 * __popc((x >> (s * g.seg)) & mask);
        acc = fmaf(Sa[ty][c * spw + s] * Sw[tx][c * spw + s], static_cast<float>(d), acc);
      }
    }
  }
  const int64_t m = m0 + ty, n = n0 + tx;
  if (m < g.M && n < g.N) g.C[m * g.ldc + n] = acc;
}

// D[m,n,t] = n_valid(t) - 2 * popc over the bits of segment t.
__global__ void __launch_bounds__(256)
partials_popc_sub_kernel(const SubArgs g, int32_t* __restrict__ D) {
  const int64_t total = g.M * g.N * g.T;
  const uint32_t mask = (1u << g.seg) - 1u;
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; idx < total; idx += static_cast<int64_t>(gridDim.x) * 256) {
    const int64_t t = idx % g.T, mn = idx / g.T;
    const int64_t n = mn % g.N, m = mn / g.N;
    const int64_t k0 = t * g.seg;
    const uint32_t x = g.a_bits[m * g.lda_w + (k0 >> 5)] ^ g.w_bits[n * g.ldw_w + (k0 >> 5)];
    const int64_t left = g.K - k0;
    const int nv = left < g.seg ? static_cast<int>(left) : g.seg;
    D[idx] = nv - 2 * __popc((x >> (k0 & 31)) & mask);
  }
}

SubArgs make_args(const PackedView& A, const PackedView& W, float* C, int64_t ldc) {
  SubArgs g;
  g.a_bits = A.bits; g.a_scales = A.scales; g.w_bits = W.bits; g.w_scales = W.scales; g.C = C;
  g.M = A.rows; g.N = W.rows; g.K = A.K;
  g.lda_w = A.ld_words; g.ldw_w = W.ld_words; g.lda_s = A.ld_scales; g.ldw_s = W.ld_scales; g.ldc = ldc;
  g.a_bf16 = A.scale_bf16; g.w_bf16 = W.scale_bf16;
  g.a_beta = A.beta >= A.K ? A.K : A.beta;
  g.w_beta = W.beta >= W.K ? W.K : W.beta;
  g.seg = static_cast<int32_t>(g.a_beta < g.w_beta ? g.a_beta : g.w_beta);
  g.n_words = (A.K + 31) / 32;
  g.T = (A.K + g.seg - 1) / g.seg;
  return g;
}

}  // namespace

// The finer of the two groupings is a sub-word power of two (and not a whole row).
bool gemm_subword(const PackedView& A, const PackedView& W) {
  const int64_t a = A.beta >= A.K ? A.K : A.beta, w = W.beta >= W.K ? W.K : W.beta;
  const int64_t seg = a < w ? a : w;
  return seg < 32 && (seg == 2 || seg == 4 || seg == 8 || seg == 16) && seg < A.K;
}

cudaError_t launch_gemm_popc_sub(const PackedView& A, const PackedView& W, float* C, int64_t ldc, cudaStream_t stream) {
  const SubArgs g = make_args(A, W, C, ldc);
  dim3 grid(static_cast<unsigned>((g.N + TS - 1) / TS), static_cast<unsigned>((g.M + TS - 1) / TS));
  gemm_popc_sub_kernel<<<grid, TS * TS, 0, stream>>>(g);
  return cudaGetLastError();
}

cudaError_t launch_partials_popc_sub(const PackedView& A, const PackedView& W, int32_t* D, cudaStream_t stream) {
  const SubArgs g = make_args(A, W, nullptr, 0);
  const int64_t total = g.M * g.N * g.T;
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  if (blocks < 1) blocks = 1;
  partials_popc_sub_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(g, D);
  return cudaGetLastError();
}

}  // namespace hbmm
