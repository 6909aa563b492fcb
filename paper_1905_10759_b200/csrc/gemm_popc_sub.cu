// HBMM contraction on the integer pipe for sub-word segments (Section 4.2, Eq. 7 with the group sizes
// of the paper's experiments, beta = 2 .. 16): the segment min(beta_a, beta_w) is 2, 4, 8 or 16 bits, so one
// XOR word holds 32 / segment group dots, each read with a shifted, masked popcount:
//   D = n_valid - 2 * popc(((a ^ w) >> shift) & mask),   C += (deltaA * deltaW) * D.
// This is the workspace-free path for these group sizes (the tensor-core kernel needs the expanded
// weights) and the source of the integer partials.  The work is one fp32 multiply-add with its own scale
// product per output and SEGMENT (M N K / segment of them: at 2-bit segments half a dense fp32 product), so
// the path is bound by the fp32 / integer pipes however it is tiled; the kernel keeps the per-segment
// sequence at six instructions and the operands in registers.
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int TT = 64;     // tile side
constexpr int KC = 2;      // K-words per chunk

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

// SEG: bits per segment.  256 threads, a 64 x 64 output tile per CTA, a 4 x 4 register tile per thread.  K is walked
// in chunks of KC words; the chunk's packed words and the scales of its segments (looked up per segment, the
// activation ones times -1 folded into nothing: see below) are staged k-major in shared memory, so a thread reads its
// four rows / columns as one 16-byte vector.  Per output and segment: one bit-field extract, one popcount, one
// integer multiply-add forming (n_valid - 2 p) + 0x4B400000 -- the bit pattern of the float 1.5 * 2^23 + (n_valid - 2 p),
// so the conversion to float is one subtraction -- one multiply for the scale product and one fused multiply-add.
template <int SEG>
__global__ void __launch_bounds__(256)
gemm_popc_sub_kernel(const SubArgs g) {
  constexpr int SPW = 32 / SEG;            // segments per word
  constexpr int SPC = SPW * KC;            // segments per chunk
  constexpr int LD = TT + 4;               // row pitch of the k-major tiles (words)
  constexpr uint32_t kMagic = 0x4B400000u; // 1.5 * 2^23: small signed integers added to it stay in its binade
  __shared__ __align__(16) uint32_t As[KC][LD], Ws[KC][LD];
  __shared__ __align__(16) float Sa[SPC][LD], Sw[SPC][LD];
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * TT, n0 = static_cast<int64_t>(blockIdx.x) * TT;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int j = 0; j < 4; j++) acc[i][j] = 0.0f;

  for (int64_t w0 = 0; w0 < g.n_words; w0 += KC) {
    __syncthreads();
    // stage: the first 64 * KC threads' worth of items are the words of A, the next those of W; then the scales
    for (int i = t; i < 2 * TT * KC; i += 256) {
      const int which = i / (TT * KC), r = (i % (TT * KC)) % TT, c = (i % (TT * KC)) / TT;
      const int64_t row = (which ? n0 : m0) + r, wi = w0 + c;
      const bool in = row < (which ? g.N : g.M) && wi < g.n_words;
      const uint32_t v = in ? __ldg((which ? g.w_bits : g.a_bits) + row * (which ? g.ldw_w : g.lda_w) + wi) : 0u;
      if (which) Ws[c][r] = v; else As[c][r] = v;
    }
    for (int i = t; i < 2 * TT * SPC; i += 256) {
      const int which = i / (TT * SPC), r = (i % (TT * SPC)) % TT, sg = (i % (TT * SPC)) / TT;
      const int64_t row = (which ? n0 : m0) + r;
      const int64_t k0 = (w0 * SPW + sg) * SEG;      // first element of the segment
      float v = 0.0f;
      if (row < (which ? g.N : g.M) && k0 < g.K)
        v = which ? load_scale(g.w_scales, g.w_bf16, row * g.ldw_s + k0 / g.w_beta)
                  : load_scale(g.a_scales, g.a_bf16, row * g.lda_s + k0 / g.a_beta);
      if (which) Sw[sg][r] = v; else Sa[sg][r] = v;
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < KC; c++) {
      const uint4 av = *reinterpret_cast<const uint4*>(&As[c][ty * 4]);
      const uint4 wv = *reinterpret_cast<const uint4*>(&Ws[c][tx * 4]);
      const uint32_t aw[4] = {av.x, av.y, av.z, av.w}, ww[4] = {wv.x, wv.y, wv.z, wv.w};
      uint32_t x[4][4];
#pragma unroll
      for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) x[i][j] = aw[i] ^ ww[j];
      // valid bits of the chunk word's segments: all SEG except in the row's last word (pad bits are zero in both operands)
      const int64_t left_word = g.K - (w0 + c) * 32;
#pragma unroll
      for (int sg = 0; sg < SPW; sg++) {
        const int64_t left = left_word - sg * SEG;
        const int nv = left >= SEG ? SEG : (left > 0 ? static_cast<int>(left) : 0);
        const uint32_t bias = kMagic + static_cast<uint32_t>(nv);
        const float4 sa4 = *reinterpret_cast<const float4*>(&Sa[c * SPW + sg][ty * 4]);
        const float4 sw4 = *reinterpret_cast<const float4*>(&Sw[c * SPW + sg][tx * 4]);
        const float sa[4] = {sa4.x, sa4.y, sa4.z, sa4.w}, sw[4] = {sw4.x, sw4.y, sw4.z, sw4.w};
#pragma unroll
        for (int i = 0; i < 4; i++)
#pragma unroll
          for (int j = 0; j < 4; j++) {
            const uint32_t p = __popc((x[i][j] >> (sg * SEG)) & ((1u << SEG) - 1u));
            const float d = __uint_as_float(bias - 2u * p) - 12582912.0f;       // n_valid - 2 p, exactly
            acc[i][j] = fmaf(sa[i] * sw[j], d, acc[i][j]);
          }
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const int64_t m = m0 + ty * 4 + i;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const int64_t n = n0 + tx * 4 + j;
      if (m < g.M && n < g.N) g.C[m * g.ldc + n] = acc[i][j];
    }
  }
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
  dim3 grid(static_cast<unsigned>((g.N + TT - 1) / TT), static_cast<unsigned>((g.M + TT - 1) / TT));
  switch (g.seg) {
    case 2: gemm_popc_sub_kernel<2><<<grid, 256, 0, stream>>>(g); break;
    case 4: gemm_popc_sub_kernel<4><<<grid, 256, 0, stream>>>(g); break;
    case 8: gemm_popc_sub_kernel<8><<<grid, 256, 0, stream>>>(g); break;
    default: gemm_popc_sub_kernel<16><<<grid, 256, 0, stream>>>(g); break;
  }
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
