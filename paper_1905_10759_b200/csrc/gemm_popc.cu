// HBMM contraction of two packed operands on the integer pipe (Section 4.2, Eq. 7).
//
// For every output element and every 32-bit K-word: p = popc(a ^ w); the signed +-1 dot of a
// K-segment is D = n_valid - 2 * sum(p); C += (deltaA * deltaW) * D in fp32.  The segment is
// min(beta_a, beta_w); the operand with the coarser groups reuses its scale across segments.
//
// Tiling: 256 threads, each owning an (4*IM) x (4*JN) register tile of C; a CTA covers
// (64*IM) x (64*JN).  K is walked in chunks of 8 words.  Packed bits and the scales of the
// chunk's segments are staged k-major in shared memory (so a thread's rows/columns are
// 16-byte vectors), double buffered, with the next chunk prefetched into registers during the
// math.  int -> float goes through the 2^23 magic number (no conversion instruction):
// float(0x4B000000 | p) - (2^23 + 16*SW) == sum(p) - n/2 exactly, and the factor -2 is folded
// into the staged A scale.  Pad bits are zero in both operands, so they add nothing to the
// popcount; a shorter tail segment is left out of the loop and added once in the epilogue.
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int kThreads = 256;
constexpr int KC = 8;      // K-words per stage
constexpr int LDS_PAD = 4; // row padding (words) of the k-major tiles: conflict-free transposed stores

__device__ __forceinline__ float load_scale(const void* s, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(s) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(s) + idx);
}

struct GemmArgs {
  const uint32_t* a_bits; const void* a_scales;
  const uint32_t* w_bits; const void* w_scales;
  float* C;
  int64_t M, N, K, lda_w, ldw_w, lda_s, ldw_s, ldc;
  int32_t a_bf16, w_bf16;
  int32_t ra, rw;        // groups: A group = segment / ra, W group = segment / rw
  int64_t Ga, Gw;        // number of groups per row
  int64_t n_words;       // ceil(K/32)
  int64_t T;             // number of segments
  int32_t seg_words;     // words per segment
  int32_t tail_pad;      // (segment bits) - (valid bits of the last segment), 0 when K % segment == 0
};

// SW: words per segment (1, 2, 4 or 8).  IM, JN: 4-row / 4-column blocks per thread.
template <int SW, int IM, int JN>
__global__ void __launch_bounds__(kThreads, SW == 1 ? 2 : 1)
gemm_popc_kernel(const GemmArgs g) {
  constexpr int TM = 64 * IM, TN = 64 * JN;
  constexpr int NSEG = KC / SW;
  constexpr int LDA = TM + LDS_PAD, LDW = TN + LDS_PAD;
  constexpr int RA = TM / 128 > 0 ? TM / 128 : 1;  // bit rows staged per thread (A): 2 threads per row
  constexpr int RW = TN / 128 > 0 ? TN / 128 : 1;
  __shared__ __align__(16) uint32_t As[2][KC][LDA];
  __shared__ __align__(16) uint32_t Ws[2][KC][LDW];
  __shared__ __align__(16) float AsS[2][NSEG][LDA];
  __shared__ __align__(16) float WsS[2][NSEG][LDW];

  const int t = threadIdx.x;
  const int tx = t & 15, ty = t >> 4;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * TM, n0 = static_cast<int64_t>(blockIdx.x) * TN;
  const int half = t & 1, lrow = t >> 1;  // staging: 2 threads per row, 4 words each

  float acc[4 * IM][4 * JN];
#pragma unroll
  for (int i = 0; i < 4 * IM; i++)
#pragma unroll
    for (int j = 0; j < 4 * JN; j++) acc[i][j] = 0.0f;

  uint4 pa[RA], pw[RW];
  float psa[RA][(NSEG + 1) / 2], psw[RW][(NSEG + 1) / 2];

  const int64_t n_chunks = (g.n_words + KC - 1) / KC;

  auto prefetch = [&](int64_t chunk) {
    const int64_t kw = chunk * KC + half * 4;
#pragma unroll
    for (int r = 0; r < RA; r++) {
      const int row = lrow + r * 128;
      const int64_t m = m0 + row;
      pa[r] = make_uint4(0, 0, 0, 0);
      const bool rin = (TM >= 128 || row < TM) && m < g.M;
      if (rin && kw < g.lda_w) pa[r] = __ldg(reinterpret_cast<const uint4*>(g.a_bits + m * g.lda_w + kw));
#pragma unroll
      for (int q = 0; q < (NSEG + 1) / 2; q++) {
        const int sq = half + 2 * q;
        const int64_t seg = chunk * NSEG + sq;
        const int64_t grp = seg / g.ra;
        const bool live = !(g.tail_pad && seg == g.T - 1);  // a short tail segment is added in the epilogue
        psa[r][q] = (rin && live && sq < NSEG && grp < g.Ga) ? -2.0f * load_scale(g.a_scales, g.a_bf16, m * g.lda_s + grp) : 0.0f;
      }
    }
#pragma unroll
    for (int r = 0; r < RW; r++) {
      const int row = lrow + r * 128;
      const int64_t n = n0 + row;
      pw[r] = make_uint4(0, 0, 0, 0);
      const bool rin = (TN >= 128 || row < TN) && n < g.N;
      if (rin && kw < g.ldw_w) pw[r] = __ldg(reinterpret_cast<const uint4*>(g.w_bits + n * g.ldw_w + kw));
#pragma unroll
      for (int q = 0; q < (NSEG + 1) / 2; q++) {
        const int sq = half + 2 * q;
        const int64_t grp = (chunk * NSEG + sq) / g.rw;
        psw[r][q] = (rin && sq < NSEG && grp < g.Gw) ? load_scale(g.w_scales, g.w_bf16, n * g.ldw_s + grp) : 0.0f;
      }
    }
  };
  auto stage = [&](int buf) {
#pragma unroll
    for (int r = 0; r < RA; r++) {
      const int row = lrow + r * 128;
      if (TM >= 128 || row < TM) {
        As[buf][half * 4 + 0][row] = pa[r].x; As[buf][half * 4 + 1][row] = pa[r].y;
        As[buf][half * 4 + 2][row] = pa[r].z; As[buf][half * 4 + 3][row] = pa[r].w;
#pragma unroll
        for (int q = 0; q < (NSEG + 1) / 2; q++)
          if (half + 2 * q < NSEG) AsS[buf][half + 2 * q][row] = psa[r][q];
      }
    }
#pragma unroll
    for (int r = 0; r < RW; r++) {
      const int row = lrow + r * 128;
      if (TN >= 128 || row < TN) {
        Ws[buf][half * 4 + 0][row] = pw[r].x; Ws[buf][half * 4 + 1][row] = pw[r].y;
        Ws[buf][half * 4 + 2][row] = pw[r].z; Ws[buf][half * 4 + 3][row] = pw[r].w;
#pragma unroll
        for (int q = 0; q < (NSEG + 1) / 2; q++)
          if (half + 2 * q < NSEG) WsS[buf][half + 2 * q][row] = psw[r][q];
      }
    }
  };

  prefetch(0);
  stage(0);
  __syncthreads();

  const float kBias = 8388608.0f + 16.0f * SW;  // 2^23 + (segment bits)/2
  for (int64_t chunk = 0; chunk < n_chunks; chunk++) {
    const int buf = static_cast<int>(chunk & 1);
    if (chunk + 1 < n_chunks) prefetch(chunk + 1);
#pragma unroll
    for (int s = 0; s < NSEG; s++) {
      uint32_t pc[4 * IM][4 * JN];
#pragma unroll
      for (int q = 0; q < SW; q++) {
        const int kw = s * SW + q;
        uint32_t a[4 * IM], w[4 * JN];
#pragma unroll
        for (int i = 0; i < IM; i++) {
          const uint4 v = *reinterpret_cast<const uint4*>(&As[buf][kw][i * 64 + ty * 4]);
          a[4 * i] = v.x; a[4 * i + 1] = v.y; a[4 * i + 2] = v.z; a[4 * i + 3] = v.w;
        }
#pragma unroll
        for (int j = 0; j < JN; j++) {
          const uint4 v = *reinterpret_cast<const uint4*>(&Ws[buf][kw][j * 64 + tx * 4]);
          w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
        }
#pragma unroll
        for (int i = 0; i < 4 * IM; i++)
#pragma unroll
          for (int j = 0; j < 4 * JN; j++) {
            const uint32_t p = __popc(a[i] ^ w[j]);
            pc[i][j] = (q == 0) ? p : pc[i][j] + p;
          }
      }
      float sa[4 * IM], sw[4 * JN];
#pragma unroll
      for (int i = 0; i < IM; i++) {
        const float4 v = *reinterpret_cast<const float4*>(&AsS[buf][s][i * 64 + ty * 4]);
        sa[4 * i] = v.x; sa[4 * i + 1] = v.y; sa[4 * i + 2] = v.z; sa[4 * i + 3] = v.w;
      }
#pragma unroll
      for (int j = 0; j < JN; j++) {
        const float4 v = *reinterpret_cast<const float4*>(&WsS[buf][s][j * 64 + tx * 4]);
        sw[4 * j] = v.x; sw[4 * j + 1] = v.y; sw[4 * j + 2] = v.z; sw[4 * j + 3] = v.w;
      }
#pragma unroll
      for (int i = 0; i < 4 * IM; i++)
#pragma unroll
        for (int j = 0; j < 4 * JN; j++) {
          const float f = __uint_as_float(0x4B000000u | pc[i][j]) - kBias;  // sum(p) - n/2, exact
          acc[i][j] = fmaf(f * sa[i], sw[j], acc[i][j]);                   // sa holds -2 * deltaA
        }
    }
    if (chunk + 1 < n_chunks) {
      stage(buf ^ 1);
      __syncthreads();
    }
  }

  // A tail segment shorter than the segment length was left out of the loop (its A scale was
  // staged as 0); its signed dot n_valid - 2*popc is formed here in integers, so that the term
  // added is the correctly rounded product like every other one.
  if (g.tail_pad) {
    const int64_t ga = (g.T - 1) / g.ra, gw = (g.T - 1) / g.rw;
    const int64_t w0 = (g.T - 1) * SW;
    const int n_valid = 32 * SW - g.tail_pad;
    int pc[4 * IM][4 * JN];
#pragma unroll
    for (int i = 0; i < 4 * IM; i++)
#pragma unroll
      for (int j = 0; j < 4 * JN; j++) pc[i][j] = 0;
    for (int q = 0; q < SW && w0 + q < g.n_words; q++) {
      uint32_t a[4 * IM], w[4 * JN];
#pragma unroll
      for (int i = 0; i < 4 * IM; i++) {
        const int64_t m = m0 + (i / 4) * 64 + ty * 4 + (i % 4);
        a[i] = (m < g.M) ? __ldg(g.a_bits + m * g.lda_w + w0 + q) : 0u;
      }
#pragma unroll
      for (int j = 0; j < 4 * JN; j++) {
        const int64_t n = n0 + (j / 4) * 64 + tx * 4 + (j % 4);
        w[j] = (n < g.N) ? __ldg(g.w_bits + n * g.ldw_w + w0 + q) : 0u;
      }
#pragma unroll
      for (int i = 0; i < 4 * IM; i++)
#pragma unroll
        for (int j = 0; j < 4 * JN; j++) pc[i][j] += __popc(a[i] ^ w[j]);
    }
#pragma unroll
    for (int i = 0; i < 4 * IM; i++) {
      const int64_t m = m0 + (i / 4) * 64 + ty * 4 + (i % 4);
      const float sa = (m < g.M) ? load_scale(g.a_scales, g.a_bf16, m * g.lda_s + ga) : 0.0f;
#pragma unroll
      for (int j = 0; j < 4 * JN; j++) {
        const int64_t n = n0 + (j / 4) * 64 + tx * 4 + (j % 4);
        const float sw = (n < g.N) ? load_scale(g.w_scales, g.w_bf16, n * g.ldw_s + gw) : 0.0f;
        acc[i][j] = fmaf(static_cast<float>(n_valid - 2 * pc[i][j]) * sa, sw, acc[i][j]);
      }
    }
  }

#pragma unroll
  for (int i = 0; i < 4 * IM; i++) {
    const int64_t m = m0 + (i / 4) * 64 + ty * 4 + (i % 4);
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < JN; j++) {
      const int64_t n = n0 + j * 64 + tx * 4;
      float* dst = g.C + m * g.ldc + n;
      if (n + 3 < g.N) {
        *reinterpret_cast<float4*>(dst) = make_float4(acc[i][4 * j], acc[i][4 * j + 1], acc[i][4 * j + 2], acc[i][4 * j + 3]);
      } else {
#pragma unroll
        for (int e = 0; e < 4; e++)
          if (n + e < g.N) dst[e] = acc[i][4 * j + e];
      }
    }
  }
}

// Any segment length (in whole words): integer popcounts are carried across K-words and flushed
// with the scales at each segment end.  One thread per 4x4 outputs, operands read through L1.
__global__ void __launch_bounds__(kThreads)
gemm_popc_generic_kernel(const GemmArgs g) {
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * 64 + ty * 4, n0 = static_cast<int64_t>(blockIdx.x) * 64 + tx * 4;
  float acc[4][4];
  int pc[4][4];
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int j = 0; j < 4; j++) { acc[i][j] = 0.0f; pc[i][j] = 0; }
  int64_t seg = 0;
  int in_seg = 0;
  for (int64_t kw = 0; kw < g.n_words; kw++) {
    uint32_t a[4], w[4];
#pragma unroll
    for (int i = 0; i < 4; i++) a[i] = (m0 + i < g.M) ? __ldg(g.a_bits + (m0 + i) * g.lda_w + kw) : 0u;
#pragma unroll
    for (int j = 0; j < 4; j++) w[j] = (n0 + j < g.N) ? __ldg(g.w_bits + (n0 + j) * g.ldw_w + kw) : 0u;
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
      for (int j = 0; j < 4; j++) pc[i][j] += __popc(a[i] ^ w[j]);
    in_seg++;
    if (in_seg == g.seg_words || kw == g.n_words - 1) {
      const int64_t k0 = seg * g.seg_words * 32;
      int64_t nv = g.K - k0;
      if (nv > static_cast<int64_t>(g.seg_words) * 32) nv = static_cast<int64_t>(g.seg_words) * 32;
      const int64_t ga = seg / g.ra, gw = seg / g.rw;
      float sa[4], sw[4];
#pragma unroll
      for (int i = 0; i < 4; i++) sa[i] = (m0 + i < g.M) ? load_scale(g.a_scales, g.a_bf16, (m0 + i) * g.lda_s + ga) : 0.0f;
#pragma unroll
      for (int j = 0; j < 4; j++) sw[j] = (n0 + j < g.N) ? load_scale(g.w_scales, g.w_bf16, (n0 + j) * g.ldw_s + gw) : 0.0f;
#pragma unroll
      for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) {
          const float d = static_cast<float>(static_cast<int>(nv) - 2 * pc[i][j]);
          acc[i][j] = fmaf(d * sa[i], sw[j], acc[i][j]);
          pc[i][j] = 0;
        }
      seg++;
      in_seg = 0;
    }
  }
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int j = 0; j < 4; j++)
      if (m0 + i < g.M && n0 + j < g.N) g.C[(m0 + i) * g.ldc + n0 + j] = acc[i][j];
}

// Integer partial sums only: D[m,n,t] = n_valid(t) - 2 * popc over the words of segment t.
__global__ void __launch_bounds__(kThreads)
partials_popc_kernel(const GemmArgs g, int32_t* __restrict__ D) {
  const int64_t total = g.M * g.N * g.T;
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; idx < total;
       idx += static_cast<int64_t>(gridDim.x) * kThreads) {
    const int64_t t = idx % g.T, mn = idx / g.T;
    const int64_t n = mn % g.N, m = mn / g.N;
    const int64_t w0 = t * g.seg_words;
    int64_t w1 = w0 + g.seg_words;
    if (w1 > g.n_words) w1 = g.n_words;
    int p = 0;
    for (int64_t w = w0; w < w1; w++) p += __popc(g.a_bits[m * g.lda_w + w] ^ g.w_bits[n * g.ldw_w + w]);
    int64_t nv = g.K - w0 * 32;
    if (nv > static_cast<int64_t>(g.seg_words) * 32) nv = static_cast<int64_t>(g.seg_words) * 32;
    D[idx] = static_cast<int32_t>(nv) - 2 * p;
  }
}

GemmArgs make_args(const PackedView& A, const PackedView& W, float* C, int64_t ldc) {
  GemmArgs g;
  g.a_bits = A.bits; g.a_scales = A.scales; g.w_bits = W.bits; g.w_scales = W.scales; g.C = C;
  g.M = A.rows; g.N = W.rows; g.K = A.K;
  g.lda_w = A.ld_words; g.ldw_w = W.ld_words; g.lda_s = A.ld_scales; g.ldw_s = W.ld_scales; g.ldc = ldc;
  g.a_bf16 = A.scale_bf16; g.w_bf16 = W.scale_bf16;
  g.n_words = (A.K + 31) / 32;
  const bool a_one = A.beta >= A.K, w_one = W.beta >= W.K;  // one group per row
  int64_t seg;
  if (a_one && w_one) seg = g.n_words * 32;
  else if (a_one) seg = W.beta;
  else if (w_one) seg = A.beta;
  else seg = A.beta < W.beta ? A.beta : W.beta;
  g.seg_words = static_cast<int32_t>(seg / 32);
  g.T = (A.K + seg - 1) / seg;
  g.ra = static_cast<int32_t>(a_one ? g.T : A.beta / seg);
  g.rw = static_cast<int32_t>(w_one ? g.T : W.beta / seg);
  g.Ga = num_groups(A.K, A.beta);
  g.Gw = num_groups(W.K, W.beta);
  const int64_t last_valid = A.K - (g.T - 1) * seg;
  g.tail_pad = static_cast<int32_t>(seg - last_valid);
  return g;
}

template <int SW>
cudaError_t launch_fast(const GemmArgs& g, cudaStream_t stream) {
  // Narrow N (<= 64): a 256 x 64 tile keeps every column of the tile useful.
  if (g.N <= 64) {
    dim3 grid(static_cast<unsigned>((g.N + 63) / 64), static_cast<unsigned>((g.M + 255) / 256));
    gemm_popc_kernel<SW, 4, 1><<<grid, kThreads, 0, stream>>>(g);
  } else {
    dim3 grid(static_cast<unsigned>((g.N + 127) / 128), static_cast<unsigned>((g.M + 127) / 128));
    gemm_popc_kernel<SW, 2, 2><<<grid, kThreads, 0, stream>>>(g);
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_gemm_popc(const PackedView& A, const PackedView& W, float* C, int64_t ldc,
                             cudaStream_t stream) {
  const GemmArgs g = make_args(A, W, C, ldc);
  switch (g.seg_words) {
    case 1: return launch_fast<1>(g, stream);
    case 2: return launch_fast<2>(g, stream);
    case 4: return launch_fast<4>(g, stream);
    case 8: return launch_fast<8>(g, stream);
    default: break;
  }
  dim3 grid(static_cast<unsigned>((g.N + 63) / 64), static_cast<unsigned>((g.M + 63) / 64));
  gemm_popc_generic_kernel<<<grid, kThreads, 0, stream>>>(g);
  return cudaGetLastError();
}

cudaError_t launch_partials_popc(const PackedView& A, const PackedView& W, int32_t* D, cudaStream_t stream) {
  const GemmArgs g = make_args(A, W, nullptr, 0);
  const int64_t total = g.M * g.N * g.T;
  int64_t blocks = (total + kThreads - 1) / kThreads;
  if (blocks > 148 * 32) blocks = 148 * 32;
  if (blocks < 1) blocks = 1;
  partials_popc_kernel<<<static_cast<unsigned>(blocks), kThreads, 0, stream>>>(g, D);
  return cudaGetLastError();
}

}  // namespace hbmm
