// HBWN contraction: full-precision activations times Hadamard-binary weights (beta_a = 1).
//   C[m,n] = sum_g deltaW[n,g] * sum_{k in g} s(W[n,k]) * A[m,k],   fp32 accumulation.
//
// Sign-select form: the sign bit of W[n,k] is XOR-ed into the fp32 activation and the result is
// added to a per-group partial sum; at the end of each weight group the partial sum is scaled by
// deltaW and folded into the accumulator (one FMA per output and group).
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float load_scale(const void* s, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(s) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(s) + idx);
}
__device__ __forceinline__ float load_dense(const void* p, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(p) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(p) + idx);
}

struct HbwnArgs {
  const void* a; int64_t lda; int32_t a_bf16;
  const uint32_t* w_bits; const void* w_scales; int64_t ldw_w, ldw_s; int32_t w_bf16;
  float* C; int64_t ldc;
  int64_t M, N, K, n_words, Gw;
  int64_t group_words;  // words per weight group (whole padded row when one group per row)
};

// 64 x 64 tile, 4 x 4 outputs per thread, one K-word (32 elements) per stage.
// SUB: weight scale groups per K-word (1: groups of whole words; 2 .. 16: beta_w = 16 .. 2, the group
// sizes of the paper's experiments -- the partial sum is then folded into the output inside the word).
template <int SUB>
__global__ void __launch_bounds__(kThreads)
hbwn_select_kernel(const HbwnArgs g) {
  __shared__ __align__(16) float As[2][32][64 + 4];  // k-major
  __shared__ uint32_t Ws[2][64];
  __shared__ float WsS[2][64][SUB];
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * 64, n0 = static_cast<int64_t>(blockIdx.x) * 64;
  float acc[4][4], part[4][4];
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int j = 0; j < 4; j++) { acc[i][j] = 0.0f; part[i][j] = 0.0f; }

  // staging: thread -> (row = t / 4, 8 consecutive k = (t % 4) * 8 ..)
  const int srow = t >> 2, sk = (t & 3) * 8;
  float pa[8];
  uint32_t pw = 0;
  float ps[SUB];
  auto prefetch = [&](int64_t kw) {
    const int64_t m = m0 + srow;
#pragma unroll
    for (int e = 0; e < 8; e++) {
      const int64_t k = kw * 32 + sk + e;
      pa[e] = (m < g.M && k < g.K) ? load_dense(g.a, g.a_bf16, m * g.lda + k) : 0.0f;
    }
    if (t < 64) {
      const int64_t n = n0 + t;
      pw = (n < g.N) ? __ldg(g.w_bits + n * g.ldw_w + kw) : 0u;
#pragma unroll
      for (int u = 0; u < SUB; u++) {
        const int64_t grp = SUB > 1 ? kw * SUB + u : kw / g.group_words;
        ps[u] = (n < g.N && grp < g.Gw) ? load_scale(g.w_scales, g.w_bf16, n * g.ldw_s + grp) : 0.0f;
      }
    }
  };
  auto stage = [&](int buf) {
#pragma unroll
    for (int e = 0; e < 8; e++) As[buf][sk + e][srow] = pa[e];
    if (t < 64) {
      Ws[buf][t] = pw;
#pragma unroll
      for (int u = 0; u < SUB; u++) WsS[buf][t][u] = ps[u];
    }
  };
  prefetch(0);
  stage(0);
  __syncthreads();
  for (int64_t kw = 0; kw < g.n_words; kw++) {
    const int buf = static_cast<int>(kw & 1);
    if (kw + 1 < g.n_words) prefetch(kw + 1);
    uint32_t nw[4];
#pragma unroll
    for (int j = 0; j < 4; j++) nw[j] = ~Ws[buf][tx * 4 + j];  // bit set <=> weight sign is -1
#pragma unroll
    for (int k = 0; k < 32; k++) {
      const float4 av = *reinterpret_cast<const float4*>(&As[buf][k][ty * 4]);
      const float a[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const uint32_t flip = (nw[j] << (31 - k)) & 0x80000000u;
#pragma unroll
        for (int i = 0; i < 4; i++) part[i][j] += __uint_as_float(__float_as_uint(a[i]) ^ flip);
      }
      if (SUB > 1 && (k + 1) % (32 / SUB) == 0) {      // a sub-word group ends here
#pragma unroll
        for (int j = 0; j < 4; j++) {
          const float s = WsS[buf][tx * 4 + j][k / (32 / SUB)];
#pragma unroll
          for (int i = 0; i < 4; i++) { acc[i][j] = fmaf(s, part[i][j], acc[i][j]); part[i][j] = 0.0f; }
        }
      }
    }
    const bool group_end = SUB == 1 && (((kw + 1) % g.group_words == 0) || (kw + 1 == g.n_words));
    if (group_end) {
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const float s = WsS[buf][tx * 4 + j][0];
#pragma unroll
        for (int i = 0; i < 4; i++) { acc[i][j] = fmaf(s, part[i][j], acc[i][j]); part[i][j] = 0.0f; }
      }
    }
    if (kw + 1 < g.n_words) {
      stage(buf ^ 1);
      __syncthreads();
    }
  }
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const int64_t m = m0 + ty * 4 + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const int64_t n = n0 + tx * 4 + j;
      if (n < g.N) g.C[m * g.ldc + n] = acc[i][j];
    }
  }
}

}  // namespace

cudaError_t launch_hbwn_select(const DenseView& A, const PackedView& W, float* C, int64_t ldc, cudaStream_t stream) {
  HbwnArgs g;
  g.a = A.data; g.lda = A.ld; g.a_bf16 = A.bf16;
  g.w_bits = W.bits; g.w_scales = W.scales; g.ldw_w = W.ld_words; g.ldw_s = W.ld_scales; g.w_bf16 = W.scale_bf16;
  g.C = C; g.ldc = ldc; g.M = A.rows; g.N = W.rows; g.K = A.K;
  g.n_words = (A.K + 31) / 32;
  g.Gw = num_groups(W.K, W.beta);
  const bool subword = W.beta < 32 && W.beta < W.K;
  g.group_words = W.beta >= W.K ? g.n_words : (subword ? 1 : W.beta / 32);
  dim3 grid(static_cast<unsigned>((g.N + 63) / 64), static_cast<unsigned>((g.M + 63) / 64));
  switch (subword ? 32 / W.beta : 1) {
    case 2: hbwn_select_kernel<2><<<grid, kThreads, 0, stream>>>(g); break;
    case 4: hbwn_select_kernel<4><<<grid, kThreads, 0, stream>>>(g); break;
    case 8: hbwn_select_kernel<8><<<grid, kThreads, 0, stream>>>(g); break;
    case 16: hbwn_select_kernel<16><<<grid, kThreads, 0, stream>>>(g); break;
    default: hbwn_select_kernel<1><<<grid, kThreads, 0, stream>>>(g); break;
  }
  return cudaGetLastError();
}

}  // namespace hbmm
