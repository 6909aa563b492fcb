// HBMM contraction for a handful of activation rows (batch 1 .. 8 of a fully connected layer): a matrix-vector
// shaped product that is bound by reading the packed weights once (Section 4.2: K / 8 bytes of sign bits plus
// 4 K / beta bytes of scales per weight row) and by launch latency, not by arithmetic.
//
// One warp per weight row.  The activation rows (bits and the per-segment scales) sit in shared memory; a lane
// walks the weight row in 16-byte pieces (four K-words, a whole number of segments), forms per segment the
// signed +-1 dot D = n_valid - 2 popc(a ^ w) in integers (Eq. 7) and adds (deltaA deltaW) D in fp32; the lanes'
// partial sums meet in a shuffle tree.  Segments of one, two or four K-words (beta 32, 64, 128 and their
// mixes); K any length (rows are padded with zero words to a multiple of four, pad bits are zero in both
// operands and the tail segment counts only its valid bits).
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {
namespace {

constexpr int kWarps = 8;
constexpr int kMaxRows = 8;

struct GemvArgs {
  const uint32_t* a_bits; const void* a_scales;
  const uint32_t* w_bits; const void* w_scales;
  float* C;
  int64_t N, K, lda_w, ldw_w, lda_s, ldw_s, ldc;
  int32_t M, a_bf16, w_bf16;
  int32_t ra, rw;        // segments per A group / per W group
  int32_t n_quads;       // 16-byte pieces per row: ceil(K / 128)
  int32_t T;             // segments per row
};

__device__ __forceinline__ float load_scale(const void* s, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(s) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(s) + idx);
}

// SW: K-words per segment; MR: activation rows held in registers.
template <int SW, int MR>
__global__ void __launch_bounds__(kWarps * 32)
gemv_popc_kernel(const GemvArgs g) {
  constexpr int SEGS = 4 / SW;                          // segments per 16-byte piece
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* a_bits = reinterpret_cast<uint4*>(smem_raw);                                    // [MR][n_quads]
  float* a_seg = reinterpret_cast<float*>(a_bits + static_cast<size_t>(MR) * g.n_quads);  // [MR][n_quads * SEGS]
  const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
  const int seg_stride = g.n_quads * SEGS;
  for (int i = t; i < MR * g.n_quads; i += kWarps * 32) {
    const int m = i / g.n_quads, q = i - m * g.n_quads;
    a_bits[i] = m < g.M ? __ldg(reinterpret_cast<const uint4*>(g.a_bits + m * g.lda_w) + q) : make_uint4(0, 0, 0, 0);
  }
  for (int i = t; i < MR * seg_stride; i += kWarps * 32) {
    const int m = i / seg_stride, s = i - m * seg_stride;
    a_seg[i] = (m < g.M && s < g.T) ? load_scale(g.a_scales, g.a_bf16, m * g.lda_s + s / g.ra) : 0.0f;
  }
  __syncthreads();

  for (int64_t n = static_cast<int64_t>(blockIdx.x) * kWarps + warp; n < g.N; n += static_cast<int64_t>(gridDim.x) * kWarps) {
    const uint4* wrow = reinterpret_cast<const uint4*>(g.w_bits + n * g.ldw_w);
    float acc[MR];
#pragma unroll
    for (int m = 0; m < MR; m++) acc[m] = 0.0f;
#pragma unroll 2
    for (int q = lane; q < g.n_quads; q += 32) {
      const uint4 wv = __ldg(wrow + q);
      const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
      float sw[SEGS];
      int nv[SEGS];
#pragma unroll
      for (int s = 0; s < SEGS; s++) {
        const int seg = q * SEGS + s;
        sw[s] = seg < g.T ? load_scale(g.w_scales, g.w_bf16, n * g.ldw_s + seg / g.rw) : 0.0f;
        const int64_t left = g.K - static_cast<int64_t>(seg) * (32 * SW);      // valid bits from the segment's start
        nv[s] = left >= 32 * SW ? 32 * SW : (left > 0 ? static_cast<int>(left) : 0);
      }
#pragma unroll
      for (int m = 0; m < MR; m++) {
        const uint4 av = a_bits[m * g.n_quads + q];
        const uint32_t aw[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
        for (int s = 0; s < SEGS; s++) {
          int p = 0;
#pragma unroll
          for (int e = 0; e < SW; e++) p += __popc(aw[s * SW + e] ^ ww[s * SW + e]);
          const float d = static_cast<float>(nv[s] - 2 * p);
          acc[m] = fmaf(a_seg[m * seg_stride + q * SEGS + s] * sw[s], d, acc[m]);
        }
      }
    }
#pragma unroll
    for (int m = 0; m < MR; m++) {
      float v = acc[m];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
      if (lane == 0 && m < g.M) g.C[m * g.ldc + n] = v;
    }
  }
}

bool make_args(const PackedView& A, const PackedView& W, GemvArgs& g) {
  if (A.rows > kMaxRows || A.rows < 1 || A.K != W.K) return false;
  const bool a_one = A.beta >= A.K, w_one = W.beta >= W.K;
  if ((!a_one && A.beta % 32 != 0) || (!w_one && W.beta % 32 != 0)) return false;
  if (a_one && w_one) return false;
  const int64_t seg = a_one ? W.beta : (w_one ? A.beta : (A.beta < W.beta ? A.beta : W.beta));
  if (seg != 32 && seg != 64 && seg != 128) return false;
  const int64_t T = (A.K + seg - 1) / seg, quads = (A.K + 127) / 128;
  if (T > (int64_t{1} << 24)) return false;
  g.a_bits = A.bits; g.a_scales = A.scales; g.w_bits = W.bits; g.w_scales = W.scales; g.C = nullptr;
  g.N = W.rows; g.K = A.K; g.lda_w = A.ld_words; g.ldw_w = W.ld_words; g.lda_s = A.ld_scales; g.ldw_s = W.ld_scales; g.ldc = 0;
  g.M = static_cast<int32_t>(A.rows); g.a_bf16 = A.scale_bf16; g.w_bf16 = W.scale_bf16;
  g.ra = static_cast<int32_t>(a_one ? T : A.beta / seg);
  g.rw = static_cast<int32_t>(w_one ? T : W.beta / seg);
  g.n_quads = static_cast<int32_t>(quads);
  g.T = static_cast<int32_t>(T);
  return true;
}

size_t smem_bytes(const GemvArgs& g, int mr, int sw) {
  return static_cast<size_t>(mr) * g.n_quads * (16 + (4 / sw) * 4);
}

template <int SW>
cudaError_t launch_sw(const GemvArgs& g, int sms, cudaStream_t stream) {
  const int mr = g.M <= 1 ? 1 : (g.M <= 2 ? 2 : (g.M <= 4 ? 4 : 8));
  const size_t smem = smem_bytes(g, mr, SW);
  int64_t blocks = (g.N + kWarps - 1) / kWarps;
  if (blocks > static_cast<int64_t>(sms) * 8) blocks = static_cast<int64_t>(sms) * 8;
  const unsigned grid = static_cast<unsigned>(blocks);
  switch (mr) {
    case 1: gemv_popc_kernel<SW, 1><<<grid, kWarps * 32, smem, stream>>>(g); break;
    case 2: gemv_popc_kernel<SW, 2><<<grid, kWarps * 32, smem, stream>>>(g); break;
    case 4: gemv_popc_kernel<SW, 4><<<grid, kWarps * 32, smem, stream>>>(g); break;
    default: gemv_popc_kernel<SW, 8><<<grid, kWarps * 32, smem, stream>>>(g); break;
  }
  return cudaGetLastError();
}

}  // namespace

// At most eight activation rows, groups of whole words with a finer grouping of 32, 64 or 128 elements, and
// the activation rows fit the default 48 KB of shared memory.
bool gemv_popc_supported(const PackedView& A, const PackedView& W) {
  GemvArgs g;
  if (!make_args(A, W, g)) return false;
  return smem_bytes(g, 8, 1) <= 48 * 1024;
}

cudaError_t launch_gemv_popc(const PackedView& A, const PackedView& W, float* C, int64_t ldc, cudaStream_t stream) {
  GemvArgs g;
  if (!make_args(A, W, g)) return cudaErrorNotSupported;
  g.C = C; g.ldc = ldc;
  int dev = 0, sms = 0;
  if (current_device(&dev, &sms) != cudaSuccess) return cudaErrorInvalidDevice;
  const int sw = static_cast<int>(((A.beta >= A.K) ? W.beta : ((W.beta >= W.K) ? A.beta : (A.beta < W.beta ? A.beta : W.beta))) / 32);
  switch (sw) {
    case 1: return launch_sw<1>(g, sms, stream);
    case 2: return launch_sw<2>(g, sms, stream);
    default: return launch_sw<4>(g, sms, stream);
  }
}

}  // namespace hbmm
