// Packed convolution front end (beta = 32, fp32 NCHW input) with the input tile staged by tensor
// copies.  A block handles RB output rows of one image and a range of 32-channel chunks.  For every
// chunk one 4-D tensor copy brings [32 channels][rows_in input rows][pitch columns] into shared
// memory, zero halo included (the copy starts left of and above the image where the padding asks
// for it, and whatever lies outside the tensor arrives as zeros); the copy of the next chunk is in
// flight while the current one is binarized.  One thread then produces one (output pixel, K-word):
// the 32 lanes of a warp hold 32 consecutive pixels of the same word, so tile reads are consecutive.
// Words and scales are collected in shared memory and leave the block as contiguous runs per row.
#include <cuda_bf16.h>
#include "kernels.h"
#include "tensor_map.h"
#include "umma_common.cuh"
#include "im2col_gather.cuh"

namespace hbmm {
namespace {

using namespace umma;

constexpr int kCC = 32;   // channels per chunk: 32 * kh * kw elements = whole K-words

struct Plan {
  int RB;                 // output rows per block
  int rows_in;            // staged input rows: (RB - 1) * sh + kh
  int pitch;              // staged columns (multiple of 4)
  int x0;                 // tile column of input x = -pw (the first tap of output column 0)
  int yo_blocks;          // ceil(Ho / RB)
  int splits;             // channel ranges (grid.y)
  int chunks_per_split;
  int n_chunks;           // ceil(C / 32)
};

__device__ __forceinline__ void store_scale(void* scales, int bf16, int64_t idx, float v) {
  if (bf16) reinterpret_cast<__nv_bfloat16*>(scales)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(scales)[idx] = v;
}

__global__ void __launch_bounds__(256)
im2col_quantize_tma_kernel(const __grid_constant__ CUtensorMap x_map, const ConvGeom g, const Plan tp,
                           uint32_t* __restrict__ bits, int64_t ld_words, void* __restrict__ scales, int64_t ld_scales,
                           int scale_bf16) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int taps = g.kh * g.kw;
  const int tile_elems = kCC * tp.rows_in * tp.pitch;           // floats per buffer; bytes are a multiple of 128
  const int max_pixels = tp.RB * g.Wo;
  const int split_words = tp.chunks_per_split * taps;          // words this block produces per pixel (upper bound)
  const int ldo = split_words + 1;                             // odd-ish pitch: fewer bank conflicts on the column writes
  float* tile0 = reinterpret_cast<float*>(smem_raw);                                   // two tile buffers
  uint64_t* bar = reinterpret_cast<uint64_t*>(tile0 + 2 * tile_elems);                // two "tile landed" barriers
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar + 2);
  uint32_t* out_bits = reinterpret_cast<uint32_t*>(bar + 4);                          // [max_pixels][ldo]
  float* out_scale = reinterpret_cast<float*>(out_bits + max_pixels * ldo);           // same shape
  unsigned short* off = reinterpret_cast<unsigned short*>(out_scale + max_pixels * ldo);

  const int64_t b = blockIdx.x / tp.yo_blocks;
  const int yo0 = static_cast<int>(blockIdx.x % tp.yo_blocks) * tp.RB;
  const int rows = (g.Ho - yo0 < tp.RB) ? g.Ho - yo0 : tp.RB;
  const int pixels = rows * g.Wo;
  const int pix_pad = (pixels + 31) / 32 * 32;                 // keep a warp on one word
  const int chunk_first = blockIdx.y * tp.chunks_per_split;
  const int n_my = (tp.n_chunks - chunk_first < tp.chunks_per_split) ? tp.n_chunks - chunk_first : tp.chunks_per_split;
  const int cs = tp.rows_in * tp.pitch;

  if (threadIdx.x == 0) {
    mbar_init(&bar[0], 1);
    mbar_init(&bar[1], 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // chunk-local k -> offset of tap (c, i, j) inside the tile, for filter sizes without an unrolled gather
  for (int k = threadIdx.x; k < kCC * taps; k += blockDim.x) {
    const int c = k / taps, r = k - c * taps, i = r / g.kw, j = r - i * g.kw;
    off[k] = static_cast<unsigned short>(c * cs + i * tp.pitch + j);
  }
  __syncthreads();

  const uint32_t tile_bytes = static_cast<uint32_t>(tile_elems) * 4;
  auto issue = [&](int it) {
    // x starts at -(x0 + pw), a multiple of 4 elements = 16 bytes; y may be negative too
    fence_async_proxy();            // earlier reads of this buffer are ordered before the copy's writes
    mbar_arrive_expect_tx(&bar[it & 1], tile_bytes);
    tma_load_4d(tile0 + (it & 1) * tile_elems, &x_map, -(tp.x0 + g.pw), yo0 * g.sh - g.ph, (chunk_first + it) * kCC, static_cast<int32_t>(b),
                &bar[it & 1]);
  };
  if (threadIdx.x == 0 && n_my > 0) issue(0);

  int words_done = 0;                                          // words produced so far by this block
  bool wrote_last = false;
  for (int it = 0; it < n_my; it++) {
    const int c0 = (chunk_first + it) * kCC;
    const int cc = (g.C - c0 < kCC) ? g.C - c0 : kCC;
    wrote_last = c0 + cc == g.C;
    // the other buffer was last read in iteration it - 1, which ended with a block-wide barrier
    if (threadIdx.x == 0 && it + 1 < n_my) issue(it + 1);
    mbar_wait(&bar[it & 1], static_cast<uint32_t>((it >> 1) & 1), abort_flag, 1);   // bounded; on expiry the output is undefined
    const float* t = tile0 + (it & 1) * tile_elems;
    const int chunk_elems = cc * taps;
    const int words = (chunk_elems + 31) / 32;
    for (int idx = threadIdx.x; idx < pix_pad * words; idx += 256) {
      const int w = idx / pix_pad, pix = idx - w * pix_pad;
      if (pix >= pixels) continue;
      const int ry = pix / g.Wo, xo = pix - ry * g.Wo;
      const int k_begin = w * 32;
      const int nk = (chunk_elems - k_begin < 32) ? chunk_elems - k_begin : 32;
      const float* base = t + ry * g.sh * tp.pitch + xo + tp.x0;
      uint32_t word = 0;
      float sum = 0.f;
      if (cc == kCC && g.kh == 3 && g.kw == 3) {
        gather_word_dispatch<3, 3>(w, base, cs, tp.pitch, word, sum);
      } else if (cc == kCC && taps == 1) {
        gather_word_dispatch<1, 1>(w, base, cs, tp.pitch, word, sum);
      } else {
        const unsigned short* o = off + k_begin;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
        int e = 0;
        for (; e + 4 <= nk; e += 4) {
          const float v0 = base[o[e]], v1 = base[o[e + 1]], v2 = base[o[e + 2]], v3 = base[o[e + 3]];
          word |= (v0 >= 0.0f ? 1u : 0u) << e;
          word |= (v1 >= 0.0f ? 1u : 0u) << (e + 1);
          word |= (v2 >= 0.0f ? 1u : 0u) << (e + 2);
          word |= (v3 >= 0.0f ? 1u : 0u) << (e + 3);
          s0 += fabsf(v0); s1 += fabsf(v1); s2 += fabsf(v2); s3 += fabsf(v3);
        }
        for (; e < nk; e++) {
          const float v = base[o[e]];
          word |= (v >= 0.0f ? 1u : 0u) << e;
          s0 += fabsf(v);
        }
        sum = (s0 + s1) + (s2 + s3);
      }
      out_bits[pix * ldo + words_done + w] = word;
      out_scale[pix * ldo + words_done + w] = sum / static_cast<float>(nk);
    }
    words_done += words;
    __syncthreads();
  }

  // contiguous runs: for each pixel the block's words, then (last range only) the zero padding
  const int64_t word0 = static_cast<int64_t>(chunk_first) * kCC * taps / 32;
  const int run_bits = wrote_last ? static_cast<int>(ld_words - word0) : words_done;
  const int run_scale = wrote_last ? static_cast<int>(ld_scales - word0) : words_done;
  const int64_t m_base = (b * g.Ho + yo0) * g.Wo;
  if ((word0 & 3) == 0 && (run_bits & 3) == 0) {
    const int q_per = run_bits >> 2;                         // 16-byte pieces per pixel
    for (int idx = threadIdx.x; idx < pixels * q_per; idx += 256) {
      const int pix = idx / q_per, w = (idx - pix * q_per) * 4;
      const uint32_t* src = out_bits + pix * ldo + w;
      uint4 o;
      o.x = (w < words_done) ? src[0] : 0u; o.y = (w + 1 < words_done) ? src[1] : 0u;
      o.z = (w + 2 < words_done) ? src[2] : 0u; o.w = (w + 3 < words_done) ? src[3] : 0u;
      *reinterpret_cast<uint4*>(bits + (m_base + pix) * ld_words + word0 + w) = o;
    }
  } else {
    for (int idx = threadIdx.x; idx < pixels * run_bits; idx += 256) {
      const int pix = idx / run_bits, w = idx - pix * run_bits;
      bits[(m_base + pix) * ld_words + word0 + w] = (w < words_done) ? out_bits[pix * ldo + w] : 0u;
    }
  }
  if (!scale_bf16 && (word0 & 3) == 0 && (run_scale & 3) == 0) {
    const int q_per = run_scale >> 2;
    float* sc = reinterpret_cast<float*>(scales);
    for (int idx = threadIdx.x; idx < pixels * q_per; idx += 256) {
      const int pix = idx / q_per, w = (idx - pix * q_per) * 4;
      const float* src = out_scale + pix * ldo + w;
      float4 o;
      o.x = (w < words_done) ? src[0] : 0.f; o.y = (w + 1 < words_done) ? src[1] : 0.f;
      o.z = (w + 2 < words_done) ? src[2] : 0.f; o.w = (w + 3 < words_done) ? src[3] : 0.f;
      *reinterpret_cast<float4*>(sc + (m_base + pix) * ld_scales + word0 + w) = o;
    }
  } else {
    for (int idx = threadIdx.x; idx < pixels * run_scale; idx += 256) {
      const int pix = idx / run_scale, w = idx - pix * run_scale;
      store_scale(scales, scale_bf16, (m_base + pix) * ld_scales + word0 + w, (w < words_done) ? out_scale[pix * ldo + w] : 0.0f);
    }
  }
}

inline int round_up4(int v) { return (v + 3) / 4 * 4; }

bool make_plan(const ConvGeom& g, int sms, Plan* out, size_t* smem_bytes) {
  Plan p;
  p.RB = 112 / g.Wo;
  if (p.RB < 1) p.RB = 1;
  if (p.RB > g.Ho) p.RB = g.Ho;
  p.rows_in = (p.RB - 1) * g.sh + g.kh;
  const int span = g.Wo - 1 + g.kw;                            // input columns the block's taps touch (stride 1 along x)
  p.x0 = round_up4(g.pw) - g.pw;
  p.pitch = round_up4(p.x0 + span);
  p.yo_blocks = (g.Ho + p.RB - 1) / p.RB;
  p.n_chunks = (g.C + kCC - 1) / kCC;
  const int64_t row_blocks = static_cast<int64_t>(g.B) * p.yo_blocks;
  int splits = 1;
  while (row_blocks * splits < 2LL * sms && splits * 2 <= p.n_chunks) splits *= 2;
  p.chunks_per_split = (p.n_chunks + splits - 1) / splits;
  p.splits = (p.n_chunks + p.chunks_per_split - 1) / p.chunks_per_split;
  const int taps = g.kh * g.kw;
  const int64_t tile_elems = static_cast<int64_t>(kCC) * p.rows_in * p.pitch;
  *smem_bytes = static_cast<size_t>(2 * tile_elems * 4 + 32 +
                                    2LL * p.RB * g.Wo * (p.chunks_per_split * taps + 1) * 4 + static_cast<int64_t>(kCC) * taps * 2 + 16);
  *out = p;
  return p.pitch <= 256 && p.rows_in <= 256 && tile_elems < 65536 && *smem_bytes <= 200 * 1024;
}

}  // namespace

// fp32 input whose rows start on 16-byte boundaries (a tensor map wants 16-byte strides), stride 1
// along x, groups of exactly one K-word.
bool im2col_quantize_tma_supported(const void* x, int x_bf16, const ConvGeom& g, int32_t beta) {
  const int64_t K = static_cast<int64_t>(g.C) * g.kh * g.kw;
  if (x_bf16 || beta != 32 || beta >= K || g.sw != 1 || g.W % 4 != 0 || reinterpret_cast<uintptr_t>(x) % 16 != 0) return false;
  if (encode_tiled_fn() == nullptr) return false;
  Plan p;
  size_t smem;
  return make_plan(g, 148, &p, &smem);
}

cudaError_t launch_im2col_quantize_tma(const void* x, const ConvGeom& g, uint32_t* bits, int64_t ld_words, void* scales,
                                       int64_t ld_scales, int scale_bf16, cudaStream_t stream) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  Plan p;
  size_t smem;
  if (!make_plan(g, sms, &p, &smem)) return cudaErrorNotSupported;
  CUtensorMap map;
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(g.W), static_cast<cuuint64_t>(g.H), static_cast<cuuint64_t>(g.C),
                              static_cast<cuuint64_t>(g.B)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(g.W) * 4, static_cast<cuuint64_t>(g.H) * g.W * 4,
                                 static_cast<cuuint64_t>(g.C) * g.H * g.W * 4};
  const cuuint32_t box[4] = {static_cast<cuuint32_t>(p.pitch), static_cast<cuuint32_t>(p.rows_in), kCC, 1};
  const cuuint32_t elem[4] = {1, 1, 1, 1};
  if (encode_tiled_fn()(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void*>(x), dims, strides, box, elem,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorNotSupported;
  static size_t configured = 0;
  if (smem > 48 * 1024 && smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(im2col_quantize_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    configured = 200 * 1024;
  }
  dim3 grid(static_cast<unsigned>(static_cast<int64_t>(g.B) * p.yo_blocks), static_cast<unsigned>(p.splits));
  im2col_quantize_tma_kernel<<<grid, 256, smem, stream>>>(map, g, p, bits, ld_words, scales, ld_scales, scale_bf16);
  return cudaGetLastError();
}

cudaError_t read_im2col_tma_error(int* code) {
  return cudaMemcpyFromSymbol(code, umma::g_error_word, sizeof(int));
}

}  // namespace hbmm
