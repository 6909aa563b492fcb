// Convolution front end: implicit im2col gather from an NCHW activation tensor.
//   A[m,k] = x[b, c, yo*sh + i - ph, xo*sw + j - pw]  (0 outside the image),
//   m = (b, yo, xo), k = (c, i, j) with c slowest -- the column order of Reshape(W, (filters, -1)).
// The packed variant binarizes each gathered row along k on the fly (Eq. 1-4 applied to the
// im2col row, the grouping Eq. 7 is stated for) and never writes the fp32 matrix; the dense
// variant writes bf16 rows for the HBWN mode.
#include <cuda_bf16.h>
#include "kernels.h"
#include "im2col_gather.cuh"

namespace hbmm {
namespace {

constexpr int kThreads = 128;

__device__ __forceinline__ float load_x(const void* p, int bf16, int64_t idx) {
  if (bf16) return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(p) + idx)) << 16);
  return __ldg(reinterpret_cast<const float*>(p) + idx);
}
__device__ __forceinline__ void store_scale(void* scales, int bf16, int64_t idx, float v) {
  if (bf16) reinterpret_cast<__nv_bfloat16*>(scales)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(scales)[idx] = v;
}

// One thread per output row m: consecutive lanes hold consecutive xo, so every tap is a
// coalesced read along the image row.  Words and scales are produced in k order.
__global__ void __launch_bounds__(kThreads)
im2col_quantize_kernel(const void* __restrict__ x, int x_bf16, const ConvGeom g, int64_t M, int64_t K,
                       int64_t beta, int64_t G, uint32_t* __restrict__ bits, int64_t ld_words,
                       void* __restrict__ scales, int64_t ld_scales, int scale_bf16) {
  const int64_t m = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
  if (m >= M) return;
  const int xo = static_cast<int>(m % g.Wo);
  const int yo = static_cast<int>((m / g.Wo) % g.Ho);
  const int64_t b = m / (static_cast<int64_t>(g.Wo) * g.Ho);
  uint32_t* brow = bits + m * ld_words;
  uint32_t word = 0;
  float wsum[4] = {0.f, 0.f, 0.f, 0.f};
  float gsum = 0.0f;
  int64_t k = 0, grp = 0, in_grp = 0;
  for (int c = 0; c < g.C; c++) {
    const int64_t plane = (b * g.C + c) * static_cast<int64_t>(g.H) * g.W;
    for (int i = 0; i < g.kh; i++) {
      const int y = yo * g.sh + i - g.ph;
      const bool yin = y >= 0 && y < g.H;
      for (int j = 0; j < g.kw; j++) {
        const int xx = xo * g.sw + j - g.pw;
        float v = 0.0f;
        if (yin && xx >= 0 && xx < g.W) v = load_x(x, x_bf16, plane + static_cast<int64_t>(y) * g.W + xx);
        word |= (v >= 0.0f ? 1u : 0u) << (k & 31);
        wsum[k & 3] += fabsf(v);
        k++;
        in_grp++;
        if ((k & 31) == 0) { brow[(k >> 5) - 1] = word; word = 0; }
        if ((k & 31) == 0 || in_grp == beta) {
          gsum += (wsum[0] + wsum[1]) + (wsum[2] + wsum[3]);
          wsum[0] = wsum[1] = wsum[2] = wsum[3] = 0.0f;
        }
        if (in_grp == beta) {
          store_scale(scales, scale_bf16, m * ld_scales + grp, gsum / static_cast<float>(beta));
          grp++; in_grp = 0; gsum = 0.0f;
        }
      }
    }
  }
  if (k & 31) brow[k >> 5] = word;
  for (int64_t w = (k + 31) >> 5; w < ld_words; w++) brow[w] = 0u;
  if (in_grp > 0) {
    gsum += (wsum[0] + wsum[1]) + (wsum[2] + wsum[3]);
    store_scale(scales, scale_bf16, m * ld_scales + grp, gsum / static_cast<float>(in_grp));
    grp++;
  }
  for (int64_t z = grp; z < ld_scales; z++) store_scale(scales, scale_bf16, m * ld_scales + z, 0.0f);
}

// One thread per (row m, scale group g): the 32 lanes of a warp hold 32 consecutive m for the
// same group, so every tap is a coalesced read along an image row and each thread emits whole
// words plus the group's scale.  Used when beta < K; blocks are 32 rows x 8 groups.
__global__ void __launch_bounds__(256)
im2col_quantize_groups_kernel(const void* __restrict__ x, int x_bf16, const ConvGeom g, int64_t M, int64_t K,
                              int beta_words, int64_t G, int64_t n_words, uint32_t* __restrict__ bits,
                              int64_t ld_words, void* __restrict__ scales, int64_t ld_scales, int scale_bf16) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t m = static_cast<int64_t>(blockIdx.x) * 32 + lane;
  const int64_t grp = static_cast<int64_t>(blockIdx.y) * 8 + warp;
  if (m >= M || grp >= G) return;
  const int xo = static_cast<int>(m % g.Wo);
  const int yo = static_cast<int>((m / g.Wo) % g.Ho);
  const int64_t b = m / (static_cast<int64_t>(g.Wo) * g.Ho);
  const int taps = g.kh * g.kw;
  const int64_t HW = static_cast<int64_t>(g.H) * g.W;
  const int y0 = yo * g.sh - g.ph, x0 = xo * g.sw - g.pw;
  const int64_t k_begin = grp * beta_words * 32;
  int64_t k_end = k_begin + static_cast<int64_t>(beta_words) * 32;
  if (k_end > K) k_end = K;
  int c = static_cast<int>(k_begin / taps);
  int r = static_cast<int>(k_begin - static_cast<int64_t>(c) * taps);
  int i = r / g.kw, j = r - i * g.kw;
  const int64_t base = b * g.C * HW;
  uint32_t* brow = bits + m * ld_words;
  float gsum = 0.0f;
  for (int64_t kw0 = k_begin; kw0 < k_end; kw0 += 32) {
    uint32_t word = 0;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    const int nk = (k_end - kw0 < 32) ? static_cast<int>(k_end - kw0) : 32;
#pragma unroll 4
    for (int e = 0; e < nk; e++) {
      const int y = y0 + i, xx = x0 + j;
      float v = 0.0f;
      if (y >= 0 && y < g.H && xx >= 0 && xx < g.W) v = load_x(x, x_bf16, base + c * HW + static_cast<int64_t>(y) * g.W + xx);
      word |= (v >= 0.0f ? 1u : 0u) << e;
      const float av = fabsf(v);
      if ((e & 3) == 0) s0 += av; else if ((e & 3) == 1) s1 += av; else if ((e & 3) == 2) s2 += av; else s3 += av;
      if (++j == g.kw) { j = 0; if (++i == g.kh) { i = 0; c++; } }
    }
    brow[kw0 >> 5] = word;
    gsum += (s0 + s1) + (s2 + s3);
  }
  store_scale(scales, scale_bf16, m * ld_scales + grp, gsum / static_cast<float>(k_end - k_begin));
  if (grp == G - 1) {
    for (int64_t w = n_words; w < ld_words; w++) brow[w] = 0u;
    for (int64_t z = G; z < ld_scales; z++) store_scale(scales, scale_bf16, m * ld_scales + z, 0.0f);
  }
}

__global__ void __launch_bounds__(256)
im2col_bf16_kernel(const void* __restrict__ x, int x_bf16, const ConvGeom g, int64_t M, int64_t K,
                   __nv_bfloat16* __restrict__ out, int64_t ld) {
  const int64_t total = M * ld;
  const int taps = g.kh * g.kw;
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; idx < total;
       idx += static_cast<int64_t>(gridDim.x) * 256) {
    const int64_t m = idx / ld;
    const int k = static_cast<int>(idx - m * ld);
    float v = 0.0f;
    if (k < K) {
      const int c = k / taps, r = k - c * taps, i = r / g.kw, j = r - i * g.kw;
      const int xo = static_cast<int>(m % g.Wo);
      const int yo = static_cast<int>((m / g.Wo) % g.Ho);
      const int64_t b = m / (static_cast<int64_t>(g.Wo) * g.Ho);
      const int y = yo * g.sh + i - g.ph, xx = xo * g.sw + j - g.pw;
      if (y >= 0 && y < g.H && xx >= 0 && xx < g.W)
        v = load_x(x, x_bf16, ((b * g.C + c) * static_cast<int64_t>(g.H) + y) * g.W + xx);
    }
    out[idx] = __float2bfloat16_rn(v);
  }
}

// ---- shared-memory tiled front ends (stride_w == 1, any kh x kw / padding / stride_h) ----------------
// A block owns RB consecutive output rows (b, yo .. yo+RB-1) and a contiguous range of input
// channels that it walks in chunks of 32.  The input rows a chunk needs are staged in shared
// memory with their zero halo (coalesced reads, each element fetched once per block), a small
// table maps the chunk-local k to its tile offset, and the results leave the block as contiguous
// runs per output row.

constexpr int kTileCC = 32;   // channels per chunk: 32 * kh * kw elements = whole K-words and whole 16-byte pieces

struct TilePlan {
  int RB;             // output rows per block
  int rows_in;        // staged input rows: (RB - 1) * sh + kh
  int span;           // staged row length: Wo - 1 + kw
  int yo_blocks;      // ceil(Ho / RB)
  int splits;         // channel ranges (grid.y)
  int chunks_per_split;
};

inline TilePlan make_plan(const ConvGeom& g, int sms) {
  TilePlan p;
  p.RB = 112 / g.Wo;
  if (p.RB < 1) p.RB = 1;
  if (p.RB > g.Ho) p.RB = g.Ho;
  p.rows_in = (p.RB - 1) * g.sh + g.kh;
  p.span = g.Wo - 1 + g.kw;
  p.yo_blocks = (g.Ho + p.RB - 1) / p.RB;
  const int chunks = (g.C + kTileCC - 1) / kTileCC;
  const int64_t row_blocks = static_cast<int64_t>(g.B) * p.yo_blocks;
  int splits = 1;
  while (row_blocks * splits < 2LL * sms && splits * 2 <= chunks) splits *= 2;
  p.chunks_per_split = (chunks + splits - 1) / splits;
  p.splits = (chunks + p.chunks_per_split - 1) / p.chunks_per_split;
  return p;
}

template <typename T, typename Conv>
__device__ __forceinline__ void stage_tile(T* tile, const void* __restrict__ x, int x_bf16, const ConvGeom& g,
                                           int64_t b, int c0, int cc, int yo0, const TilePlan& tp, Conv conv) {
  // A warp stages four tile rows (c, r) per pass, 64 columns of each at a time: the eight global
  // loads of a pass are issued before the first shared-memory store, and all index arithmetic that
  // needs a division is done once per row.
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int y_base = yo0 * g.sh - g.ph;
  const int rows_total = cc * tp.rows_in;
  for (int row0 = warp * 4; row0 < rows_total; row0 += nwarps * 4) {
    int64_t src[4];
    bool rin[4];
#pragma unroll
    for (int u = 0; u < 4; u++) {
      const int row = row0 + u;
      const int c = row / tp.rows_in, r = row - c * tp.rows_in;
      const int y = y_base + r;
      rin[u] = row < rows_total && y >= 0 && y < g.H;
      src[u] = ((b * g.C + c0 + c) * static_cast<int64_t>(g.H) + (rin[u] ? y : 0)) * g.W - g.pw;
    }
    for (int xx0 = 0; xx0 < tp.span; xx0 += 64) {
      float v[4][2];
#pragma unroll
      for (int u = 0; u < 4; u++)
#pragma unroll
        for (int h = 0; h < 2; h++) {
          const int xx = xx0 + h * 32 + lane, xi = xx - g.pw;
          v[u][h] = 0.0f;
          if (rin[u] && xx < tp.span && xi >= 0 && xi < g.W) v[u][h] = load_x(x, x_bf16, src[u] + xx);
        }
#pragma unroll
      for (int u = 0; u < 4; u++)
#pragma unroll
        for (int h = 0; h < 2; h++) {
          const int xx = xx0 + h * 32 + lane;
          if (row0 + u < rows_total && xx < tp.span) tile[(row0 + u) * tp.span + xx] = conv(v[u][h]);
        }
    }
  }
}

// chunk-local k -> offset of tap (c, i, j) inside the staged tile (for the pixel at the tile origin)
__device__ __forceinline__ void build_offsets(unsigned short* off, int cc, const ConvGeom& g, const TilePlan& tp) {
  const int taps = g.kh * g.kw;
  for (int k = threadIdx.x; k < cc * taps; k += blockDim.x) {
    const int c = k / taps, r = k - c * taps, i = r / g.kw, j = r - i * g.kw;
    off[k] = static_cast<unsigned short>((c * tp.rows_in + i) * tp.span + j);
  }
}

struct ToBf16 { __device__ unsigned short operator()(float v) const { return __bfloat16_as_ushort(__float2bfloat16_rn(v)); } };
struct KeepF32 { __device__ float operator()(float v) const { return v; } };

// bf16 rows for HBWN.  Each thread writes 16-byte pieces (8 consecutive k) of an output row.
__global__ void __launch_bounds__(256)
im2col_bf16_tiled_kernel(const void* __restrict__ x, int x_bf16, const ConvGeom g, const TilePlan tp, int64_t K,
                         __nv_bfloat16* __restrict__ out, int64_t ld) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int taps = g.kh * g.kw;
  unsigned short* off = reinterpret_cast<unsigned short*>(smem_raw);                       // [32 * taps]
  unsigned short* tile = off + ((kTileCC * taps + 7) / 8) * 8;                             // [32 * rows_in * span]
  const int64_t b = blockIdx.x / tp.yo_blocks;
  const int yo0 = static_cast<int>(blockIdx.x % tp.yo_blocks) * tp.RB;
  const int rows = (g.Ho - yo0 < tp.RB) ? g.Ho - yo0 : tp.RB;
  const int pixels = rows * g.Wo;
  const int chunk_first = blockIdx.y * tp.chunks_per_split;
  for (int ch = chunk_first; ch < chunk_first + tp.chunks_per_split; ch++) {
    const int c0 = ch * kTileCC;
    if (c0 >= g.C) break;
    const int cc = (g.C - c0 < kTileCC) ? g.C - c0 : kTileCC;
    const bool last_chunk = c0 + cc == g.C;
    __syncthreads();                              // previous chunk's readers are done with tile / off
    if (ch == chunk_first || cc != kTileCC) build_offsets(off, cc, g, tp);
    stage_tile<unsigned short>(tile, x, x_bf16, g, b, c0, cc, yo0, tp, ToBf16());
    __syncthreads();
    const int k_lo = c0 * taps;                                               // multiple of 8
    const int k_end = k_lo + cc * taps;                                       // valid elements end here
    const int k_hi = last_chunk ? static_cast<int>(ld) : k_end;               // the last chunk also writes the padding
    const int pieces = (k_hi - k_lo + 7) / 8;
    // walk (pixel, piece) pairs with piece fastest, without divisions
    int pc = threadIdx.x % pieces, pix = threadIdx.x / pieces;
    const int dpc = 256 % pieces, dpix = 256 / pieces;
    int ry = pix / g.Wo, xo = pix - ry * g.Wo;
    while (pix < pixels) {
      const int kl = pc * 8;                                                  // chunk-local k of the piece
      const unsigned short* base = tile + ry * g.sh * tp.span + xo;
      unsigned short v[8];
#pragma unroll
      for (int e = 0; e < 8; e++) v[e] = (k_lo + kl + e < k_end) ? base[off[kl + e]] : static_cast<unsigned short>(0);
      const int64_t m = (b * g.Ho + yo0 + ry) * g.Wo + xo;
      uint4 o;
      o.x = v[0] | (static_cast<uint32_t>(v[1]) << 16); o.y = v[2] | (static_cast<uint32_t>(v[3]) << 16);
      o.z = v[4] | (static_cast<uint32_t>(v[5]) << 16); o.w = v[6] | (static_cast<uint32_t>(v[7]) << 16);
      *reinterpret_cast<uint4*>(out + m * ld + k_lo + kl) = o;
      pc += dpc; pix += dpix; xo += dpix;
      if (pc >= pieces) { pc -= pieces; pix++; xo++; }
      while (xo >= g.Wo) { xo -= g.Wo; ry++; }
    }
  }
}

// Packed front end for beta = 32: one thread per (output pixel, K-word); the 32 lanes of a warp
// hold 32 consecutive pixels of the same word, so the tap offsets are warp-uniform and the tile
// reads are consecutive.  Words and scales of the block's channel range are collected in shared
// memory and written out as contiguous runs per output row.
__global__ void __launch_bounds__(256)
im2col_quantize_tiled_kernel(const void* __restrict__ x, int x_bf16, const ConvGeom g, const TilePlan tp, int64_t K,
                             int64_t G, int64_t n_words, uint32_t* __restrict__ bits, int64_t ld_words,
                             void* __restrict__ scales, int64_t ld_scales, int scale_bf16) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int taps = g.kh * g.kw;
  const int max_pixels = tp.RB * g.Wo;
  const int split_words = tp.chunks_per_split * taps;          // words this block produces per pixel (upper bound)
  float* tile = reinterpret_cast<float*>(smem_raw);                                        // [32 * rows_in * span]
  uint32_t* out_bits = reinterpret_cast<uint32_t*>(tile + kTileCC * tp.rows_in * tp.span);  // [max_pixels][split_words + 1]
  float* out_scale = reinterpret_cast<float*>(out_bits + max_pixels * (split_words + 1));  // same shape
  unsigned short* off = reinterpret_cast<unsigned short*>(out_scale + max_pixels * (split_words + 1));
  const int ldo = split_words + 1;                             // odd-ish pitch: fewer bank conflicts on the column writes
  const int64_t b = blockIdx.x / tp.yo_blocks;
  const int yo0 = static_cast<int>(blockIdx.x % tp.yo_blocks) * tp.RB;
  const int rows = (g.Ho - yo0 < tp.RB) ? g.Ho - yo0 : tp.RB;
  const int pixels = rows * g.Wo;
  const int pix_pad = (pixels + 31) / 32 * 32;                 // keep a warp on one word
  const int chunk_first = blockIdx.y * tp.chunks_per_split;
  int words_done = 0;                                          // words produced so far by this block
  bool wrote_last = false;
  for (int ch = chunk_first; ch < chunk_first + tp.chunks_per_split; ch++) {
    const int c0 = ch * kTileCC;
    if (c0 >= g.C) break;
    const int cc = (g.C - c0 < kTileCC) ? g.C - c0 : kTileCC;
    wrote_last = c0 + cc == g.C;
    __syncthreads();
    if (ch == chunk_first || cc != kTileCC) build_offsets(off, cc, g, tp);
    stage_tile<float>(tile, x, x_bf16, g, b, c0, cc, yo0, tp, KeepF32());
    __syncthreads();
    const int chunk_elems = cc * taps;
    const int words = (chunk_elems + 31) / 32;
    for (int idx = threadIdx.x; idx < pix_pad * words; idx += 256) {
      const int w = idx / pix_pad, pix = idx - w * pix_pad;
      if (pix >= pixels) continue;
      const int ry = pix / g.Wo, xo = pix - ry * g.Wo;
      const int k_begin = w * 32;
      const int nk = (chunk_elems - k_begin < 32) ? chunk_elems - k_begin : 32;
      const float* base = tile + ry * g.sh * tp.span + xo;
      const unsigned short* o = off + k_begin;
      uint32_t word = 0;
      float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
      if (cc == kTileCC && g.kh == 3 && g.kw == 3) {
        gather_word_dispatch<3, 3>(w, static_cast<uint32_t>(__cvta_generic_to_shared(base)), tp.rows_in * tp.span * 4, tp.span * 4, 0u, word, s0);
      } else if (cc == kTileCC && taps == 1) {
        gather_word_dispatch<1, 1>(w, static_cast<uint32_t>(__cvta_generic_to_shared(base)), tp.rows_in * tp.span * 4, tp.span * 4, 0u, word, s0);
      } else if (nk == 32) {
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          const float v0 = base[o[e]], v1 = base[o[e + 1]], v2 = base[o[e + 2]], v3 = base[o[e + 3]];
          word |= (v0 >= 0.0f ? 1u : 0u) << e;
          word |= (v1 >= 0.0f ? 1u : 0u) << (e + 1);
          word |= (v2 >= 0.0f ? 1u : 0u) << (e + 2);
          word |= (v3 >= 0.0f ? 1u : 0u) << (e + 3);
          s0 += fabsf(v0); s1 += fabsf(v1); s2 += fabsf(v2); s3 += fabsf(v3);
        }
      } else {
        for (int e = 0; e < nk; e++) {
          const float v = base[o[e]];
          word |= (v >= 0.0f ? 1u : 0u) << e;
          s0 += fabsf(v);
        }
      }
      out_bits[pix * ldo + words_done + w] = word;
      out_scale[pix * ldo + words_done + w] = ((s0 + s1) + (s2 + s3)) / static_cast<float>(nk);
    }
    words_done += words;
  }
  __syncthreads();
  // contiguous runs: for each pixel the block's words, then (last range only) the zero padding
  const int64_t word0 = static_cast<int64_t>(chunk_first) * kTileCC * taps / 32;
  const int run_bits = wrote_last ? static_cast<int>(ld_words - word0) : words_done;
  const int run_scale = wrote_last ? static_cast<int>(ld_scales - word0) : words_done;
  const int64_t m_base = (b * g.Ho + yo0) * g.Wo;
  for (int idx = threadIdx.x; idx < pixels * run_bits; idx += 256) {
    const int pix = idx / run_bits, w = idx - pix * run_bits;
    bits[(m_base + pix) * ld_words + word0 + w] = (w < words_done) ? out_bits[pix * ldo + w] : 0u;
  }
  for (int idx = threadIdx.x; idx < pixels * run_scale; idx += 256) {
    const int pix = idx / run_scale, w = idx - pix * run_scale;
    store_scale(scales, scale_bf16, (m_base + pix) * ld_scales + word0 + w, (w < words_done) ? out_scale[pix * ldo + w] : 0.0f);
  }
}

}  // namespace

cudaError_t launch_im2col_quantize(const void* x, int x_bf16, const ConvGeom& g, int32_t beta,
                                   uint32_t* bits, int64_t ld_words, void* scales, int64_t ld_scales,
                                   int scale_bf16, cudaStream_t stream) {
  const int64_t M = static_cast<int64_t>(g.B) * g.Ho * g.Wo, K = static_cast<int64_t>(g.C) * g.kh * g.kw;
  const int64_t beta_eff = beta >= K ? K : beta;
  const int64_t G = num_groups(K, beta);
  if (im2col_quantize_tma_supported(x, x_bf16, g, beta))
    return launch_im2col_quantize_tma(x, g, beta, bits, ld_words, scales, ld_scales, scale_bf16, stream);
  if (beta == 32 && beta < K && g.sw == 1) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const TilePlan tp = make_plan(g, sms);
    const int taps = g.kh * g.kw;
    const size_t smem = static_cast<size_t>(kTileCC) * tp.rows_in * tp.span * 4 +
                        2 * static_cast<size_t>(tp.RB) * g.Wo * (tp.chunks_per_split * taps + 1) * 4 +
                        static_cast<size_t>(kTileCC) * taps * 2 + 16;
    if (smem <= 160 * 1024 && static_cast<int64_t>(kTileCC) * tp.rows_in * tp.span < 65536) {
      static DeviceOnce configured;            // the opt-in shared-memory size is a per-device attribute
      if (smem > 48 * 1024 && configured.pending(dev)) {
        if (cudaFuncSetAttribute(im2col_quantize_tiled_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 160 * 1024) != cudaSuccess) return cudaGetLastError();
        configured.mark(dev);
      }
      dim3 grid(static_cast<unsigned>(static_cast<int64_t>(g.B) * tp.yo_blocks), static_cast<unsigned>(tp.splits));
      im2col_quantize_tiled_kernel<<<grid, 256, smem, stream>>>(x, x_bf16, g, tp, K, G, (K + 31) / 32, bits, ld_words,
                                                                scales, ld_scales, scale_bf16);
      return cudaGetLastError();
    }
  }
  if (beta < K && beta % 32 == 0) {
    dim3 grid(static_cast<unsigned>((M + 31) / 32), static_cast<unsigned>((G + 7) / 8));
    im2col_quantize_groups_kernel<<<grid, 256, 0, stream>>>(x, x_bf16, g, M, K, beta / 32, G, (K + 31) / 32, bits,
                                                             ld_words, scales, ld_scales, scale_bf16);
    return cudaGetLastError();
  }
  const int64_t blocks = (M + kThreads - 1) / kThreads;
  im2col_quantize_kernel<<<static_cast<unsigned>(blocks), kThreads, 0, stream>>>(
      x, x_bf16, g, M, K, beta_eff, G, bits, ld_words, scales, ld_scales, scale_bf16);
  return cudaGetLastError();
}

cudaError_t launch_im2col_bf16(const void* x, int x_bf16, const ConvGeom& g, void* out, int64_t ld,
                               cudaStream_t stream) {
  const int64_t M = static_cast<int64_t>(g.B) * g.Ho * g.Wo, K = static_cast<int64_t>(g.C) * g.kh * g.kw;
  if (g.sw == 1 && ld % 8 == 0 && reinterpret_cast<uintptr_t>(out) % 16 == 0) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const TilePlan tp = make_plan(g, sms);
    const int taps = g.kh * g.kw;
    const size_t smem = static_cast<size_t>((kTileCC * taps + 7) / 8 * 8) * 2 + static_cast<size_t>(kTileCC) * tp.rows_in * tp.span * 2;
    if (smem <= 48 * 1024 && static_cast<int64_t>(kTileCC) * tp.rows_in * tp.span < 65536) {
      dim3 grid(static_cast<unsigned>(static_cast<int64_t>(g.B) * tp.yo_blocks), static_cast<unsigned>(tp.splits));
      im2col_bf16_tiled_kernel<<<grid, 256, smem, stream>>>(x, x_bf16, g, tp, K, reinterpret_cast<__nv_bfloat16*>(out), ld);
      return cudaGetLastError();
    }
  }
  int64_t blocks = (M * ld + 255) / 256;
  if (blocks > 148 * 64) blocks = 148 * 64;
  im2col_bf16_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(x, x_bf16, g, M, K,
                                                                         reinterpret_cast<__nv_bfloat16*>(out), ld);
  return cudaGetLastError();
}

}  // namespace hbmm
