// Packed convolution front end (fp32 NCHW input; groups of 2, 4, 8, 16 elements or of whole K-words) with the
// input tile staged by tensor copies.  A work item is RB output rows of one image and a range of 32-channel chunks.  For every
// chunk one 4-D tensor copy brings [32 channels][rows_in input rows][pitch columns] into shared
// memory, zero halo included (the copy starts left of and above the image where the padding asks
// for it, and whatever lies outside the tensor arrives as zeros).  Two persistent CTAs per SM: a
// loader thread keeps a ring of tile buffers full across chunks and items, twelve compute warps
// binarize.  A warp-item is 32 consecutive pixels of one K-word, so tile reads are consecutive.
// Words and scales of an item are collected in shared memory and leave as contiguous 16-byte runs.
// Every wait is bounded (error word + CTA-wide abort flag, as in the tensor-core kernels).
#include <cuda_bf16.h>
#include "kernels.h"
#include "tensor_map.h"
#include "umma_common.cuh"
#include "im2col_gather.cuh"
#include "gemm_umma_prep.cuh"
#include "gemm_fold_prep.cuh"
#include "pdl.cuh"

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
  int ring;               // tile buffers per CTA
  int flat;               // 1: whole channel planes staged by one bulk copy per chunk, no halo (pitch = W, rows_in = H)
  int tile_stride;        // floats between ring buffers (tile rounded up to 128 bytes)
  int sub;                // scale groups per K-word (beta = 32 / sub), 1 for groups of whole words
  int gw;                 // K-words per scale group (beta = 32 * gw), 1 for groups of at most a word
  int vec_scales;         // sub > 1: a word's fp32 scales may leave as 16-byte (8-byte for sub = 2) stores
};

// One K-word of a full 32-channel chunk whose groups are shorter than a word: the packed word, and the word's SUB
// group means stored straight to the operand's scale row (`dst`: the word's first scale).
template <int SUB>
__device__ __forceinline__ void gather_word_sub(int taps, bool flat, int w, uint32_t addr, uint32_t cs_bytes, uint32_t pitch_bytes,
                                                uint32_t pm, uint32_t& word, void* scales, int scale_bf16, int64_t idx, bool vec) {
  float sums[SUB];
  if (taps == 9) {
    if (flat) gather_word_dispatch_sub<3, 3, true, SUB>(w, addr, cs_bytes, pitch_bytes, pm, word, sums);
    else gather_word_dispatch_sub<3, 3, false, SUB>(w, addr, cs_bytes, pitch_bytes, 0u, word, sums);
  } else {
    if (flat) gather_word_dispatch_sub<1, 1, true, SUB>(w, addr, cs_bytes, pitch_bytes, pm, word, sums);
    else gather_word_dispatch_sub<1, 1, false, SUB>(w, addr, cs_bytes, pitch_bytes, 0u, word, sums);
  }
  constexpr float inv = static_cast<float>(SUB) / 32.0f;          // 1 / beta
#pragma unroll
  for (int i = 0; i < SUB; i++) sums[i] *= inv;
  if (vec) {
    float* d = reinterpret_cast<float*>(scales) + idx;
    if constexpr (SUB == 2) {
      *reinterpret_cast<float2*>(d) = make_float2(sums[0], sums[1]);
    } else {
#pragma unroll
      for (int i = 0; i < SUB; i += 4) *reinterpret_cast<float4*>(d + i) = make_float4(sums[i], sums[i + 1], sums[i + 2], sums[i + 3]);
    }
  } else {
#pragma unroll
    for (int i = 0; i < SUB; i++) {
      if (scale_bf16) reinterpret_cast<__nv_bfloat16*>(scales)[idx + i] = __float2bfloat16_rn(sums[i]);
      else reinterpret_cast<float*>(scales)[idx + i] = sums[i];
    }
  }
}

__device__ __forceinline__ void store_scale(void* scales, int bf16, int64_t idx, float v) {
  if (bf16) reinterpret_cast<__nv_bfloat16*>(scales)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(scales)[idx] = v;
}

constexpr int kComputeWarps = 12;                    // 36 warp-items per chunk of 112..128 pixels: three rounds
constexpr int kLoaderWarp = kComputeWarps;
constexpr int kThreadsTma = (kComputeWarps + 1) * 32;
constexpr int kMaxRing = 6;

// Work item = (row block of one image, channel range).  A CTA is persistent: it walks items
// blockIdx.x, blockIdx.x + gridDim.x, ... and the ring of tile buffers simply continues across items,
// so the copies of the next item are in flight while the current one is binarized and written out.
struct ItemCoords {
  int32_t b, yo0, chunk_first, n_my;
};
__device__ __forceinline__ ItemCoords item_coords(int item, const Plan& tp) {
  ItemCoords c;
  const int rb = item / tp.splits, sp = item - rb * tp.splits;
  c.b = rb / tp.yo_blocks;
  c.yo0 = (rb - c.b * tp.yo_blocks) * tp.RB;
  c.chunk_first = sp * tp.chunks_per_split;
  c.n_my = (tp.n_chunks - c.chunk_first < tp.chunks_per_split) ? tp.n_chunks - c.chunk_first : tp.chunks_per_split;
  return c;
}

// GROUPS: 0 -- groups of exactly one K-word; 1 -- groups shorter than a word; 2 -- groups of several words.  The three are
// separate instantiations so that the one-word kernel carries none of the others' code or registers.
template <int GROUPS>
__global__ void __launch_bounds__(kThreadsTma, 2)
im2col_quantize_tma_kernel(const __grid_constant__ CUtensorMap x_map, const float* __restrict__ x, const ConvGeom g, const Plan tp,
                           const __grid_constant__ UmmaPrepJob prep, int n_prep, int n_items, int ring,
                           uint32_t* __restrict__ bits, int64_t ld_words, void* __restrict__ scales, int64_t ld_scales,
                           int scale_bf16) {
  pdl_launch_dependents();      // the next kernel of the stream may start its own set-up
  // The first n_prep CTAs expand the weight operand of the contraction that follows (one task each:
  // a stage of one column tile, one thread per weight row); they are scheduled first and leave at once.
  if (static_cast<int>(blockIdx.x) < n_prep) {
    pdl_wait();                 // the workspace may still be read by the kernel before this one
    const int st = blockIdx.x % prep.n_stages, tile_n = blockIdx.x / prep.n_stages;
    if (prep.folded) {
      if (prep.tn == 64) { if (threadIdx.x < 64) fold::prepare_w_task<64>(prep.f, prep.out, prep.out_down, st, tile_n, threadIdx.x); }
      else if (threadIdx.x < 128) fold::prepare_w_task<128>(prep.f, prep.out, prep.out_down, st, tile_n, threadIdx.x);
    } else {
      if (prep.tn == 64) { if (threadIdx.x < 64) umma_prep::prepare_w_task<64>(prep.g, prep.out, st, tile_n, threadIdx.x); }
      else if (threadIdx.x < 128) umma_prep::prepare_w_task<128>(prep.g, prep.out, st, tile_n, threadIdx.x);
    }
    return;
  }
  const int cta = blockIdx.x - n_prep, n_ctas = gridDim.x - n_prep;      // the persistent CTAs of the front end
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int taps = g.kh * g.kw;
  const int tile_elems = tp.tile_stride;                        // floats per ring buffer; bytes are a multiple of 128
  const int max_pixels = tp.RB * g.Wo;
  const int split_words = tp.chunks_per_split * taps;          // words an item produces per pixel (upper bound)
  const int ldo = split_words + 1;                             // odd-ish pitch: fewer bank conflicts on the column writes
  float* tile0 = reinterpret_cast<float*>(smem_raw);                                   // `ring` tile buffers
  uint64_t* full = reinterpret_cast<uint64_t*>(tile0 + static_cast<size_t>(ring) * tile_elems);
  uint64_t* empty = full + kMaxRing;
  uint64_t* computed = empty + kMaxRing;                       // all compute warps are done with an item's chunks
  uint64_t* written = computed + 1;                            // ... and with its write-out
  volatile int* abort_flag = reinterpret_cast<volatile int*>(written + 1);
  uint32_t* out_bits = reinterpret_cast<uint32_t*>(written + 2);                      // [max_pixels][ldo]
  float* out_scale = reinterpret_cast<float*>(out_bits + max_pixels * ldo);           // same shape
  unsigned short* off = reinterpret_cast<unsigned short*>(out_scale + max_pixels * ldo);    // [32 * taps]
  short* pixoff = reinterpret_cast<short*>(off + (kCC * taps + 1) / 2 * 2);                 // [max_pixels]
  unsigned short* pixmask = reinterpret_cast<unsigned short*>(pixoff + (max_pixels + 1) / 2 * 2);   // [max_pixels], flat mode

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cs = tp.rows_in * tp.pitch;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kMaxRing; s++) { mbar_init(&full[s], 1); mbar_init(&empty[s], kComputeWarps); }
    mbar_init(computed, kComputeWarps);
    mbar_init(written, kComputeWarps);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // chunk-local k -> offset of tap (c, i, j) inside the tile, for filter sizes without an unrolled gather
  for (int k = threadIdx.x; k < kCC * taps; k += blockDim.x) {
    const int c = k / taps, r = k - c * taps, i = r / g.kw, j = r - i * g.kw;
    off[k] = static_cast<unsigned short>(c * cs + i * tp.pitch + j);
  }
  // pixel of an item -> tile offset of its first tap (channel 0, filter row 0, column 0)
  for (int pix = threadIdx.x; pix < max_pixels; pix += blockDim.x) {
    const int ry = pix / g.Wo, xo = pix - ry * g.Wo;
    if (!tp.flat) {
      pixoff[pix] = static_cast<short>(ry * g.sh * tp.pitch + xo + tp.x0);
      pixmask[pix] = 0;
    } else {
      // no halo: the offset of tap (0, 0) may point before the plane; the masks say which taps exist
      const int y0 = ry * g.sh - g.ph, x0 = xo - g.pw;
      pixoff[pix] = static_cast<short>(y0 * tp.pitch + x0);
      unsigned m = 0;
      for (int j = 0; j < g.kw; j++) if (x0 + j >= 0 && x0 + j < g.W) m |= 1u << j;
      for (int i = 0; i < g.kh; i++) if (y0 + i >= 0 && y0 + i < g.H) m |= 1u << (8 + i);
      pixmask[pix] = static_cast<unsigned short>(m);
    }
  }
  pdl_wait();                   // the tables above live in shared memory; global memory is touched from here on
  __syncthreads();

  if (warp == kLoaderWarp) {
    // =========================== loader ===========================
    if (lane == 0) {
      const uint32_t tile_bytes = static_cast<uint32_t>(kCC) * tp.rows_in * tp.pitch * 4;
      const int64_t plane = static_cast<int64_t>(g.H) * g.W;
      asm volatile("prefetch.tensormap [%0];" ::"l"(&x_map) : "memory");
      int s = 0;
      uint32_t round = 0;
      int issued = 0;                                          // copies issued so far (for the abort path)
      bool ok = true;
      for (int item = cta; item < n_items && ok; item += n_ctas) {
        const ItemCoords ic = item_coords(item, tp);
        for (int it = 0; it < ic.n_my; it++) {
          if (round > 0 && !mbar_wait(&empty[s], (round & 1) ^ 1, abort_flag, 1)) { ok = false; break; }
          mbar_arrive_expect_tx(&full[s], tile_bytes);
          // x starts at -(x0 + pw), a multiple of 4 elements = 16 bytes; y may be negative too; what lies
          // outside the tensor (halo, channels past C) arrives as zeros
          if (tp.flat)   // 32 whole channel planes are one contiguous, 16-byte aligned run of the NCHW tensor
            bulk_copy_g2s(tile0 + static_cast<size_t>(s) * tile_elems,
                          x + (static_cast<int64_t>(ic.b) * g.C + (ic.chunk_first + it) * kCC) * plane, tile_bytes, &full[s]);
          else
            tma_load_4d(tile0 + static_cast<size_t>(s) * tile_elems, &x_map, -(tp.x0 + g.pw), ic.yo0 * g.sh - g.ph,
                        (ic.chunk_first + it) * kCC, ic.b, &full[s]);
          issued++;
          if (++s == ring) { s = 0; round++; }
        }
      }
      if (!ok) {
        // aborted: let the copies already issued land before the CTA's shared memory goes away
        const int pending = issued < ring ? issued : ring;
        for (int q = 0; q < pending; q++) {
          const int idx = issued - 1 - q, slot = idx % ring;
          mbar_wait_quiet(&full[slot], static_cast<uint32_t>((idx / ring) & 1), kDrainPolls);
        }
      }
    }
    __syncwarp();
    return;
  }

  // =========================== compute warps ===========================
  int s = 0;
  uint32_t round = 0, phase = 0;                               // ring position; parity of `computed` / `written`
  for (int item = cta; item < n_items; item += n_ctas) {
    const ItemCoords ic = item_coords(item, tp);
    const int rows = (g.Ho - ic.yo0 < tp.RB) ? g.Ho - ic.yo0 : tp.RB;
    const int pixels = rows * g.Wo;
    const int pix_warps = (pixels + 31) / 32;                  // a warp stays on one word: 32 pixels x 1 word per warp-item
    int words_done = 0;                                        // words produced so far for this item
    bool wrote_last = false;
    for (int it = 0; it < ic.n_my; it++) {
      const int c0 = (ic.chunk_first + it) * kCC;
      const int cc = (g.C - c0 < kCC) ? g.C - c0 : kCC;
      wrote_last = c0 + cc == g.C;
      if (!mbar_wait(&full[s], round & 1, abort_flag, 2)) return;
      const float* t = tile0 + static_cast<size_t>(s) * tile_elems;
      const int chunk_elems = cc * taps;
      const int words = (chunk_elems + 31) / 32;
      // warp-items (w, pw): word w of pixel group pw; walked with a stride of kComputeWarps, indices carried along
      int pw = warp % pix_warps, w = warp / pix_warps;
      const int dpw = kComputeWarps % pix_warps, dw = kComputeWarps / pix_warps;
      const uint32_t t_addr = smem_u32(t);
      for (; w < words; ) {
        const int pix = pw * 32 + lane;
        if (pix < pixels) {
          const int k_begin = w * 32;
          const int nk = (chunk_elems - k_begin < 32) ? chunk_elems - k_begin : 32;
          const int po = pixoff[pix];                          // tile offset of the pixel's first tap, in elements
          const uint32_t pm = pixmask[pix];
          uint32_t word = 0;
          float mean = 0.0f;
          const int word_abs = static_cast<int>(static_cast<int64_t>(ic.chunk_first) * kCC * taps / 32) + words_done + w;
          const int64_t m_pix = (static_cast<int64_t>(ic.b) * g.Ho + ic.yo0) * g.Wo + pix;
          if (GROUPS == 1 && cc == kCC && (taps == 9 ? (g.kh == 3 && g.kw == 3) : taps == 1)) {
            // groups shorter than a word: the word's means go straight to the scale row
            const int64_t sidx = m_pix * ld_scales + static_cast<int64_t>(word_abs) * tp.sub;
            const uint32_t a = t_addr + po * 4;
            const bool vec = tp.vec_scales != 0;
            switch (tp.sub) {
              case 2: gather_word_sub<2>(taps, tp.flat != 0, w, a, cs * 4, tp.pitch * 4, pm, word, scales, scale_bf16, sidx, vec); break;
              case 4: gather_word_sub<4>(taps, tp.flat != 0, w, a, cs * 4, tp.pitch * 4, pm, word, scales, scale_bf16, sidx, vec); break;
              case 8: gather_word_sub<8>(taps, tp.flat != 0, w, a, cs * 4, tp.pitch * 4, pm, word, scales, scale_bf16, sidx, vec); break;
              default: gather_word_sub<16>(taps, tp.flat != 0, w, a, cs * 4, tp.pitch * 4, pm, word, scales, scale_bf16, sidx, vec); break;
            }
          } else if (GROUPS == 1) {
            // any filter size, short last chunk: group by group (the last group of the row may be short)
            const float* base = t + po;
            const unsigned short* o = off + k_begin;
            const int beta = 32 / tp.sub;
            for (int e0 = 0; e0 < nk; e0 += beta) {
              const int cnt = (nk - e0 < beta) ? nk - e0 : beta;
              float sum = 0.0f;
              for (int e = e0; e < e0 + cnt; e++) {
                const float v = base[o[e]];
                word |= (v >= 0.0f ? 1u : 0u) << e;
                sum += fabsf(v);
              }
              store_scale(scales, scale_bf16, m_pix * ld_scales + static_cast<int64_t>(word_abs) * tp.sub + e0 / beta, sum / static_cast<float>(cnt));
            }
          } else if (cc == kCC && g.kh == 3 && g.kw == 3) {
            float sum;
            if (tp.flat) gather_word_dispatch<3, 3, true>(w, t_addr + po * 4, cs * 4, tp.pitch * 4, pm, word, sum);
            else gather_word_dispatch<3, 3, false>(w, t_addr + po * 4, cs * 4, tp.pitch * 4, 0u, word, sum);
            mean = GROUPS == 2 ? sum : sum * 0.03125f;
          } else if (cc == kCC && taps == 1) {
            float sum;
            if (tp.flat) gather_word_dispatch<1, 1, true>(w, t_addr + po * 4, cs * 4, tp.pitch * 4, pm, word, sum);
            else gather_word_dispatch<1, 1, false>(w, t_addr + po * 4, cs * 4, tp.pitch * 4, 0u, word, sum);
            mean = GROUPS == 2 ? sum : sum * 0.03125f;
          } else {
            const float* base = t + po;
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
            mean = ((s0 + s1) + (s2 + s3)) / static_cast<float>(nk);
            if (GROUPS == 2) mean = (s0 + s1) + (s2 + s3);
          }
          out_bits[pix * ldo + words_done + w] = word;
          out_scale[pix * ldo + words_done + w] = mean;          // gw > 1: the word's sum of |x| (see the two fast branches)
        }
        pw += dpw; w += dw;
        if (pw >= pix_warps) { pw -= pix_warps; w++; }
      }
      words_done += words;
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);                   // this warp is done with the tile
      if (++s == ring) { s = 0; round++; }
    }
    // every compute warp has produced its part of the item
    __syncwarp();
    if (lane == 0) mbar_arrive(computed);
    if (!mbar_wait(computed, phase, abort_flag, 3)) return;

    // contiguous runs: for each pixel the item's words, then (last range only) the zero padding
    const int tid = threadIdx.x, nthr = kComputeWarps * 32;
    const int64_t word0 = static_cast<int64_t>(ic.chunk_first) * kCC * taps / 32;
    const int run_bits = wrote_last ? static_cast<int>(ld_words - word0) : words_done;
    const int run_scale = wrote_last ? static_cast<int>(ld_scales - word0) : words_done;
    const int64_t m_base = (static_cast<int64_t>(ic.b) * g.Ho + ic.yo0) * g.Wo;
    if ((word0 & 3) == 0 && (run_bits & 3) == 0) {
      const int q_per = run_bits >> 2;                         // 16-byte pieces per pixel
      for (int idx = tid; idx < pixels * q_per; idx += nthr) {
        const int pix = idx / q_per, w = (idx - pix * q_per) * 4;
        const uint32_t* src = out_bits + pix * ldo + w;
        uint4 o;
        o.x = (w < words_done) ? src[0] : 0u; o.y = (w + 1 < words_done) ? src[1] : 0u;
        o.z = (w + 2 < words_done) ? src[2] : 0u; o.w = (w + 3 < words_done) ? src[3] : 0u;
        *reinterpret_cast<uint4*>(bits + (m_base + pix) * ld_words + word0 + w) = o;
      }
    } else {
      for (int idx = tid; idx < pixels * run_bits; idx += nthr) {
        const int pix = idx / run_bits, w = idx - pix * run_bits;
        bits[(m_base + pix) * ld_words + word0 + w] = (w < words_done) ? out_bits[pix * ldo + w] : 0u;
      }
    }
    if (GROUPS == 1) {
      // the means were stored by the gather; the last channel range zeroes the row's padding
      if (wrote_last) {
        const int64_t K = static_cast<int64_t>(g.C) * taps;
        const int beta = 32 / tp.sub;
        const int64_t G = (K + beta - 1) / beta;
        const int pad = static_cast<int>(ld_scales - G);
        for (int idx = tid; idx < pixels * pad; idx += nthr) {
          const int pix = idx / pad, q = idx - pix * pad;
          store_scale(scales, scale_bf16, (m_base + pix) * ld_scales + G + q, 0.0f);
        }
      }
    } else if (GROUPS == 2) {
      // groups of gw words: add the words' sums (word0 is a multiple of gw, and so is the item's word count unless
      // it ends the row); the row's last group may be short
      const int64_t K = static_cast<int64_t>(g.C) * taps;
      const int64_t beta = 32LL * tp.gw;
      const int64_t group0 = word0 / tp.gw;
      const int n_groups = (words_done + tp.gw - 1) / tp.gw;
      const int run = wrote_last ? static_cast<int>(ld_scales - group0) : n_groups;
      for (int idx = tid; idx < pixels * run; idx += nthr) {
        const int pix = idx / run, q = idx - pix * run;
        float v = 0.0f;
        if (q < n_groups) {
          const int w_end = ((q + 1) * tp.gw < words_done) ? (q + 1) * tp.gw : words_done;
          for (int w = q * tp.gw; w < w_end; w++) v += out_scale[pix * ldo + w];
          const int64_t left = K - (group0 + q) * beta;
          v /= static_cast<float>(left < beta ? left : beta);
        }
        store_scale(scales, scale_bf16, (m_base + pix) * ld_scales + group0 + q, v);
      }
    } else if (!scale_bf16 && (word0 & 3) == 0 && (run_scale & 3) == 0) {
      const int q_per = run_scale >> 2;
      float* sc = reinterpret_cast<float*>(scales);
      for (int idx = tid; idx < pixels * q_per; idx += nthr) {
        const int pix = idx / q_per, w = (idx - pix * q_per) * 4;
        const float* src = out_scale + pix * ldo + w;
        float4 o;
        o.x = (w < words_done) ? src[0] : 0.f; o.y = (w + 1 < words_done) ? src[1] : 0.f;
        o.z = (w + 2 < words_done) ? src[2] : 0.f; o.w = (w + 3 < words_done) ? src[3] : 0.f;
        *reinterpret_cast<float4*>(sc + (m_base + pix) * ld_scales + word0 + w) = o;
      }
    } else {
      for (int idx = tid; idx < pixels * run_scale; idx += nthr) {
        const int pix = idx / run_scale, w = idx - pix * run_scale;
        store_scale(scales, scale_bf16, (m_base + pix) * ld_scales + word0 + w, (w < words_done) ? out_scale[pix * ldo + w] : 0.0f);
      }
    }
    // the staging arrays may be overwritten once every warp has read its part of them
    __syncwarp();
    if (lane == 0) mbar_arrive(written);
    if (!mbar_wait(written, phase, abort_flag, 4)) return;
    phase ^= 1;
  }
}

inline int round_up4(int v) { return (v + 3) / 4 * 4; }

bool make_plan(const ConvGeom& g, int sms, bool flat, int32_t beta, Plan* out, size_t* smem_bytes) {
  Plan p;
  p.flat = flat ? 1 : 0;
  p.sub = beta < 32 ? 32 / beta : 1;
  p.gw = beta > 32 ? beta / 32 : 1;
  p.vec_scales = 0;
  if (flat) {
    p.RB = g.Ho;                                               // an item covers the whole image
    p.rows_in = g.H;
    p.x0 = 0;
    p.pitch = g.W;
  } else {
    p.RB = 112 / g.Wo;
    if (p.RB < 1) p.RB = 1;
    if (p.RB > g.Ho) p.RB = g.Ho;
    p.rows_in = (p.RB - 1) * g.sh + g.kh;
    const int span = g.Wo - 1 + g.kw;                          // input columns the item's taps touch (stride 1 along x)
    p.x0 = round_up4(g.pw) - g.pw;
    p.pitch = round_up4(p.x0 + span);
  }
  p.yo_blocks = (g.Ho + p.RB - 1) / p.RB;
  p.n_chunks = (g.C + kCC - 1) / kCC;
  const int64_t row_blocks = static_cast<int64_t>(g.B) * p.yo_blocks;
  int splits = 1;
  while (row_blocks * splits < 2LL * sms && splits * 2 <= p.n_chunks) splits *= 2;
  const int taps = g.kh * g.kw;
  p.chunks_per_split = (p.n_chunks + splits - 1) / splits;
  // groups of several words must not straddle two channel ranges
  while (splits > 1 && (p.chunks_per_split * taps) % p.gw != 0) {
    splits /= 2;
    p.chunks_per_split = (p.n_chunks + splits - 1) / splits;
  }
  p.splits = (p.n_chunks + p.chunks_per_split - 1) / p.chunks_per_split;
  const int64_t tile_elems = static_cast<int64_t>(kCC) * p.rows_in * p.pitch;
  p.tile_stride = static_cast<int>((tile_elems + 31) / 32 * 32);
  const int64_t max_pixels = static_cast<int64_t>(p.RB) * g.Wo;
  // everything but the tile ring: barriers, staging arrays of one item, offset / pixel tables
  const int64_t fixed = (2 * kMaxRing + 4) * 8 + 2 * max_pixels * (p.chunks_per_split * taps + 1) * 4 +
                        static_cast<int64_t>(kCC) * taps * 2 + 4 * max_pixels + 64;
  const int64_t budget = 100 * 1024;                           // two CTAs per SM: one computes while the other synchronises or writes
  int64_t ring = (budget - fixed) / (p.tile_stride * 4);
  if (ring > kMaxRing) ring = kMaxRing;
  p.ring = static_cast<int>(ring);
  *smem_bytes = static_cast<size_t>(ring * p.tile_stride * 4 + fixed);
  *out = p;
  // offsets are 16-bit (signed for the pixel table)
  return (flat || (p.pitch <= 256 && p.rows_in <= 256)) && tile_elems < 32768 && max_pixels < 32768 && ring >= 2;
}

// 0: not supported, 1: tensor-copy tiles with halo, 2: flat channel planes
int tma_mode(const void* x, int x_bf16, const ConvGeom& g, int32_t beta) {
  const int64_t K = static_cast<int64_t>(g.C) * g.kh * g.kw;
  const bool beta_ok = beta == 2 || beta == 4 || beta == 8 || beta == 16 || (beta >= 32 && beta % 32 == 0 && beta / 32 <= 64);
  if (x_bf16 || !beta_ok || beta >= K || g.sw != 1 || reinterpret_cast<uintptr_t>(x) % 16 != 0) return 0;
  Plan p;
  size_t smem;
  int dev = 0, sms = 0;
  if (current_device(&dev, &sms) != cudaSuccess) return 0;       // the plan's channel split follows the device's SM count
  if (g.W % 4 == 0 && encode_tiled_fn() != nullptr && make_plan(g, sms, false, beta, &p, &smem)) return 1;
  // small images whose rows are not multiples of 16 bytes: whole planes, masked 3x3 / 1x1 gather
  const bool filt = (g.kh == 3 && g.kw == 3) || (g.kh == 1 && g.kw == 1);
  if (filt && g.C % kCC == 0 && (static_cast<int64_t>(g.C) * g.H * g.W) % 4 == 0 && make_plan(g, sms, true, beta, &p, &smem)) return 2;
  return 0;
}

}  // namespace

// fp32 input, stride 1 along x, groups of 2, 4, 8, 16 elements or of whole K-words (fewer than the row has); rows that are multiples of 16 bytes (a
// tensor map wants 16-byte strides), or small images with 3x3 / 1x1 filters and whole 32-channel chunks.
bool im2col_quantize_tma_supported(const void* x, int x_bf16, const ConvGeom& g, int32_t beta) {
  return tma_mode(x, x_bf16, g, beta) != 0;
}

cudaError_t launch_im2col_quantize_tma(const void* x, const ConvGeom& g, int32_t beta, uint32_t* bits, int64_t ld_words, void* scales,
                                       int64_t ld_scales, int scale_bf16, cudaStream_t stream, const UmmaPrepJob* prep) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int mode = tma_mode(x, 0, g, beta);
  Plan p;
  size_t smem;
  if (mode == 0 || !make_plan(g, sms, mode == 2, beta, &p, &smem)) return cudaErrorNotSupported;
  p.vec_scales = (p.sub > 1 && !scale_bf16 && reinterpret_cast<uintptr_t>(scales) % 16 == 0 && ld_scales % 4 == 0) ? 1 : 0;
  CUtensorMap map{};
  if (mode == 1) {
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
  }
  static DeviceOnce configured;
  if (configured.pending(dev)) {
    cudaError_t e = cudaFuncSetAttribute(im2col_quantize_tma_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 104 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(im2col_quantize_tma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 104 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(im2col_quantize_tma_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 104 * 1024);
    if (e != cudaSuccess) return e;
    configured.mark(dev);
  }
  const int64_t n_items = static_cast<int64_t>(g.B) * p.yo_blocks * p.splits;
  if (n_items > (int64_t{1} << 30)) return cudaErrorNotSupported;
  const unsigned grid = static_cast<unsigned>(n_items < 2 * sms ? n_items : 2 * sms);     // two persistent CTAs per SM
  UmmaPrepJob job{};
  int n_prep = 0;
  if (prep) {
    job = *prep;
    n_prep = job.n_stages * job.tiles_n;
    if (n_prep > 4096) return cudaErrorNotSupported;       // the caller expands large weight operands on its own
  }
  auto kernel = p.sub > 1 ? im2col_quantize_tma_kernel<1> : (p.gw > 1 ? im2col_quantize_tma_kernel<2> : im2col_quantize_tma_kernel<0>);
  return launch_pdl(kernel, dim3(grid + n_prep), dim3(kThreadsTma), smem, stream, map, static_cast<const float*>(x), g, p,
                    job, n_prep, static_cast<int>(n_items), p.ring, bits, ld_words, scales, ld_scales, scale_bf16);
}

cudaError_t im2col_tma_health(int op, int* value) {
  switch (op) {
    case kHealthRead: return umma::read_error_word(value);
    case kHealthClear: return umma::clear_error_word();
    case kHealthSetSpinLimit: return umma::set_spin_limit(static_cast<uint32_t>(*value));
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace hbmm
