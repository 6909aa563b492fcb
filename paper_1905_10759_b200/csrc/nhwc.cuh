// NCHW (fp32 or bf16) -> NHWC bf16 transposition of one 64-channel x PB-pixel patch (a 256-thread
// block's work), shared by the stand-alone copy kernel and by the kernel that fuses the copy with the
// weight-piece preparation of the HBWN convolution.
#pragma once
#include <cuda_bf16.h>
#include <cstdint>

namespace hbmm {

constexpr int kNhwcCB = 64;
// Pixels per block: 128 for planes of 512 pixels or more (a lane then reads 8 or 16 bytes per channel row),
// 64 for small planes, where longer blocks would be mostly empty.
constexpr int kNhwcPBLarge = 128, kNhwcPBSmall = 64;
__host__ __device__ constexpr int nhwc_pitch(int pb) { return pb + 2; }
inline int nhwc_pixels_per_block(int64_t HW) { return HW >= 512 ? kNhwcPBLarge : kNhwcPBSmall; }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  return __bfloat16_as_ushort(__float2bfloat16_rn(lo)) | (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(hi))) << 16);
}

// Reads run along the pixels (contiguous in NCHW; PB / 32 pixels per lane and channel row, as one vector load when
// the planes allow it), writes are 16-byte pieces of 8 channels, eight neighbouring lanes filling one 128-byte run
// of a pixel.  Channels C..Cp-1 are written as zeros.
template <int PB>
__device__ __forceinline__ void nchw_to_nhwc_block(const void* __restrict__ x, int x_bf16, int C, int64_t HW, int Cp,
                                                   unsigned short* __restrict__ out, int64_t b, int cblock, int64_t pblock,
                                                   unsigned short (*tile)[nhwc_pitch(PB)]) {
  constexpr int PPL = PB / 32;                                // pixels per lane: 2 or 4
  const int c0 = cblock * kNhwcCB;
  const int64_t p0 = pblock * PB;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 pixel runs x 8 channel rows per pass
  // one vector load per run when every channel plane starts on a multiple of the run and the tensor is aligned for it
  const bool vec = (HW % PPL) == 0 && reinterpret_cast<uintptr_t>(x) % (x_bf16 ? 2 * PPL : 4 * PPL) == 0;
  uint32_t v[kNhwcCB / 8][PPL / 2];
#pragma unroll
  for (int r = 0; r < kNhwcCB / 8; r++) {
    const int c = c0 + ty + 8 * r;
    const int64_t p = p0 + PPL * tx;
#pragma unroll
    for (int q = 0; q < PPL / 2; q++) v[r][q] = 0;
    if (c < C && p < HW) {
      const int64_t idx = (b * C + c) * HW + p;
      if (x_bf16) {
        const unsigned short* xs = reinterpret_cast<const unsigned short*>(x);
        if (vec) {
          if constexpr (PPL == 2) v[r][0] = __ldg(reinterpret_cast<const uint32_t*>(xs + idx));
          else { const uint2 u = __ldg(reinterpret_cast<const uint2*>(xs + idx)); v[r][0] = u.x; v[r][1] = u.y; }
        } else {
#pragma unroll
          for (int e = 0; e < PPL; e++)
            if (p + e < HW) v[r][e >> 1] |= static_cast<uint32_t>(__ldg(xs + idx + e)) << ((e & 1) * 16);
        }
      } else {
        const float* xf = reinterpret_cast<const float*>(x);
        float f[PPL];
#pragma unroll
        for (int e = 0; e < PPL; e++) f[e] = 0.0f;
        if (vec) {
          if constexpr (PPL == 2) { const float2 t = __ldg(reinterpret_cast<const float2*>(xf + idx)); f[0] = t.x; f[1] = t.y; }
          else { const float4 t = __ldg(reinterpret_cast<const float4*>(xf + idx)); f[0] = t.x; f[1] = t.y; f[2] = t.z; f[3] = t.w; }
        } else {
#pragma unroll
          for (int e = 0; e < PPL; e++)
            if (p + e < HW) f[e] = __ldg(xf + idx + e);
        }
#pragma unroll
        for (int q = 0; q < PPL / 2; q++) v[r][q] = pack_bf16x2(f[2 * q], f[2 * q + 1]);
      }
    }
  }
#pragma unroll
  for (int r = 0; r < kNhwcCB / 8; r++)
#pragma unroll
    for (int q = 0; q < PPL / 2; q++) *reinterpret_cast<uint32_t*>(&tile[ty + 8 * r][PPL * tx + 2 * q]) = v[r][q];
  __syncthreads();
  const int piece = threadIdx.x & 7;                           // 8 pieces of 8 channels
  const int c = c0 + piece * 8;
#pragma unroll
  for (int h = 0; h < PB / 32; h++) {                          // PB pixels: PB / 32 per thread
    const int pix = (threadIdx.x >> 3) + 32 * h;
    const int64_t p = p0 + pix;
    if (p < HW && c < Cp) {                                    // Cp is a multiple of 8: whole pieces
      uint32_t o[4];
#pragma unroll
      for (int e = 0; e < 4; e++)
        o[e] = tile[piece * 8 + 2 * e][pix] | (static_cast<uint32_t>(tile[piece * 8 + 2 * e + 1][pix]) << 16);
      *reinterpret_cast<uint4*>(out + (b * HW + p) * Cp + c) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

}  // namespace hbmm
