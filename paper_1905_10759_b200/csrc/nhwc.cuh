// NCHW (fp32 or bf16) -> NHWC bf16 transposition of one 64-channel x 32-pixel patch (a 256-thread
// block's work), shared by the stand-alone copy kernel and by the kernel that fuses the copy with the
// weight-piece preparation of the HBWN convolution.
#pragma once
#include <cuda_bf16.h>
#include <cstdint>

namespace hbmm {

constexpr int kNhwcCB = 64, kNhwcPB = 64, kNhwcPitch = kNhwcPB + 2;

// Reads run along the pixels (contiguous in NCHW; two pixels per load when the rows allow 4-byte
// accesses), writes are 16-byte pieces of 8 channels, eight neighbouring lanes filling one 128-byte run
// of a pixel.  Channels C..Cp-1 are written as zeros.
__device__ __forceinline__ void nchw_to_nhwc_block(const void* __restrict__ x, int x_bf16, int C, int64_t HW, int Cp,
                                                   unsigned short* __restrict__ out, int64_t b, int cblock, int64_t pblock,
                                                   unsigned short (*tile)[kNhwcPitch]) {
  const int c0 = cblock * kNhwcCB;
  const int64_t p0 = pblock * kNhwcPB;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 pixel pairs x 8 channel rows per pass
  // two pixels per load when every channel plane starts on an even element and the tensor is aligned for it
  const bool pairs = (HW & 1) == 0 && reinterpret_cast<uintptr_t>(x) % (x_bf16 ? 4 : 8) == 0;
  uint32_t v[kNhwcCB / 8];
#pragma unroll
  for (int r = 0; r < kNhwcCB / 8; r++) {
    const int c = c0 + ty + 8 * r;
    const int64_t p = p0 + 2 * tx;
    v[r] = 0;
    if (c < C && p < HW) {
      const int64_t idx = (b * C + c) * HW + p;
      if (x_bf16) {
        const unsigned short* xs = reinterpret_cast<const unsigned short*>(x);
        if (pairs) v[r] = __ldg(reinterpret_cast<const uint32_t*>(xs + idx));
        else v[r] = __ldg(xs + idx) | (p + 1 < HW ? static_cast<uint32_t>(__ldg(xs + idx + 1)) << 16 : 0u);
      } else {
        const float* xf = reinterpret_cast<const float*>(x);
        float f0, f1 = 0.0f;
        if (pairs) { const float2 f = __ldg(reinterpret_cast<const float2*>(xf + idx)); f0 = f.x; f1 = f.y; }
        else { f0 = __ldg(xf + idx); if (p + 1 < HW) f1 = __ldg(xf + idx + 1); }
        v[r] = __bfloat16_as_ushort(__float2bfloat16_rn(f0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(f1))) << 16);
      }
    }
  }
#pragma unroll
  for (int r = 0; r < kNhwcCB / 8; r++) *reinterpret_cast<uint32_t*>(&tile[ty + 8 * r][2 * tx]) = v[r];
  __syncthreads();
  const int piece = threadIdx.x & 7;                           // 8 pieces of 8 channels
  const int c = c0 + piece * 8;
#pragma unroll
  for (int h = 0; h < 2; h++) {                                // 64 pixels: two per thread
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
