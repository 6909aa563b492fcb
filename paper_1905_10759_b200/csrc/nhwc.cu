// NCHW (fp32 or bf16) -> NHWC bf16 copy of a convolution input, channels padded with zeros to a
// multiple of 8 (16-byte pixels).  The HBWN convolution reads its activation tiles from this copy
// with im2col-mode tensor copies, which want the channel as the contiguous dimension.
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {
namespace {

// One block transposes a 64-channel x 32-pixel patch of one image: reads run along the pixels
// (contiguous in NCHW), writes are 16-byte pieces of 8 channels, eight neighbouring lanes filling one
// 128-byte run of a pixel.
constexpr int kCB = 64, kPB = 32, kPitch = kPB + 2;

__global__ void __launch_bounds__(256)
nchw_to_nhwc_bf16_kernel(const void* __restrict__ x, int x_bf16, int C, int64_t HW, int Cp,
                         unsigned short* __restrict__ out) {
  __shared__ unsigned short tile[kCB][kPitch];
  const int64_t b = blockIdx.z;
  const int c0 = blockIdx.y * kCB;
  const int64_t p0 = static_cast<int64_t>(blockIdx.x) * kPB;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 pixels x 8 channel rows per pass
  unsigned short v[kCB / 8];
#pragma unroll
  for (int r = 0; r < kCB / 8; r++) {
    const int c = c0 + ty + 8 * r;
    const int64_t p = p0 + tx;
    v[r] = 0;
    if (c < C && p < HW) {
      const int64_t idx = (b * C + c) * HW + p;
      v[r] = x_bf16 ? __ldg(reinterpret_cast<const unsigned short*>(x) + idx)
                    : __bfloat16_as_ushort(__float2bfloat16_rn(__ldg(reinterpret_cast<const float*>(x) + idx)));
    }
  }
#pragma unroll
  for (int r = 0; r < kCB / 8; r++) tile[ty + 8 * r][tx] = v[r];
  __syncthreads();
  const int piece = threadIdx.x & 7, pix = threadIdx.x >> 3;   // 8 pieces of 8 channels x 32 pixels
  const int64_t p = p0 + pix;
  const int c = c0 + piece * 8;
  if (p < HW && c < Cp) {                                      // Cp is a multiple of 8: whole pieces
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; e++)
      o[e] = tile[piece * 8 + 2 * e][pix] | (static_cast<uint32_t>(tile[piece * 8 + 2 * e + 1][pix]) << 16);
    *reinterpret_cast<uint4*>(out + (b * HW + p) * Cp + c) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

}  // namespace

cudaError_t launch_nchw_to_nhwc_bf16(const void* x, int x_bf16, const ConvGeom& g, void* out, int Cp, cudaStream_t stream) {
  const int64_t HW = static_cast<int64_t>(g.H) * g.W;
  dim3 grid(static_cast<unsigned>((HW + kPB - 1) / kPB), static_cast<unsigned>((Cp + kCB - 1) / kCB), static_cast<unsigned>(g.B));
  nchw_to_nhwc_bf16_kernel<<<grid, 256, 0, stream>>>(x, x_bf16, g.C, HW, Cp, static_cast<unsigned short*>(out));
  return cudaGetLastError();
}

}  // namespace hbmm
