// NCHW (fp32 or bf16) -> NHWC bf16 copy of a convolution input, channels padded with zeros to a
// multiple of 8 (16-byte pixels).  The HBWN convolution reads its activation tiles from this copy
// with im2col-mode tensor copies, which want the channel as the contiguous dimension.
#include <cuda_bf16.h>
#include "kernels.h"

namespace hbmm {
namespace {

// One block transposes a 32-channel x 32-pixel patch of one image: reads run along the pixels
// (contiguous in NCHW), writes along the channels (contiguous in NHWC).
__global__ void __launch_bounds__(256)
nchw_to_nhwc_bf16_kernel(const void* __restrict__ x, int x_bf16, int C, int64_t HW, int Cp,
                         unsigned short* __restrict__ out) {
  __shared__ unsigned short tile[32][33];
  const int64_t b = blockIdx.z;
  const int c0 = blockIdx.y * 32;
  const int64_t p0 = static_cast<int64_t>(blockIdx.x) * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
#pragma unroll
  for (int r = 0; r < 4; r++) {
    const int c = c0 + ty + 8 * r;
    const int64_t p = p0 + tx;
    unsigned short v = 0;
    if (c < C && p < HW) {
      const int64_t idx = (b * C + c) * HW + p;
      v = x_bf16 ? __ldg(reinterpret_cast<const unsigned short*>(x) + idx)
                 : __bfloat16_as_ushort(__float2bfloat16_rn(__ldg(reinterpret_cast<const float*>(x) + idx)));
    }
    tile[ty + 8 * r][tx] = v;
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < 4; r++) {
    const int64_t p = p0 + ty + 8 * r;
    const int c = c0 + tx;
    if (p < HW && c < Cp) out[(b * HW + p) * Cp + c] = tile[tx][ty + 8 * r];
  }
}

}  // namespace

cudaError_t launch_nchw_to_nhwc_bf16(const void* x, int x_bf16, const ConvGeom& g, void* out, int Cp, cudaStream_t stream) {
  const int64_t HW = static_cast<int64_t>(g.H) * g.W;
  dim3 grid(static_cast<unsigned>((HW + 31) / 32), static_cast<unsigned>((Cp + 31) / 32), static_cast<unsigned>(g.B));
  nchw_to_nhwc_bf16_kernel<<<grid, 256, 0, stream>>>(x, x_bf16, g.C, HW, Cp, static_cast<unsigned short*>(out));
  return cudaGetLastError();
}

}  // namespace hbmm
