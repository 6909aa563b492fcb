// NCHW (fp32 or bf16) -> NHWC bf16 copy of a convolution input, channels padded with zeros to a
// multiple of 8 (16-byte pixels).  The HBWN convolution reads its activation tiles from this copy
// with im2col-mode tensor copies, which want the channel as the contiguous dimension.
#include "kernels.h"
#include "nhwc.cuh"

namespace hbmm {
namespace {

template <int PB>
__global__ void __launch_bounds__(256)
nchw_to_nhwc_bf16_kernel(const void* __restrict__ x, int x_bf16, int C, int64_t HW, int Cp, unsigned short* __restrict__ out) {
  __shared__ unsigned short tile[kNhwcCB][nhwc_pitch(PB)];
  nchw_to_nhwc_block<PB>(x, x_bf16, C, HW, Cp, out, blockIdx.z, blockIdx.y, blockIdx.x, tile);
}

}  // namespace

cudaError_t launch_nchw_to_nhwc_bf16(const void* x, int x_bf16, const ConvGeom& g, void* out, int Cp, cudaStream_t stream) {
  const int64_t HW = static_cast<int64_t>(g.H) * g.W;
  const int pb = nhwc_pixels_per_block(HW);
  dim3 grid(static_cast<unsigned>((HW + pb - 1) / pb), static_cast<unsigned>((Cp + kNhwcCB - 1) / kNhwcCB),
            static_cast<unsigned>(g.B));
  if (pb == kNhwcPBLarge)
    nchw_to_nhwc_bf16_kernel<kNhwcPBLarge><<<grid, 256, 0, stream>>>(x, x_bf16, g.C, HW, Cp, static_cast<unsigned short*>(out));
  else
    nchw_to_nhwc_bf16_kernel<kNhwcPBSmall><<<grid, 256, 0, stream>>>(x, x_bf16, g.C, HW, Cp, static_cast<unsigned short*>(out));
  return cudaGetLastError();
}

}  // namespace hbmm
