// Convolution entry point for callers that must not allocate device memory.
//
// hbmm_conv_im2col needs a scratch buffer for the packed activation operand and expects the
// caller to provide it.  Some callers cannot: code that runs inside another runtime's memory
// arena where every byte of the device is already handed out, plugins that only receive tensor
// pointers and a stream, or latency-critical loops in which a cudaMalloc (which synchronises the
// device) is forbidden.  For them the scratch lives in a fixed array inside this library's device
// image, so the call itself allocates nothing.
#include <mutex>
#include <cuda_runtime.h>
#include "../../include/hbmm.h"

namespace {

// Every GPU that loads the library holds this array until the process exits.
constexpr size_t kStaticScratchBytes = HBMM_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_conv_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_conv_scratch on each device
bool g_scratch_ready[kMaxDevices] = {};

// The array's name is only a host-side handle; the device address has to be asked for, once per
// device and with that device current.
hbmm_status scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return HBMM_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_ready[dev]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_conv_scratch);
    if (e != cudaSuccess || p == nullptr) return HBMM_ERR_CUDA;
    g_scratch_addr[dev] = p;
    g_scratch_ready[dev] = true;
  }
  *out = g_scratch_addr[dev];
  return HBMM_OK;
}

}  // namespace

extern "C" hbmm_status hbmm_conv_im2col_static(const void* x, int32_t x_dtype, const hbmm_conv_geom* g,
                                               int32_t beta_a, int32_t a_scale_dtype, const hbmm_operand* W,
                                               float* C_out, int64_t ldc, void* stream) {
  size_t need = 0;
  hbmm_status st = hbmm_conv_workspace_bytes(g, beta_a, a_scale_dtype, W, &need);
  if (st != HBMM_OK) return st;
  if (need > kStaticScratchBytes) return HBMM_ERR_WORKSPACE;   // problem too large for the fixed scratch
  void* scratch = nullptr;
  if ((st = scratch_for_current_device(&scratch)) != HBMM_OK) return st;
  // The front end overwrites every word and scale (padding included) of the region it uses
  // before the contraction reads it, so nothing left by an earlier call is ever read.
  return hbmm_conv_im2col(x, x_dtype, g, beta_a, a_scale_dtype, W, C_out, ldc, scratch, need, stream);
}
