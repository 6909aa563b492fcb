// Programmatic dependent launch: a kernel launched with launch_pdl may be scheduled while the kernel before
// it in the stream is still running (as soon as every CTA of that kernel has executed
// pdl_launch_dependents or exited), so its launch latency and per-CTA set-up (barrier initialisation,
// tensor-memory allocation, address tables) overlap the predecessor's tail.  It must execute pdl_wait in
// every thread before it touches global memory: the wait returns when the preceding kernel has completed
// and its writes are visible -- which also keeps the ordering transitive along a chain of such kernels.
#pragma once
#include <cuda_runtime.h>
#include <utility>

namespace hbmm {

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(std::forward<Args>(args))...);
}

}  // namespace hbmm
