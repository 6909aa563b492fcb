// Host-side access to the driver's tensor-map encoders.  They are host-only routines that fill a
// 128-byte descriptor; they are looked up through the runtime so that the library does not link
// against the driver.  Each function returns nullptr when the driver does not offer the routine.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

namespace hbmm {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
using EncodeIm2colFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline void* driver_entry_point(const char* name) {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
  if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) p = nullptr;
  return p;
}
inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(driver_entry_point("cuTensorMapEncodeTiled"));
  return fn;
}
inline EncodeIm2colFn encode_im2col_fn() {
  static EncodeIm2colFn fn = reinterpret_cast<EncodeIm2colFn>(driver_entry_point("cuTensorMapEncodeIm2col"));
  return fn;
}

}  // namespace hbmm
