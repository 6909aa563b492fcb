// Placeholder until the b1 tensor-instruction path is written.
#include "kernels.h"
namespace hbmm {
bool gemm_b1_supported(const PackedView&, const PackedView&) { return false; }
cudaError_t launch_gemm_b1(const PackedView&, const PackedView&, float*, int64_t, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t launch_partials_b1(const PackedView&, const PackedView&, int32_t*, cudaStream_t) { return cudaErrorNotSupported; }
}
