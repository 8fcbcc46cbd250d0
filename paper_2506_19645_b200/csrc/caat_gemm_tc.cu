// Tensor-core GEMMs (placeholder translation unit; replaced by the tcgen05 kernels).
#include "caat_internal.h"

namespace caat {
bool tc_gemm_usable(const caat_ctx*, int) { return false; }
cudaError_t launch_tc_forward(const RowparShapes&, const void*, const void*, void*, void*, cudaStream_t) {
  return cudaErrorNotSupported;
}
cudaError_t launch_tc_dgrad(const RowparShapes&, const void*, const void*, const void*, void*, cudaStream_t) {
  return cudaErrorNotSupported;
}
cudaError_t launch_tc_wgrad(const RowparShapes&, const void*, const void*, const void*, float*, void*, size_t,
                            cudaStream_t) {
  return cudaErrorNotSupported;
}
size_t tc_wgrad_splitk_bytes(const RowparShapes&) { return 0; }
}  // namespace caat
