// Tensor-core path of surgeon_weight_grad (tcgen05 / TMEM).  Not built yet: the entry point
// reports SURGEON_ERR_UNSUPPORTED for path 0 until the kernel lands.
#include "surgeon_internal.cuh"

namespace surgeon {
size_t weight_grad_tc_workspace(const surgeon_layer_desc&) { return 0; }
cudaError_t launch_weight_grad_tc(const surgeon_compressed&, const surgeon_layer_desc&,
                                  const float*, float*, int, void*, cudaStream_t) {
  return cudaErrorNotSupported;
}
}  // namespace surgeon
