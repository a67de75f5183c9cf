// Tensor-core kernels (placeholder until the tcgen05 path lands): reports the
// path as unavailable so that AUTO selects the fp32 CUDA-core kernels.
#include "la_common.cuh"

namespace la {
bool tc_supported() { return false; }
cudaError_t launch_tc_walk(const OpArgs&, const DecayTable&, int, int, cudaStream_t) {
  return cudaErrorNotSupported;
}
cudaError_t launch_tc_prepass(const OpArgs&, const DecayTable&, int, cudaStream_t) {
  return cudaErrorNotSupported;
}
}  // namespace la
