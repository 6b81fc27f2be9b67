// Tensor-core path (placeholder until the kernel lands): reports "not handled".
#include "common.cuh"

namespace tri_inv {
cudaError_t launch_tc(const KParams&, int, cudaStream_t, bool* handled) {
  *handled = false;
  return cudaSuccess;
}
}  // namespace tri_inv
