// Instantiations of the tensor-core kernel: block recursion followed by one step of iterative refinement (Alg. 6).
#include "tc_kernel.cuh"

namespace tri_inv {
cudaError_t launch_tc_refine(const KParams& p, int C, cudaStream_t stream, bool raw) {
  if (C == 64) return raw ? launch_one<64, 128, false, true, false, true>(p, stream) : launch_one<64, 128, false, false, false, true>(p, stream);
  return raw ? launch_one<128, 128, false, true, false, true>(p, stream) : launch_one<128, 128, false, false, false, true>(p, stream);
}
}  // namespace tri_inv
