// Instantiations of the tensor-core kernel: C = 128, block recursion.
#include "tc_kernel.cuh"

namespace tri_inv {
cudaError_t launch_tc_c128_br(const KParams& p, cudaStream_t stream, bool raw) {
  return raw ? launch_one<128, 128, false, true>(p, stream) : launch_one<128, 128, false, false>(p, stream);
}
}  // namespace tri_inv
