// Instantiations of the tensor-core kernel: C = 64, product series.
#include "tc_kernel.cuh"

namespace tri_inv {
cudaError_t launch_tc_c64_series(const KParams& p, cudaStream_t stream, bool raw) {
  return raw ? launch_one<64, 128, true, true>(p, stream) : launch_one<64, 128, true, false>(p, stream);
}
}  // namespace tri_inv
