// Instantiation of the tensor-core kernel: C = 64, build only (tri_inv_build).
#include "tc_kernel.cuh"

namespace tri_inv {
cudaError_t launch_tc_c64_build(const KParams& p, cudaStream_t stream) { return launch_one<64, 128, false, false, true>(p, stream); }
}  // namespace tri_inv
