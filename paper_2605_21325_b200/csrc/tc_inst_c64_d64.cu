// Instantiations of the tensor-core kernel for head dimension 64 (bf16, C = 64, block recursion and mixed recursion):
// the build-only kernel, and one kernel with the calls' paths chosen at run time for the fused call and tri_inv_wy.
#include "tc_kernel.cuh"

namespace tri_inv {
cudaError_t launch_tc_c64_d64(const KParams& p, cudaStream_t stream) {
  if (!(p.ops & (kDoWY | kLoadA))) return launch_one<64, 64, false, false, true>(p, stream);   // tri_inv_build
  return launch_one<64, 64, false, false>(p, stream);
}
}  // namespace tri_inv
