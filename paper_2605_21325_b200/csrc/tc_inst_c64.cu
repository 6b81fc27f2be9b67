// Instantiations of the tensor-core kernel: C = 64, block recursion (fused call, tri_inv_wy, raw front end).
#define TRI_INV_DEV_DEFINE_EXPORTS  // only read by the development header, which the default build never includes
#include "tc_kernel.cuh"

namespace tri_inv {
cudaError_t launch_tc_c64_br(const KParams& p, cudaStream_t stream, bool raw) {
  return raw ? launch_one<64, 128, false, true>(p, stream) : launch_one<64, 128, false, false>(p, stream);
}
}  // namespace tri_inv
