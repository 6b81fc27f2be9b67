// Instantiations of the tensor-core kernel: C = 64, block recursion (fused call, tri_inv_wy, raw front end).
#define TRI_INV_DEV_DEFINE_EXPORTS  // only read by the development header, which the default build never includes
#include "tc_kernel.cuh"

namespace tri_inv {
cudaError_t launch_tc_c64_br(const KParams& p, cudaStream_t stream, bool raw) {
  if (raw) return launch_one<64, 128, false, true>(p, stream);
  // the common calls get kernels of their own, without the code of the paths they do not take
  if (p.ops & kLoadA) return launch_one<64, 128, false, false, false, false, false, 2>(p, stream);
  if (p.method & TRI_INV_LEAF_SERIES) return launch_one<64, 128, false, false, false, false, false, 1>(p, stream);
  return launch_one<64, 128, false, false, false, false, false, 0>(p, stream);
}
}  // namespace tri_inv
