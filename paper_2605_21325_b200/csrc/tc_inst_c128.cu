// Instantiations of the tensor-core kernel: C = 128, block recursion.
#include "tc_kernel.cuh"

namespace tri_inv {
cudaError_t launch_tc_c128_br(const KParams& p, cudaStream_t stream, bool raw) {
  if (raw) return launch_one<128, 128, false, true>(p, stream);
  // the common calls get kernels of their own, without the code of the paths they do not take
  if (p.ops & kLoadA) return launch_one<128, 128, false, false, false, false, false, 2>(p, stream);
  if (p.method & TRI_INV_LEAF_SERIES) return launch_one<128, 128, false, false, false, false, false, 1>(p, stream);
  return launch_one<128, 128, false, false, false, false, false, 0>(p, stream);
}
}  // namespace tri_inv
