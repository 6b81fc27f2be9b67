// Instantiations of the tensor-core kernel: product series with fp16 operands (TRI_INV_OPERANDS_F16).
#include "tc_kernel.cuh"

namespace tri_inv {
cudaError_t launch_tc_series_f16(const KParams& p, int C, cudaStream_t stream, bool raw) {
  if (C == 64) return raw ? launch_one<64, 128, true, true, false, false, true>(p, stream) : launch_one<64, 128, true, false, false, false, true>(p, stream);
  return raw ? launch_one<128, 128, true, true, false, false, true>(p, stream) : launch_one<128, 128, true, false, false, false, true>(p, stream);
}
}  // namespace tri_inv
