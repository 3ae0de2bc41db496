// Tensor-core hybrid-attention kernel (placeholder translation unit until the kernel lands).
#include "k2_tc.cuh"

namespace delta {
bool tc_kernel_available(int) { return false; }
cudaError_t launch_hybrid_attn_tc(const Shape&, const Workspace&, const void*, const void*,
                                  const void*, void*, int, int, int, cudaStream_t) {
  return cudaErrorNotSupported;
}
}  // namespace delta
