// Tensor-core prefill (placeholder translation unit until the tcgen05 kernel lands).
#include "la_common.cuh"

namespace la {
cudaError_t launch_prefill_tc(la_ctx*, int, int, const void*, const void*, const void*, const float*, int,
                              const la_state&, void*, cudaStream_t, bool* handled) {
  *handled = false;
  return cudaSuccess;
}
}  // namespace la
