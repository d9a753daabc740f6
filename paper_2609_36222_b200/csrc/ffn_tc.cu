#include "ffn_tc.cuh"

namespace base {
// Bring-up placeholder: routed to the CUDA-core kernels until the tcgen05 path lands.
cudaError_t launch_ffn_tc(const base_layer_shape& s, const base_layer_weights& w, const Workspace& ws, int T,
                          cudaStream_t st, int* launches) {
  (void)T;
  return launch_ffn_simple(s, w, ws, st, launches);
}
}  // namespace base
