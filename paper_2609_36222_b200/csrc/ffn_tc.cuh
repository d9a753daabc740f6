// Tensor-core streaming FFN (tcgen05 + TMA) launcher.
#pragma once
#include "common.cuh"

namespace base {
cudaError_t launch_ffn_tc(const base_layer_shape& s, const base_layer_weights& w, const void* hidden,
                          const Workspace& ws, int T, int budget, cudaStream_t st, int* launches, int* n_split);
}
