// Tensor-core streaming FFN (tcgen05 + TMA) launcher.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace base {
// [rows, cols] row-major bf16 matrix as a tensor map {64 elements, rows, k-blocks} with 128-byte swizzle and a box
// of box_rows x box_kb k-blocks (cached by key). False if the driver refuses the encoding.
bool tc_map_rows_kblocks(const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_kb,
                          CUtensorMap* out);
int tc_sm_count();
// Gate/up units that the FFN kernel's CTAs take statically (CTA c takes unit c); the ticket counter starts behind them.
int ffn_tc_static_units(const base_layer_shape& s, int T, int budget, const Workspace& ws);
// ahead: two [E,d] bf16 matrices (or nullptr) that the kernel requests into the L2 for whoever runs next.
cudaError_t launch_ffn_tc(const base_layer_shape& s, const base_layer_weights& w, const void* hidden,
                          const Workspace& ws, int T, int budget, const void* const ahead[2], cudaStream_t st,
                          int* launches, int* n_split);
}
