// Internal: launcher of the segmented top-k / MinMax kernel.
#pragma once
#include "common.cuh"

namespace relaxkv {

// raw, norm (may be NULL): [n_layers, sum_b T_c];  anchors: [n_layers, sum_b k_b].  rt.k / rt.k_cu filled.
relaxkv_status launch_select(const ReqTable& rt, int n_layers, const float* raw, float* norm, int* anchors,
                             cudaStream_t stream);

}  // namespace relaxkv
