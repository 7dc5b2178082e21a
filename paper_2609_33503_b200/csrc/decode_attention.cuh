// Internal: the streaming kernel for cache-only attention calls with at most one target per request (a decode step);
// relaxkv_cache_attention routes there.
#pragma once
#include "attention_common.cuh"

namespace relaxkv {

// plan: request table with bound_a = the host bounds (each <= 1), the cache pointers and strides, the split workspace.
relaxkv_status launch_decode_attention(const relaxkv_shape* shape, const AttnPlan& plan, const void* q, const int32_t* tgt_pos,
                                       const int32_t* tgt_cu, int64_t n_target_rows, void* out, float* lse_out,
                                       cudaStream_t stream);

// Merges the normalised partial results [n_splits][n_target_rows][H][D] and their log-sum-exp by a fixed-order sum
// (attention_sm100.cu).  rows_bound: sum of the host bounds on the targets.
relaxkv_status launch_combine_splits(const float* part_o, const float* part_lse, int n_splits, long long n_target_rows, int H,
                                     int D, const int32_t* r_cu, int n_req, long long rows_bound, void* out, float* lse_out,
                                     cudaStream_t stream);

}  // namespace relaxkv
