// Internal: launcher of the mixed-context gather, shared by the attention entry points.
#pragma once
#include "common.cuh"

namespace relaxkv {

// Materialises rows [0, rows_to_cover) of the context (rows past the true total are zero-filled for
// kCtxPadRows rows, the rest left alone) into k_out / v_out [ctx_rows, H_kv, D].  fresh_row (may be NULL):
// per context row, the row of k_new/v_new that replaces it (-1: read the cache) - used by the explicit-list path
// instead of looking the entry up in r_rank; only its first fresh_map_rows entries are valid.  n_new_rows: rows of
// k_new / v_new (a fresh-row index past it is reported in the status word and the row zero-filled).
relaxkv_status launch_gather(const relaxkv_shape* shape, int mode, const relaxkv_cache_view* cache,
                             const void* k_new, const void* v_new, const int32_t* u_pos, const int32_t* u_cu,
                             const int32_t* r_rank, const int32_t* r_cu_layer, const int32_t* fresh_row,
                             long long fresh_map_rows, long long n_new_rows, long long rows_to_cover, void* k_out, void* v_out, long long ctx_rows, cudaStream_t stream);

}  // namespace relaxkv
