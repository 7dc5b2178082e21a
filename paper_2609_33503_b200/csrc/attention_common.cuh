// Internal: argument checks and the gather step shared by the two attention entry points.
#pragma once
#include "common.cuh"
#include "kv_move.cuh"

namespace relaxkv {

struct AttnPlan {
  ReqTable rt;            // bound_a = max targets, bound_b = max ctx rows (mode-adjusted)
  uint16_t* kctx;         // materialised context  [ctx_rows, H_kv, D]
  uint16_t* vctx;
  long long ctx_rows;     // rows the two buffers hold (tensor-map extent)
  long long sum_targets;  // sum of the host bounds on |R_{l,b}|
  float* split_o;         // workspace for a context split across blocks: [kSplitRowsCap, H, D] and [kSplitRowsCap, H]
  float* split_lse;
  // what the attention kernel's K/V tensor maps cover: the materialised context, or the cache itself
  const void* k_base; const void* v_base;
  unsigned long long kv_token_stride_bytes, kv_head_stride_bytes;
  int dense_ctx;          // 1: context = the cache's own rows (request b starts at rt.tok_off[b]), limits are positions
};

// Validates the arguments of an attention call and enqueues the gather of the mixed context into
// the workspace.  On success `plan` describes what the attention kernel reads.
inline relaxkv_status prepare_attention(
    const relaxkv_shape* shape, relaxkv_ctx_mode mode, const relaxkv_cache_view* cache,
    const void* q_new, const void* k_new, const void* v_new,
    const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank, const int32_t* r_cu_layer,
    int64_t n_target_rows, const int32_t* h_max_targets, const int32_t* h_max_ctx,
    void* out, void* workspace, size_t workspace_bytes, cudaStream_t stream, AttnPlan& plan,
    const int32_t* fresh_row = nullptr) {
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if ((rc = check_cache(shape, cache, true)) != RELAXKV_OK) return rc;
  if (mode != RELAXKV_CTX_UNION && mode != RELAXKV_CTX_FULL_PREFIX) return RELAXKV_ERR_INVALID_ARG;
  if (!q_new || !out || !u_pos || !u_cu || !r_rank || !r_cu_layer || !h_max_targets || !h_max_ctx || !workspace)
    return RELAXKV_ERR_INVALID_ARG;
  if ((k_new == nullptr) != (v_new == nullptr)) return RELAXKV_ERR_INVALID_ARG;
  if (!aligned16(q_new) || !aligned16(out) || (k_new && (!aligned16(k_new) || !aligned16(v_new))))
    return RELAXKV_ERR_INVALID_ARG;
  if (n_target_rows < 1) return RELAXKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return RELAXKV_ERR_INVALID_ARG;
  const WsLayout ws = ws_layout(shape, 1);
  if (workspace_bytes < ws.total) return RELAXKV_ERR_WORKSPACE_TOO_SMALL;

  fill_req_table(plan.rt, shape, cache, nullptr);
  long long need_ctx = 0;
  plan.sum_targets = 0;
  for (int b = 0; b < shape->n_req; ++b) {
    if (h_max_targets[b] < 0 || h_max_ctx[b] < 0 || h_max_ctx[b] > shape->h_ctx_len[b] ||
        h_max_targets[b] > shape->h_ctx_len[b])
      return RELAXKV_ERR_INVALID_ARG;
    plan.rt.bound_a[b] = h_max_targets[b];
    plan.rt.bound_b[b] = (mode == RELAXKV_CTX_UNION) ? h_max_ctx[b] : shape->h_ctx_len[b];
    need_ctx += plan.rt.bound_b[b];
    plan.sum_targets += h_max_targets[b];
  }
  if (plan.sum_targets > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  char* base = static_cast<char*>(workspace);
  plan.kctx = reinterpret_cast<uint16_t*>(base + ws.kctx);
  plan.vctx = reinterpret_cast<uint16_t*>(base + ws.vctx);
  plan.ctx_rows = ws.ctx_rows_cap;
  plan.split_o = reinterpret_cast<float*>(base + ws.split_o);
  plan.split_lse = reinterpret_cast<float*>(base + ws.split_lse);
  plan.k_base = plan.kctx;
  plan.v_base = plan.vctx;
  plan.kv_head_stride_bytes = (unsigned long long)shape->head_dim * 2;
  plan.kv_token_stride_bytes = (unsigned long long)shape->n_kv_heads * shape->head_dim * 2;
  plan.dense_ctx = 0;
  return launch_gather(shape, mode, cache, k_new, v_new, u_pos, u_cu, r_rank, r_cu_layer, fresh_row,
                       fresh_row ? need_ctx : 0, n_target_rows, need_ctx + kCtxPadRows, plan.kctx, plan.vctx, plan.ctx_rows, stream);
}

}  // namespace relaxkv
