// Query-attention scoring (Section 3.2, score equation): two passes over the cached keys.
//   pass 1: log-normaliser of every query row's softmax over the context (skipped if supplied)
//   pass 2: column sums of exp(s - lse) over all query rows of a KV head, then the mean over heads
// followed by the segmented top-k (select.cu).  The two passes run on the tensor cores
// (score_sm100.cu); this file holds the entry point and the small kernels that combine their partial
// results in a fixed order, so results are bit-reproducible from run to run.
#include "common.cuh"
#include "score_sm100.cuh"
#include "select.cuh"
#include <algorithm>

namespace relaxkv {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// lse[layer, h, row] = ln sum over the partial (max, sum) pairs (log2 units in, natural log out).
// One warp per row: the lanes walk the partials (fixed lane -> partial assignment, fixed shuffle tree, so
// the result does not depend on scheduling).  part is [layer][n_part][H*sum_q].  Rows of layers whose
// log-normalisers were supplied have only empty partials and are never read afterwards.
__global__ void combine_lse_kernel(long long n_rows_total, long long n_rows, int n_part, const float2* __restrict__ part,
                                   float* __restrict__ lse) {
  const int lane = threadIdx.x & 31;
  const long long gidx = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (gidx >= n_rows_total) return;
  const long long layer = gidx / n_rows, idx = gidx - layer * n_rows;
  const float2* pl = part + layer * n_part * n_rows;
  float M = -INFINITY;
  for (int s = lane; s < n_part; s += 32) {
    const float2 p = pl[(long long)s * n_rows + idx];
    if (p.y > 0.f) M = fmaxf(M, p.x);
  }
  M = warp_reduce_max(M);
  float z = 0.f;
  for (int s = lane; s < n_part; s += 32) {
    const float2 p = pl[(long long)s * n_rows + idx];
    if (p.y > 0.f) z += p.y * exp2f(p.x - M);
  }
  z = warp_reduce_sum(z);
  if (lane == 0) lse[gidx] = (M + log2f(z)) * kLn2;
}

void launch_combine_lse(int n_layers, int H, int sum_q, int n_part, const float2* part, float* lse, cudaStream_t stream) {
  const long long n_rows = (long long)H * sum_q, total = n_rows * n_layers;
  combine_lse_kernel<<<(unsigned)((total * 32 + 255) / 256), 256, 0, stream>>>(total, n_rows, n_part, part, lse);
}

// raw[layer, i] = (sum of the partial column sums in a fixed order: KV head, query-row block, warpgroup) / (H * Q_b)
// rt.tile_cu = prefix of the query-row blocks per request; colpart is [layer][2*Hkv*max_super][sum_t].
__global__ void finalize_raw_kernel(ReqTable rt, int n_layers, int H, int Hkv, int max_super,
                                    const float* __restrict__ colpart, float* __restrict__ raw) {
  const long long sum_t = rt.ctx_cu[rt.n_req];
  const long long gi = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gi >= sum_t * n_layers) return;
  const long long layer = gi / sum_t, i = gi - layer * sum_t;
  int b = 0;
  while (b + 1 < rt.n_req && i >= rt.ctx_cu[b + 1]) ++b;
  const int n_super = rt.tile_cu[b + 1] - rt.tile_cu[b];
  const float* cp = colpart + layer * (2 * Hkv * max_super) * sum_t;
  float s = 0.f;
  for (int g = 0; g < Hkv; ++g)
    for (int sp = 0; sp < n_super; ++sp)
      for (int w = 0; w < 2; ++w) s += cp[(long long)((g * max_super + sp) * 2 + w) * sum_t + i];
  raw[gi] = s / ((float)H * (float)rt.q_len[b]);
}

template <int D>
static relaxkv_status score_layers(const relaxkv_shape* shape, ReqTable rt, const ScorePlan& plan, int n_layers,
                                   const void* const* q_layers, const relaxkv_cache_view* cache_layers,
                                   const float* const* lse_given, float* raw, char* workspace, const WsLayout& ws,
                                   cudaStream_t stream) {
  const int B = shape->n_req, H = shape->n_q_heads, Hkv = shape->n_kv_heads;
  float* lse_ws = reinterpret_cast<float*>(workspace + ws.lse);
  float2* part = reinterpret_cast<float2*>(workspace + ws.part);
  float* colpart = reinterpret_cast<float*>(workspace + ws.colpart);
  relaxkv_status rc = launch_score_sm100<D>(shape, rt, plan, n_layers, q_layers, cache_layers, lse_given, lse_ws, part,
                                            colpart, stream);
  if (rc != RELAXKV_OK) return rc;
  for (int b = 0; b < B; ++b) rt.tile_cu[b + 1] = rt.tile_cu[b] + plan.n_super[b];
  const long long total = rt.ctx_cu[B] * n_layers;
  finalize_raw_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(rt, n_layers, H, Hkv, plan.max_super, colpart, raw);
  return launch_ok();
}

// Positions of the query's own tokens (they follow the context: T_c, T_c + 1, ...) and their offsets, as the target
// lists of the cache-only attention call.
__global__ void query_positions_kernel(ReqTable rt, int* __restrict__ tgt_pos, int* __restrict__ tgt_cu) {
  const int B = rt.n_req;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i <= B) tgt_cu[i] = rt.q_cu[i];
  if (i < rt.q_cu[B]) {
    const int b = find_segment(rt.q_cu, B, i);
    tgt_pos[i] = rt.ctx_len[b] + (i - rt.q_cu[b]);
  }
}

}  // namespace relaxkv

using namespace relaxkv;

extern "C" relaxkv_status relaxkv_score_select(
    const relaxkv_shape* shape, int32_t n_layers,
    const void* const* q_layers, const relaxkv_cache_view* cache_layers,
    const float* const* row_lse_layers, const int32_t* h_k,
    float* raw_scores_out, float* norm_scores_out, int32_t* anchors_out,
    void* workspace, size_t workspace_bytes, relaxkv_stream stream_) {
  RELAXKV_RANGE("relaxkv_score_select");
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if (n_layers < 1 || !q_layers || !cache_layers || !h_k || !raw_scores_out || !workspace || !shape->h_q_len)
    return RELAXKV_ERR_INVALID_ARG;
  for (int b = 0; b < shape->n_req; ++b) {
    if (shape->h_q_len[b] < 1) return RELAXKV_ERR_INVALID_ARG;
    if (h_k[b] < 1 || h_k[b] > shape->h_ctx_len[b]) return RELAXKV_ERR_INVALID_ARG;
  }
  for (int l = 0; l < n_layers; ++l) {
    if (!q_layers[l] || !aligned16(q_layers[l])) return RELAXKV_ERR_INVALID_ARG;
    if ((rc = check_cache(shape, &cache_layers[l], false)) != RELAXKV_OK) return rc;
  }
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return RELAXKV_ERR_INVALID_ARG;
  const WsLayout ws = ws_layout(shape, n_layers);
  if (workspace_bytes < ws.total) return RELAXKV_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  long long sum_t = 0;
  for (int b = 0; b < shape->n_req; ++b) sum_t += shape->h_ctx_len[b];

  const ScorePlan plan = plan_score(shape);
  // Layers are scored in groups: one launch per pass covers up to kScoreLayersPerLaunch consecutive layers whose
  // cache views place the requests at the same token offsets (the usual case: all of them).
  for (int l0 = 0; l0 < n_layers;) {
    int l1 = l0 + 1;
    while (l1 < n_layers && l1 - l0 < kScoreLayersPerLaunch) {
      bool same = true;
      for (int b = 0; b < shape->n_req; ++b)
        same = same && cache_layers[l1].h_req_token_offset[b] == cache_layers[l0].h_req_token_offset[b];
      if (!same) break;
      ++l1;
    }
    ReqTable rt;
    fill_req_table(rt, shape, &cache_layers[l0], h_k);
    const float* const* lse = row_lse_layers ? row_lse_layers + l0 : nullptr;
    float* raw = raw_scores_out + (long long)l0 * sum_t;
    if (shape->head_dim == 128)
      rc = score_layers<128>(shape, rt, plan, l1 - l0, q_layers + l0, cache_layers + l0, lse, raw, static_cast<char*>(workspace), ws, stream);
    else
      rc = score_layers<64>(shape, rt, plan, l1 - l0, q_layers + l0, cache_layers + l0, lse, raw, static_cast<char*>(workspace), ws, stream);
    if (rc != RELAXKV_OK) return rc;
    l0 = l1;
  }
  if (!anchors_out) return RELAXKV_OK;      // scoring only: the caller reduces the scores first (head-sharded serving)
  ReqTable rt;
  fill_req_table(rt, shape, nullptr, h_k);
  return launch_select(rt, n_layers, raw_scores_out, norm_scores_out, anchors_out, stream);
}

// The query's own causal attention over [context, query] with the context scores taken from the same pass: the
// attention call leaves every row's log-normaliser, the column-sum pass of the scoring kernel then reads the context
// keys once more with those normalisers.  The statistics pass of relaxkv_score_select never runs.
extern "C" relaxkv_status relaxkv_query_prefill_attention(
    const relaxkv_shape* shape, const relaxkv_cache_view* cache, const void* q, void* out, float* lse_out,
    float* raw_scores_out, void* workspace, size_t workspace_bytes, relaxkv_stream stream_) {
  RELAXKV_RANGE("relaxkv_query_prefill_attention");
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if ((rc = check_cache(shape, cache, true)) != RELAXKV_OK) return rc;
  if (!q || !out || !lse_out || !workspace || !shape->h_q_len || !aligned16(q) || !aligned16(out))
    return RELAXKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return RELAXKV_ERR_INVALID_ARG;
  const int B = shape->n_req;
  int32_t ext_len[kMaxReqInline], q_len[kMaxReqInline];
  long long sum_q = 0;
  for (int b = 0; b < B; ++b) {
    if (shape->h_q_len[b] < 1) return RELAXKV_ERR_INVALID_ARG;
    const long long e = (long long)shape->h_ctx_len[b] + shape->h_q_len[b];
    if (e > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
    ext_len[b] = (int32_t)e;
    q_len[b] = shape->h_q_len[b];
    sum_q += q_len[b];
  }
  if (sum_q > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  relaxkv_shape ext = *shape;                       // the same batch with the query's tokens counted into the cache rows
  ext.h_ctx_len = ext_len;
  const WsLayout ws = ws_layout(&ext, 1);
  if (workspace_bytes < ws.total) return RELAXKV_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  char* base = static_cast<char*>(workspace);
  int* tgt_pos = reinterpret_cast<int*>(base + ws.list_limit);        // regions the cache-only attention does not use
  int* tgt_cu = reinterpret_cast<int*>(base + ws.list_fresh);
  ReqTable rt;
  fill_req_table(rt, shape, cache, nullptr);
  const long long n = std::max<long long>(sum_q, B + 1);
  query_positions_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(rt, tgt_pos, tgt_cu);
  if ((rc = launch_ok()) != RELAXKV_OK) return rc;
  rc = relaxkv_cache_attention(&ext, cache, q, tgt_pos, tgt_cu, sum_q, q_len, out, lse_out, workspace, workspace_bytes, stream_);
  if (rc != RELAXKV_OK || !raw_scores_out) return rc;
  // column sums over the CONTEXT keys with the rows' normalisers from the attention above
  const ScorePlan plan = plan_score(shape);
  const WsLayout ws_sc = ws_layout(shape, 1);
  if (workspace_bytes < ws_sc.total) return RELAXKV_ERR_WORKSPACE_TOO_SMALL;
  const void* q_arr[1] = {q};
  const float* lse_arr[1] = {lse_out};
  if (shape->head_dim == 128)
    return score_layers<128>(shape, rt, plan, 1, q_arr, cache, lse_arr, raw_scores_out, base, ws_sc, stream);
  return score_layers<64>(shape, rt, plan, 1, q_arr, cache, lse_arr, raw_scores_out, base, ws_sc, stream);
}
