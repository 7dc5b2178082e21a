// Internal: launcher of the tensor-core scoring kernels and the small fixed-order combine kernels.
#pragma once
#include "common.cuh"

namespace relaxkv {

struct ScorePlan {
  int n_super[kMaxReqInline];   // query-row blocks (<= kScoreMaxRows resident rows each) per request
  int max_super;
  int units;                    // sum of n_super
};

ScorePlan plan_score(const relaxkv_shape* shape);

// lse[layer, h, row] = natural-log sum over n_part partial (max, sum) pairs in log2 units (score.cu).
void launch_combine_lse(int n_layers, int H, int sum_q, int n_part, const float2* part, float* lse, cudaStream_t stream);

// Scores n_layers (<= kScoreLayersPerLaunch) layers with ONE launch per pass: pass 1 for the layers without
// supplied log-normalisers + combine, then pass 2.  Fills colpart[layer][(g*max_super + super)*2 + wg][sum_t].
// All layers must share the requests' cache token offsets (rt.tok_off).
template <int D>
relaxkv_status launch_score_sm100(const relaxkv_shape* shape, ReqTable rt, const ScorePlan& plan, int n_layers,
                                  const void* const* q_layers, const relaxkv_cache_view* cache_layers,
                                  const float* const* lse_given, float* lse_ws, float2* part, float* colpart,
                                  cudaStream_t stream);

}  // namespace relaxkv
