// Internal: launcher of the tensor-core scoring kernels and the small fixed-order combine kernels.
#pragma once
#include "common.cuh"

namespace relaxkv {

struct ScorePlan {
  int n_super[kMaxReqInline];   // query-row blocks (<= kScoreMaxRows resident rows each) per request
  int max_super;
  int units;                    // sum of n_super
  int n_splits;                 // key-range splits (grid.z)
};

ScorePlan plan_score(const relaxkv_shape* shape);

// lse[h, row] = natural-log sum over n_part partial (max, sum) pairs in log2 units (score.cu).
void launch_combine_lse(int H, int sum_q, int n_part, const float2* part, float* lse, cudaStream_t stream);

// Pass 1 (unless lse_given) + combine + pass 2: fills colpart[(g*max_super + super)*2 + wg][sum_t].
template <int D>
relaxkv_status launch_score_sm100(const relaxkv_shape* shape, ReqTable rt, const ScorePlan& plan, const void* q,
                                  const relaxkv_cache_view* cache, const float* lse_given, float* lse_ws,
                                  float2* part, float* colpart, cudaStream_t stream);

}  // namespace relaxkv
