// Per-layer top-k anchors by radix select, plus MinMax normalisation (Section 3.2; Appendix A.1).
// One block per (layer, request) segment: min/max, four 8-bit radix passes that find the k-th
// largest score exactly, then an index-ordered compaction so that equal scores go to the lower
// position and the anchors come out ascending.  The segment (<= 256 KB) stays in L2 between passes.
#include "common.cuh"
#include "select.cuh"

namespace relaxkv {

constexpr int kSelThreads = 1024;

// Monotone map float -> uint32 (larger float, larger key).
__device__ __forceinline__ uint32_t order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ void block_scan2_sel(int a, int b, int& a_excl, int& b_excl) {
  __shared__ int wa[32], wb[32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int ia = a, ib = b;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int ta = __shfl_up_sync(0xffffffffu, ia, o), tb = __shfl_up_sync(0xffffffffu, ib, o);
    if (lane >= o) { ia += ta; ib += tb; }
  }
  if (lane == 31) { wa[warp] = ia; wb[warp] = ib; }
  __syncthreads();
  if (warp == 0) {
    const int va = wa[lane], vb = wb[lane];
    int sa = va, sb = vb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int ta = __shfl_up_sync(0xffffffffu, sa, o), tb = __shfl_up_sync(0xffffffffu, sb, o);
      if (lane >= o) { sa += ta; sb += tb; }
    }
    wa[lane] = sa - va; wb[lane] = sb - vb;
  }
  __syncthreads();
  a_excl = wa[warp] + ia - a;
  b_excl = wb[warp] + ib - b;
  __syncthreads();
}

__global__ void __launch_bounds__(kSelThreads)
select_topk_kernel(ReqTable rt, int n_layers, const float* __restrict__ raw, float* __restrict__ norm,
                   int* __restrict__ anchors, DeviceStatus* st) {
  const int B = rt.n_req;
  const int l = blockIdx.x / B, b = blockIdx.x % B;
  const int T = rt.ctx_len[b];
  const int k = rt.k[b];
  const long long sum_t = rt.ctx_cu[B];
  const float* x = raw + (long long)l * sum_t + rt.ctx_cu[b];
  int* out = anchors + (long long)l * rt.k_cu[B] + rt.k_cu[b];

  __shared__ int hist[256];
  __shared__ float red_lo[32], red_hi[32];
  __shared__ uint32_t s_prefix;
  __shared__ int s_krem;

  // ---- MinMax ------------------------------------------------------------------------
  if (norm != nullptr) {
    float lo = INFINITY, hi = -INFINITY;
    for (int i = threadIdx.x; i < T; i += kSelThreads) { const float v = x[i]; lo = fminf(lo, v); hi = fmaxf(hi, v); }
    lo = warp_reduce_min(lo); hi = warp_reduce_max(hi);
    if ((threadIdx.x & 31) == 0) { red_lo[threadIdx.x >> 5] = lo; red_hi[threadIdx.x >> 5] = hi; }
    __syncthreads();
    if (threadIdx.x < 32) {
      lo = warp_reduce_min(red_lo[threadIdx.x]); hi = warp_reduce_max(red_hi[threadIdx.x]);
      if (threadIdx.x == 0) { red_lo[0] = lo; red_hi[0] = hi; }
    }
    __syncthreads();
    lo = red_lo[0]; hi = red_hi[0];
    float* nb = norm + (long long)l * sum_t + rt.ctx_cu[b];
    const float range = hi - lo;
    for (int i = threadIdx.x; i < T; i += kSelThreads) nb[i] = (range > 0.f) ? (x[i] - lo) / range : 0.f;
  }

  // ---- radix select: key of the k-th largest --------------------------------------------
  if (threadIdx.x == 0) { s_prefix = 0u; s_krem = k; }
  uint32_t prefix = 0u, mask = 0u;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (threadIdx.x < 256) hist[threadIdx.x] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < T; i += kSelThreads) {
      const uint32_t key = order_key(x[i]);
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int krem = s_krem, d = 255;
      for (; d > 0; --d) {
        const int c = hist[d];
        if (c >= krem) break;
        krem -= c;
      }
      s_krem = krem;                       // still needed from bin d (>= 1)
      s_prefix = prefix | ((uint32_t)d << shift);
    }
    __syncthreads();
    prefix = s_prefix;
    mask |= (255u << shift);
  }
  const uint32_t tau = prefix;             // key of the k-th largest score
  const int need_eq = s_krem;              // how many elements equal to it are selected (lowest positions)

  // ---- ordered compaction ------------------------------------------------------------------
  const int per = (T + kSelThreads - 1) / kSelThreads;
  const int i0 = min(T, (int)threadIdx.x * per), i1 = min(T, i0 + per);
  int ngt = 0, neq = 0;
  for (int i = i0; i < i1; ++i) { const uint32_t key = order_key(x[i]); ngt += (key > tau); neq += (key == tau); }
  int egt, eeq;
  block_scan2_sel(ngt, neq, egt, eeq);
  for (int i = i0; i < i1; ++i) {
    const uint32_t key = order_key(x[i]);
    if (key > tau) {
      const int o = egt + min(eeq, need_eq);
      if (o < k) out[o] = i; else report(st, RELAXKV_ERR_BAD_INDEX, KID_SELECT, o, k);
      ++egt;
    } else if (key == tau) {
      if (eeq < need_eq) {
        const int o = egt + eeq;
        if (o < k) out[o] = i; else report(st, RELAXKV_ERR_BAD_INDEX, KID_SELECT, o, k);
      }
      ++eeq;
    }
  }
}

// g[i] = (1/L) * sum over layers (in layer order) of scores[l, i]   (Appendix B, global repair target sweep)
__global__ void mean_scores_kernel(int n_layers, long long sum_t, const float* __restrict__ scores, float* __restrict__ g) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= sum_t) return;
  float a = 0.f;
  for (int l = 0; l < n_layers; ++l) a += scores[(long long)l * sum_t + i];
  g[i] = a / (float)n_layers;
}

// scores[i] *= factor   (combining the per-shard mean scores of a head-sharded layout: mean over shards)
__global__ void scale_scores_kernel(long long n, float factor, float* __restrict__ scores) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) scores[i] *= factor;
}

relaxkv_status launch_select(const ReqTable& rt, int n_layers, const float* raw, float* norm, int* anchors,
                             cudaStream_t stream) {
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  select_topk_kernel<<<(unsigned)(n_layers * rt.n_req), kSelThreads, 0, stream>>>(rt, n_layers, raw, norm, anchors, st);
  return launch_ok();
}

}  // namespace relaxkv

using namespace relaxkv;

extern "C" relaxkv_status relaxkv_select_topk(const relaxkv_shape* shape, int32_t n_layers, const int32_t* h_k,
                                              const float* raw_scores, float* norm_scores_out, int32_t* anchors_out,
                                              relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_select_topk");
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if (n_layers < 1 || !h_k || !raw_scores || !anchors_out) return RELAXKV_ERR_INVALID_ARG;
  for (int b = 0; b < shape->n_req; ++b)
    if (h_k[b] < 1 || h_k[b] > shape->h_ctx_len[b]) return RELAXKV_ERR_INVALID_ARG;
  ReqTable rt;
  fill_req_table(rt, shape, nullptr, h_k);
  return launch_select(rt, n_layers, raw_scores, norm_scores_out, anchors_out, static_cast<cudaStream_t>(stream));
}

extern "C" relaxkv_status relaxkv_mean_scores(const relaxkv_shape* shape, int32_t n_layers, const float* scores,
                                              float* mean_out, relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_mean_scores");
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if (n_layers < 1 || !scores || !mean_out) return RELAXKV_ERR_INVALID_ARG;
  long long sum_t = 0;
  for (int b = 0; b < shape->n_req; ++b) sum_t += shape->h_ctx_len[b];
  mean_scores_kernel<<<(unsigned)((sum_t + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(n_layers, sum_t, scores, mean_out);
  return launch_ok();
}

extern "C" relaxkv_status relaxkv_scale_scores(const relaxkv_shape* shape, int32_t n_layers, float* scores, float factor,
                                               relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_scale_scores");
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if (n_layers < 1 || !scores || !(factor > 0.f)) return RELAXKV_ERR_INVALID_ARG;
  long long n = 0;
  for (int b = 0; b < shape->n_req; ++b) n += shape->h_ctx_len[b];
  n *= n_layers;
  scale_scores_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(n, factor, scores);
  return launch_ok();
}
