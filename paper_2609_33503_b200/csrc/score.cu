// Query-attention scoring (Section 3.2, score equation): two passes over the cached keys.
//   pass 1: log-normaliser of every query row's softmax over the context (skipped if supplied)
//   pass 2: column sums of exp(s - lse) over all query rows of a KV head, then the mean over heads
// followed by the segmented top-k (select.cu).  Reductions run in a fixed order: results are
// bit-reproducible from run to run.
#include "common.cuh"
#include "select.cuh"

namespace relaxkv {

constexpr int kScoreThreads = 128;   // one "owned" row per thread
constexpr int kScoreChunk = 32;      // broadcast rows staged in shared memory per step
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// A thread owns one row (pass 1: a query row; pass 2: a key) in registers and walks the rows of the
// other operand, staged in shared memory and read as broadcasts.
template <int D, bool PASS2>
__global__ void __launch_bounds__(kScoreThreads)
score_simt_kernel(ReqTable rt, int H, int Hkv, float scale_log2,
                  const uint16_t* __restrict__ q, const uint16_t* __restrict__ kc,
                  long long tok_stride, long long head_stride,
                  const float* __restrict__ lse, float2* __restrict__ part, float* __restrict__ colpart) {
  __shared__ __align__(16) float bs[kScoreChunk][D];
  __shared__ float bl[kScoreChunk];
  const int B = rt.n_req;
  const int G = H / Hkv;
  const int g = blockIdx.y;
  const int b = find_segment(rt.tile_cu, B, (int)blockIdx.x);
  const int tile = blockIdx.x - rt.tile_cu[b];
  const int T = rt.ctx_len[b];
  const int n_qrows = G * rt.q_len[b];
  const int sum_q = rt.q_cu[B];
  const long long sum_t = rt.ctx_cu[B];

  const int own = tile * kScoreThreads + threadIdx.x;
  const int n_own = PASS2 ? T : n_qrows;
  const bool valid = own < n_own;
  float a[D];
  {
    const uint16_t* src;
    if (PASS2) {
      src = kc + (rt.tok_off[b] + min(own, T - 1)) * tok_stride + g * head_stride;
    } else {
      const int r = min(own, n_qrows - 1);
      src = q + ((long long)(rt.q_cu[b] + r / G) * H + g * G + r % G) * D;
    }
#pragma unroll
    for (int d = 0; d < D; d += 8) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + d));
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        a[d + 2 * e] = __uint_as_float(w[e] << 16);
        a[d + 2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
      }
    }
  }

  // range of the other operand's rows walked by this block
  int o_begin = 0, o_end = 0;
  if (PASS2) {
    o_end = n_qrows;
  } else {
    const int len = (T + kScoreSplits - 1) / kScoreSplits;
    o_begin = min(T, (int)blockIdx.z * len);
    o_end = min(T, o_begin + len);
  }

  float m = -INFINITY, z = 0.f, acc = 0.f;
  for (int c0 = o_begin; c0 < o_end; c0 += kScoreChunk) {
    const int rows = min(kScoreChunk, o_end - c0);
    __syncthreads();
    for (int e = threadIdx.x; e < rows * (D / 8); e += kScoreThreads) {
      const int r = e / (D / 8), part8 = e % (D / 8);
      const int o = c0 + r;
      const uint16_t* src;
      if (PASS2) src = q + ((long long)(rt.q_cu[b] + o / G) * H + g * G + o % G) * D;
      else src = kc + (rt.tok_off[b] + o) * tok_stride + g * head_stride;
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + part8 * 8));
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      float* dst = &bs[r][part8 * 8];
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        dst[2 * x] = __uint_as_float(w[x] << 16);
        dst[2 * x + 1] = __uint_as_float(w[x] & 0xffff0000u);
      }
    }
    if (PASS2 && threadIdx.x < rows) {
      const int o = c0 + threadIdx.x;
      bl[threadIdx.x] = lse[(long long)(g * G + o % G) * sum_q + rt.q_cu[b] + o / G] * kLog2e;
    }
    __syncthreads();
    for (int r = 0; r < rows; ++r) {
      float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
      const float4* br = reinterpret_cast<const float4*>(&bs[r][0]);
#pragma unroll
      for (int d = 0; d < D / 4; ++d) {
        const float4 v = br[d];
        d0 = fmaf(a[4 * d], v.x, d0); d1 = fmaf(a[4 * d + 1], v.y, d1);
        d2 = fmaf(a[4 * d + 2], v.z, d2); d3 = fmaf(a[4 * d + 3], v.w, d3);
      }
      const float s2 = ((d0 + d1) + (d2 + d3)) * scale_log2;
      if (PASS2) {
        acc += exp2f(s2 - bl[r]);
      } else {
        if (s2 > m) { z *= exp2f(m - s2); m = s2; }
        z += exp2f(s2 - m);
      }
    }
  }
  if (!valid) return;
  if (PASS2) {
    colpart[(long long)g * sum_t + rt.ctx_cu[b] + own] = acc;
  } else {
    const int h = g * G + own % G;
    part[((long long)blockIdx.z * H + h) * sum_q + rt.q_cu[b] + own / G] = make_float2(m, z);
  }
}

// lse[h, row] = ln sum over the key splits (natural log).
__global__ void combine_lse_kernel(int H, int sum_q, const float2* __restrict__ part, float* __restrict__ lse) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= H * sum_q) return;
  float M = -INFINITY;
  for (int s = 0; s < kScoreSplits; ++s) {
    const float2 p = part[(long long)s * H * sum_q + idx];
    if (p.y > 0.f) M = fmaxf(M, p.x);
  }
  float z = 0.f;
  for (int s = 0; s < kScoreSplits; ++s) {
    const float2 p = part[(long long)s * H * sum_q + idx];
    if (p.y > 0.f) z += p.y * exp2f(p.x - M);
  }
  lse[idx] = (M + log2f(z)) * kLn2;
}

// raw[i] = (sum over KV heads, in head order) / (H * Q_b)
__global__ void finalize_raw_kernel(ReqTable rt, int H, int Hkv, const float* __restrict__ colpart,
                                    float* __restrict__ raw) {
  const long long sum_t = rt.ctx_cu[rt.n_req];
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= sum_t) return;
  int b = 0;
  while (b + 1 < rt.n_req && i >= rt.ctx_cu[b + 1]) ++b;
  float s = 0.f;
  for (int g = 0; g < Hkv; ++g) s += colpart[(long long)g * sum_t + i];
  raw[i] = s / ((float)H * (float)rt.q_len[b]);
}

template <int D>
static relaxkv_status score_layer(const relaxkv_shape* shape, ReqTable rt, const void* q,
                                  const relaxkv_cache_view* cache, const float* lse_given, float* raw,
                                  char* workspace, const WsLayout& ws, cudaStream_t stream) {
  const int B = shape->n_req, H = shape->n_q_heads, Hkv = shape->n_kv_heads, G = H / Hkv;
  const int sum_q = rt.q_cu[B];
  const float scale_log2 = shape->softmax_scale * kLog2e;
  float* lse_ws = reinterpret_cast<float*>(workspace + ws.lse);
  float2* part = reinterpret_cast<float2*>(workspace + ws.part);
  float* colpart = reinterpret_cast<float*>(workspace + ws.colpart);
  const uint16_t* qp = static_cast<const uint16_t*>(q);
  const uint16_t* kp = static_cast<const uint16_t*>(cache->k);
  const float* lse = lse_given;
  if (!lse) {
    for (int b = 0; b < B; ++b)
      rt.tile_cu[b + 1] = rt.tile_cu[b] + (G * rt.q_len[b] + kScoreThreads - 1) / kScoreThreads;
    dim3 grid1((unsigned)rt.tile_cu[B], (unsigned)Hkv, kScoreSplits);
    score_simt_kernel<D, false><<<grid1, kScoreThreads, 0, stream>>>(rt, H, Hkv, scale_log2, qp, kp,
        cache->token_stride, cache->head_stride, nullptr, part, nullptr);
    combine_lse_kernel<<<(H * sum_q + 255) / 256, 256, 0, stream>>>(H, sum_q, part, lse_ws);
    lse = lse_ws;
  }
  for (int b = 0; b < B; ++b)
    rt.tile_cu[b + 1] = rt.tile_cu[b] + (rt.ctx_len[b] + kScoreThreads - 1) / kScoreThreads;
  dim3 grid2((unsigned)rt.tile_cu[B], (unsigned)Hkv, 1);
  score_simt_kernel<D, true><<<grid2, kScoreThreads, 0, stream>>>(rt, H, Hkv, scale_log2, qp, kp,
      cache->token_stride, cache->head_stride, lse, nullptr, colpart);
  const long long sum_t = rt.ctx_cu[B];
  finalize_raw_kernel<<<(unsigned)((sum_t + 255) / 256), 256, 0, stream>>>(rt, H, Hkv, colpart, raw);
  return launch_ok();
}

}  // namespace relaxkv

using namespace relaxkv;

extern "C" relaxkv_status relaxkv_score_select(
    const relaxkv_shape* shape, int32_t n_layers,
    const void* const* q_layers, const relaxkv_cache_view* cache_layers,
    const float* const* row_lse_layers, const int32_t* h_k,
    float* raw_scores_out, float* norm_scores_out, int32_t* anchors_out,
    void* workspace, size_t workspace_bytes, relaxkv_stream stream_) {
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if (n_layers < 1 || !q_layers || !cache_layers || !h_k || !raw_scores_out || !anchors_out || !workspace ||
      !shape->h_q_len)
    return RELAXKV_ERR_INVALID_ARG;
  for (int b = 0; b < shape->n_req; ++b) {
    if (shape->h_q_len[b] < 1) return RELAXKV_ERR_INVALID_ARG;
    if (h_k[b] < 1 || h_k[b] > shape->h_ctx_len[b]) return RELAXKV_ERR_INVALID_ARG;
  }
  for (int l = 0; l < n_layers; ++l) {
    if (!q_layers[l] || !aligned16(q_layers[l])) return RELAXKV_ERR_INVALID_ARG;
    if ((rc = check_cache(shape, &cache_layers[l], false)) != RELAXKV_OK) return rc;
  }
  const WsLayout ws = ws_layout(shape, n_layers);
  if (workspace_bytes < ws.total) return RELAXKV_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  long long sum_t = 0;
  for (int b = 0; b < shape->n_req; ++b) sum_t += shape->h_ctx_len[b];

  for (int l = 0; l < n_layers; ++l) {
    ReqTable rt;
    fill_req_table(rt, shape, &cache_layers[l], h_k);
    const float* lse = row_lse_layers ? row_lse_layers[l] : nullptr;
    float* raw = raw_scores_out + (long long)l * sum_t;
    if (shape->head_dim == 128)
      rc = score_layer<128>(shape, rt, q_layers[l], &cache_layers[l], lse, raw, static_cast<char*>(workspace), ws, stream);
    else
      rc = score_layer<64>(shape, rt, q_layers[l], &cache_layers[l], lse, raw, static_cast<char*>(workspace), ws, stream);
    if (rc != RELAXKV_OK) return rc;
  }
  ReqTable rt;
  fill_req_table(rt, shape, nullptr, h_k);
  return launch_select(rt, n_layers, raw_scores_out, norm_scores_out, anchors_out, stream);
}
