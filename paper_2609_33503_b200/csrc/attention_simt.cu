// Test utility: sparse-context repair attention on plain SIMT lanes (no tensor cores), one warp per
// (target, query head) output row, fp32 throughout.  Same inputs, outputs and gather step as the
// tensor-core kernel; it exists as a second opinion when debugging and is far slower.
#include "attention_common.cuh"

namespace relaxkv {

constexpr float kLog2eS = 1.4426950408889634f;
constexpr float kLn2S = 0.6931471805599453f;

template <int D>
__global__ void __launch_bounds__(128)
attention_simt_kernel(ReqTable rt, int mode, int H, int Hkv, float scale_log2,
                      const uint16_t* __restrict__ q_new, const uint16_t* __restrict__ kctx,
                      const uint16_t* __restrict__ vctx,
                      const int* __restrict__ u_pos, const int* __restrict__ u_cu,
                      const int* __restrict__ r_rank, const int* __restrict__ r_cu,
                      long long n_target_rows, uint16_t* __restrict__ out, float* __restrict__ lse_out,
                      DeviceStatus* st) {
  __shared__ float qs[4][D];
  const int B = rt.n_req;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long pair = (long long)blockIdx.x * 4 + warp;
  const long long y = pair / H;                 // index into the host-bound target rows
  const int h = (int)(pair - y * H);
  if (y >= rt.tile_cu[B]) return;
  const int b = find_segment(rt.tile_cu, B, (int)y);
  const int rho = (int)y - rt.tile_cu[b];
  const int nr = r_cu[b + 1] - r_cu[b];
  if (rho >= nr) return;
  const int nu = u_cu[b + 1] - u_cu[b];
  const int c_star = r_rank[r_cu[b] + rho];
  if (c_star < 0 || c_star >= nu || nr > rt.bound_a[b] || nu > rt.bound_b[b]) {
    if (lane == 0) report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SIMT, c_star, nu);
    return;
  }
  const long long row = (long long)(r_cu[b] - r_cu[0]) + rho;
  if (row >= n_target_rows) { if (lane == 0) report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SIMT, (int)row, -1); return; }
  long long ctx_base;
  int limit;
  if (mode == RELAXKV_CTX_UNION) { ctx_base = u_cu[b]; limit = c_star; }
  else { ctx_base = rt.ctx_cu[b]; limit = u_pos[u_cu[b] + c_star]; }
  const int g = h / (H / Hkv);

  for (int d = lane; d < D; d += 32) qs[warp][d] = bf16_bits_to_float(q_new[(row * H + h) * D + d]);
  __syncwarp();

  constexpr int DPL = D / 32;                   // output dims per lane
  float acc[DPL];
#pragma unroll
  for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
  float m = -INFINITY, z = 0.f;
  for (int c0 = 0; c0 <= limit; c0 += 32) {
    const int c = c0 + lane;
    float s2 = -INFINITY;
    if (c <= limit) {
      const uint16_t* kr = kctx + ((ctx_base + c) * Hkv + g) * D;
      float dot = 0.f;
#pragma unroll 4
      for (int d = 0; d < D; d += 8) {
        const uint4 v = *reinterpret_cast<const uint4*>(kr + d);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          dot = fmaf(qs[warp][d + 2 * e], __uint_as_float(w[e] << 16), dot);
          dot = fmaf(qs[warp][d + 2 * e + 1], __uint_as_float(w[e] & 0xffff0000u), dot);
        }
      }
      s2 = dot * scale_log2;
    }
    const float m_new = fmaxf(m, warp_reduce_max(s2));
    const float alpha = exp2f(m - m_new);
    const float p = (c <= limit) ? exp2f(s2 - m_new) : 0.f;
    z = z * alpha + warp_reduce_sum(p);
    m = m_new;
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] *= alpha;
    const int n_here = min(32, limit - c0 + 1);
    for (int kk = 0; kk < n_here; ++kk) {
      const float pk = __shfl_sync(0xffffffffu, p, kk);
      const uint16_t* vr = vctx + ((ctx_base + c0 + kk) * Hkv + g) * D + lane * DPL;
#pragma unroll
      for (int i = 0; i < DPL; ++i) acc[i] = fmaf(pk, bf16_bits_to_float(vr[i]), acc[i]);
    }
  }
  const float inv = 1.f / z;
  __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(out) + (row * H + h) * D + lane * DPL;
#pragma unroll
  for (int i = 0; i < DPL; ++i) o[i] = __float2bfloat16_rn(acc[i] * inv);
  if (lse_out && lane == 0) lse_out[(long long)h * n_target_rows + row] = (m + log2f(z)) * kLn2S;
}

}  // namespace relaxkv

using namespace relaxkv;

extern "C" relaxkv_status relaxkv_sparse_ctx_attention_simt(
    const relaxkv_shape* shape, relaxkv_ctx_mode mode, const relaxkv_cache_view* cache,
    const void* q_new, const void* k_new, const void* v_new,
    const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank, const int32_t* r_cu_layer,
    int64_t n_target_rows, const int32_t* h_max_targets, const int32_t* h_max_ctx,
    void* out, float* lse_out, void* workspace, size_t workspace_bytes, relaxkv_stream stream_) {
  RELAXKV_RANGE("relaxkv_sparse_ctx_attention_simt");
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  AttnPlan plan;
  relaxkv_status rc = prepare_attention(shape, mode, cache, q_new, k_new, v_new, u_pos, u_cu, r_rank, r_cu_layer,
                                        n_target_rows, h_max_targets, h_max_ctx, out, workspace, workspace_bytes,
                                        stream, plan);
  if (rc != RELAXKV_OK) return rc;
  if (plan.sum_targets == 0) return RELAXKV_OK;
  for (int b = 0; b < shape->n_req; ++b) plan.rt.tile_cu[b + 1] = plan.rt.tile_cu[b] + plan.rt.bound_a[b];
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  const int H = shape->n_q_heads;
  const long long pairs = plan.sum_targets * H;
  const unsigned blocks = (unsigned)((pairs + 3) / 4);
  const float scale_log2 = shape->softmax_scale * kLog2eS;
  if (shape->head_dim == 128)
    attention_simt_kernel<128><<<blocks, 128, 0, stream>>>(plan.rt, mode, H, shape->n_kv_heads, scale_log2,
        static_cast<const uint16_t*>(q_new), plan.kctx, plan.vctx, u_pos, u_cu, r_rank, r_cu_layer, n_target_rows,
        static_cast<uint16_t*>(out), lse_out, st);
  else
    attention_simt_kernel<64><<<blocks, 128, 0, stream>>>(plan.rt, mode, H, shape->n_kv_heads, scale_log2,
        static_cast<const uint16_t*>(q_new), plan.kctx, plan.vctx, u_pos, u_cu, r_rank, r_cu_layer, n_target_rows,
        static_cast<uint16_t*>(out), lse_out, st);
  return launch_ok();
}
