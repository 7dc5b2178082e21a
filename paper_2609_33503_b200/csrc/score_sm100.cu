// Query-attention scoring on the Blackwell tensor cores (Section 3.2, score equation).
//
// One CTA owns (request, KV head, a block of <= 640 query rows, a range of 128-key tiles).  The query
// rows of the KV head's group - flat rows r = token*G + head-in-group - stay resident in shared
// memory; key tiles stream through a 2-stage TMA ring straight from the cache (any token/head
// strides).  Each (key tile, 128-row chunk) product goes to one of four 128-column TMEM buffers:
//   pass 1 (row statistics):  S   = Q_chunk K_tile^T   lanes = query rows, columns = keys
//   pass 2 (column sums):     S^T = K_tile Q_chunk^T   lanes = keys,       columns = query rows
// so that in both passes the reduction a thread needs runs along its own TMEM lane.  Two softmax
// warpgroups take the buffers alternately; the exponentials (one per 2*D MMA flops) bound the
// kernel, not the tensor pipe and not HBM.  Partial results are combined in a fixed order by the
// small kernels of score.cu, so scores are bit-reproducible.
#include "score_sm100.cuh"
#include "sm100_ptx.cuh"

namespace relaxkv {

using namespace ptx;

constexpr int kScThreads = 320;               // 2 softmax warpgroups, TMA warp, MMA warp
constexpr int kScBufs = 4;                    // TMEM accumulator buffers of 128 columns
constexpr int kScKStages = 2;
constexpr int kScTokBox = kScoreTokBox;        // query tokens per TMA box (keeps box starts 1024-B aligned)

template <int D>
struct ScoreSmem {
  static constexpr int kHalves = D / 64;
  static constexpr int kQHalfBytes = kScoreMaxRows * 128;          // resident query rows, one 64-dim half
  static constexpr int kKHalfBytes = 128 * 128;
  static constexpr int kQ = 0;
  static constexpr int kK = kQ + kHalves * kQHalfBytes;
  static constexpr int kLse = kK + kScKStages * kHalves * kKHalfBytes;   // fp32 [kScoreMaxRows]
  static constexpr int kBar = kLse + kScoreMaxRows * 4;
  static constexpr int kNumBars = 1 + 2 * kScKStages + 2 * kScBufs;
  static constexpr int kMisc = kBar + 8 * kNumBars;
  static constexpr int kTotal = kMisc + 16;
};

// Per-layer arguments of one launch: tensor maps of the layer's Q rows and K cache, its supplied
// log-normalisers (NULL: computed by pass 1) - by value in the kernel parameters.
struct ScoreLayers {
  CUtensorMap tm_q[kScoreLayersPerLaunch];
  CUtensorMap tm_k[kScoreLayersPerLaunch];
  const float* lse_given[kScoreLayersPerLaunch];
};

template <int D, bool PASS2>
__global__ void __launch_bounds__(kScThreads, 1)
score_sm100_kernel(const __grid_constant__ ScoreLayers layers, const __grid_constant__ ReqTable rt, int H, int Hkv,
                   float scale_log2, int n_splits, int max_super, const float* __restrict__ lse_ws,
                   float2* __restrict__ part_all, float* __restrict__ colpart_all, DeviceStatus* st) {
  using L = ScoreSmem<D>;
  constexpr int kHalves = L::kHalves;
  constexpr float kLog2e = 1.4426950408889634f;

  // ---- which unit ---------------------------------------------------------------------------------
  const int B = rt.n_req;
  const int G = H / Hkv;
  const int layer = blockIdx.z / n_splits, split = blockIdx.z - layer * n_splits;
  const int g = blockIdx.y;
  const int b = find_segment(rt.tile_cu, B, (int)blockIdx.x);     // rt.tile_cu: prefix of query-row blocks
  const int super = blockIdx.x - rt.tile_cu[b];
  const int n_super = rt.tile_cu[b + 1] - rt.tile_cu[b];
  const int Qb = rt.q_len[b], T = rt.ctx_len[b];
  const int tok_per = ((Qb + n_super - 1) / n_super + kScTokBox - 1) / kScTokBox * kScTokBox;
  const int t0 = super * tok_per;
  const int n_tok = min(tok_per, Qb - t0);
  if (n_tok <= 0) return;
  const int rows = n_tok * G;                                      // valid flat rows of this block
  const int n_chunks = (rows + 127) / 128;
  const int n_box = (n_tok + kScTokBox - 1) / kScTokBox;
  const int rows_loaded = n_box * kScTokBox * G;
  const int n_kt = (T + 127) / 128;
  const int per = (n_kt + n_splits - 1) / n_splits;
  const int kt0 = split * per, kt1 = min(n_kt, kt0 + per);
  const int sum_q = rt.q_cu[B];
  const long long sum_t = rt.ctx_cu[B];
  const CUtensorMap& tm_q = layers.tm_q[layer];
  const CUtensorMap& tm_k = layers.tm_k[layer];
  const float* given = layers.lse_given[layer];
  if (!PASS2 && given != nullptr) return;                          // this layer's log-normalisers were supplied
  const float* lse = given ? given : lse_ws + (long long)layer * H * sum_q;
  float2* part = part_all + (long long)layer * (2 * n_splits) * H * sum_q;
  float* colpart = colpart_all + (long long)layer * (2 * Hkv * max_super) * sum_t;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wg = warp >> 2;                                        // softmax warpgroup (0/1) for warps 0..7
  const int lane_row = (warp & 3) * 32 + lane;                     // TMEM lane of a softmax thread

  if (kt0 >= kt1) {
    // no keys in this split: pass 1 still owes neutral partials for its rows
    if (!PASS2 && warp < 8) {
      for (int c = 0; c < n_chunks; ++c) {
        const int r = c * 128 + lane_row;
        if (r < rows) {
          const int h = g * G + r % G;
          part[((long long)(split * 2 + wg) * H + h) * sum_q + rt.q_cu[b] + t0 + r / G] = make_float2(-INFINITY, 0.f);
        }
      }
    }
    return;
  }
  if (*reinterpret_cast<volatile int*>(&st->status) == RELAXKV_ERR_TIMEOUT) return;

  // ---- shared memory -------------------------------------------------------------------------------
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  if ((base & 1023u) != 0u) {                                      // the swizzled tiles need a 1024-B aligned base
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_BAD_INDEX, KID_SCORE_SM100, (int)base, -1);
    return;
  }
  const uint32_t q_smem = base + L::kQ, k_smem = base + L::kK;
  float* lse2s = reinterpret_cast<float*>(smem_raw + L::kLse);
  const uint32_t bar0 = base + L::kBar;
  const uint32_t bar_q = bar0;
  const uint32_t bar_kfull = bar0 + 8, bar_kempty = bar_kfull + 8 * kScKStages;
  const uint32_t bar_sfull = bar_kempty + 8 * kScKStages, bar_sempty = bar_sfull + 8 * kScBufs;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_raw + L::kMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + L::kMisc + 4);

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    for (int s = 0; s < kScKStages; ++s) { mbar_init(bar_kfull + 8 * s, 1); mbar_init(bar_kempty + 8 * s, 1); }
    for (int i = 0; i < kScBufs; ++i) { mbar_init(bar_sfull + 8 * i, 1); mbar_init(bar_sempty + 8 * i, 128); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 9) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
    tmem_relinquish();
  }
  // zero the resident rows that no TMA box fills (they feed unused MMA rows / masked columns)
  for (int i = threadIdx.x; i < (n_chunks * 128 - rows_loaded) * 8 * kHalves; i += kScThreads) {
    const int n_pad = n_chunks * 128 - rows_loaded;
    const int piece = i & 7, r = (i >> 3) % n_pad, hf = (i >> 3) / n_pad;
    *reinterpret_cast<uint4*>(smem_raw + L::kQ + hf * L::kQHalfBytes + (rows_loaded + r) * 128 + piece * 16) = make_uint4(0, 0, 0, 0);
  }
  if (PASS2) {
    // log-normalisers of the resident rows in log2 units; rows past the block's end can never contribute
    for (int r = threadIdx.x; r < n_chunks * 128; r += kScThreads)
      lse2s[r] = (r < rows) ? lse[(long long)(g * G + r % G) * sum_q + rt.q_cu[b] + t0 + r / G] * kLog2e : INFINITY;
  }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int n_items = (kt1 - kt0) * n_chunks;

  if (warp == 8) {
    // ================= TMA producer =================
    if (lane == 0) {
      prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k);
      mbar_expect_tx(bar_q, (uint32_t)(n_box * kHalves * kScTokBox * G * 128));
      for (int i = 0; i < n_box; ++i)
        for (int hf = 0; hf < kHalves; ++hf)
          tma_load_3d(q_smem + hf * L::kQHalfBytes + i * kScTokBox * G * 128, &tm_q, bar_q, hf * 64, g * G,
                      rt.q_cu[b] + t0 + i * kScTokBox);
      for (int kt = kt0; kt < kt1; ++kt) {
        const int u = kt - kt0, s = u % kScKStages;
        if (u >= kScKStages && !mbar_wait(bar_kempty + 8 * s, ((u / kScKStages) - 1) & 1, abort_flag)) break;
        mbar_expect_tx(bar_kfull + 8 * s, kHalves * L::kKHalfBytes);
        for (int hf = 0; hf < kHalves; ++hf)
          tma_load_3d(k_smem + (s * kHalves + hf) * L::kKHalfBytes, &tm_k, bar_kfull + 8 * s, hf * 64, g,
                      (int)(rt.tok_off[b] + (long long)kt * 128));
      }
    }
  } else if (warp == 9) {
    // ================= MMA issuer =================
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(128, 128, 0);
      bool ok = mbar_wait(bar_q, 0, abort_flag);
      int it = 0;
      for (int kt = kt0; ok && kt < kt1; ++kt) {
        const int u = kt - kt0, s = u % kScKStages;
        if (!(ok = mbar_wait(bar_kfull + 8 * s, (u / kScKStages) & 1, abort_flag))) break;
        for (int c = 0; c < n_chunks; ++c, ++it) {
          const int buf = it % kScBufs;
          if (it >= kScBufs && !(ok = mbar_wait(bar_sempty + 8 * buf, ((it / kScBufs) - 1) & 1, abort_flag))) break;
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t hf = kk >> 2, off = (kk & 3) * 32;
            const uint64_t dq = smem_desc_sw128(q_smem + hf * L::kQHalfBytes + c * 128 * 128 + off, 16, 1024);
            const uint64_t dk = smem_desc_sw128(k_smem + (s * kHalves + hf) * L::kKHalfBytes + off, 16, 1024);
            if (PASS2) mma_ss(tmem_base + buf * 128, dk, dq, idesc, kk > 0);
            else       mma_ss(tmem_base + buf * 128, dq, dk, idesc, kk > 0);
          }
          mma_commit(bar_sfull + 8 * buf);
        }
        if (!ok) break;
        mma_commit(bar_kempty + 8 * s);
      }
    }
  } else {
    // ================= softmax warpgroups: warpgroup w consumes the buffers of items it % 2 == w =================
    // (whole 128-column buffers: one barrier wait - ~145 cycles even when it succeeds at once - per 128
    //  exponentials of a thread instead of per 64)
    const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    float m_row[kScoreMaxRows / 128], z_row[kScoreMaxRows / 128];
#pragma unroll
    for (int c = 0; c < kScoreMaxRows / 128; ++c) { m_row[c] = -INFINITY; z_row[c] = 0.f; }
    bool ok = true;
    int it = 0;
    for (int kt = kt0; ok && kt < kt1; ++kt) {
      float acc = 0.f;
#pragma unroll
      for (int c = 0; c < kScoreMaxRows / 128; ++c) {
        if (c < n_chunks) {
          const int my_it = it++;
          if ((my_it & 1) == wg) {
            const int buf = my_it % kScBufs;
            ok = mbar_wait(bar_sfull + 8 * buf, (my_it / kScBufs) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t s[128];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) tmem_ld32(t_lane + buf * 128 + q4 * 32, &s[q4 * 32]);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar_sempty + 8 * buf);                      // the values are in registers: release the buffer
            if (PASS2) {
              const float4* l4 = reinterpret_cast<const float4*>(lse2s + c * 128);
              float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                const float4 lv = l4[i];
                a0 += fast_exp2(fmaf(__uint_as_float(s[4 * i]), scale_log2, -lv.x));
                a1 += fast_exp2(fmaf(__uint_as_float(s[4 * i + 1]), scale_log2, -lv.y));
                a2 += fast_exp2(fmaf(__uint_as_float(s[4 * i + 2]), scale_log2, -lv.z));
                a3 += fast_exp2(fmaf(__uint_as_float(s[4 * i + 3]), scale_log2, -lv.w));
              }
              acc += (a0 + a1) + (a2 + a3);
            } else {
              const int key0 = kt * 128;
              if (key0 + 127 >= T) {
#pragma unroll
                for (int i = 0; i < 128; ++i)
                  if (key0 + i >= T) s[i] = 0xff800000u;             // keys past the context: -inf
              }
              float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
              for (int i = 0; i < 128; i += 4) {
#pragma unroll
                for (int e = 0; e < 4; ++e) mx4[e] = fmaxf(mx4[e], __uint_as_float(s[i + e]));
              }
              const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
              const float m_new = fmaxf(m_row[c], mx * scale_log2);
              if (m_new > -INFINITY) {
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
                for (int i = 0; i < 128; i += 4) {
                  a0 += fast_exp2(fmaf(__uint_as_float(s[i]), scale_log2, -m_new));
                  a1 += fast_exp2(fmaf(__uint_as_float(s[i + 1]), scale_log2, -m_new));
                  a2 += fast_exp2(fmaf(__uint_as_float(s[i + 2]), scale_log2, -m_new));
                  a3 += fast_exp2(fmaf(__uint_as_float(s[i + 3]), scale_log2, -m_new));
                }
                z_row[c] = z_row[c] * fast_exp2(m_row[c] - m_new) + ((a0 + a1) + (a2 + a3));
                m_row[c] = m_new;
              }
            }
          }
        }
      }
      if (!ok) break;
      if (PASS2) {
        const int key = kt * 128 + lane_row;
        if (key < T)
          colpart[(long long)((g * max_super + super) * 2 + wg) * sum_t + rt.ctx_cu[b] + key] = acc;
      }
    }
    if (ok && !PASS2) {
#pragma unroll
      for (int c = 0; c < kScoreMaxRows / 128; ++c) {
        const int r = c * 128 + lane_row;
        if (c < n_chunks && r < rows) {
          const int h = g * G + r % G;
          part[((long long)(split * 2 + wg) * H + h) * sum_q + rt.q_cu[b] + t0 + r / G] = make_float2(m_row[c], z_row[c]);
        }
      }
    }
  }

  // ---- teardown --------------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_TIMEOUT, KID_SCORE_SM100, (int)blockIdx.x, split);
    const uint64_t tw = global_timer_ns();
    while (global_timer_ns() - tw < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
  (void)n_items;
}

// ---- host side ------------------------------------------------------------------------------------------
bool make_map_3d(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_bytes,
                 uint64_t stride2_bytes, uint32_t b1, uint32_t b2);          // attention_sm100.cu

ScorePlan plan_score(const relaxkv_shape* shape) {
  ScorePlan p{};
  const int G = shape->n_q_heads / shape->n_kv_heads;
  p.max_super = 1;
  p.units = 0;
  for (int b = 0; b < shape->n_req; ++b) {
    const int ns = score_blocks(shape->h_q_len ? shape->h_q_len[b] : 0, G);
    p.n_super[b] = ns;
    p.units += ns;
    if (ns > p.max_super) p.max_super = ns;
  }
  return p;
}

template <int D>
relaxkv_status launch_score_sm100(const relaxkv_shape* shape, ReqTable rt, const ScorePlan& plan, int n_layers,
                                  const void* const* q_layers, const relaxkv_cache_view* cache_layers,
                                  const float* const* lse_given, float* lse_ws, float2* part, float* colpart,
                                  cudaStream_t stream) {
  const int B = shape->n_req, H = shape->n_q_heads, Hkv = shape->n_kv_heads, G = H / Hkv;
  const int sum_q = rt.q_cu[B];
  if (n_layers < 1 || n_layers > kScoreLayersPerLaunch) return RELAXKV_ERR_INVALID_ARG;
  long long tok_extent = 0;
  for (int b = 0; b < B; ++b) {
    rt.tile_cu[b + 1] = rt.tile_cu[b] + plan.n_super[b];
    const long long e = rt.tok_off[b] + rt.ctx_len[b];
    if (e > tok_extent) tok_extent = e;
  }
  if (tok_extent > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  ScoreLayers layers;
  bool need_pass1 = false;
  for (int l = 0; l < n_layers; ++l) {
    const relaxkv_cache_view* c = &cache_layers[l];
    if (!make_map_3d(&layers.tm_q[l], q_layers[l], D, H, (uint64_t)sum_q, (uint64_t)D * 2, (uint64_t)H * D * 2, (uint32_t)G,
                     kScTokBox) ||
        !make_map_3d(&layers.tm_k[l], c->k, D, Hkv, (uint64_t)tok_extent, (uint64_t)c->head_stride * 2,
                     (uint64_t)c->token_stride * 2, 1u, 128u))
      return RELAXKV_ERR_CUDA;
    layers.lse_given[l] = lse_given ? lse_given[l] : nullptr;
    if (!layers.lse_given[l]) need_pass1 = true;
  }
  for (int l = n_layers; l < kScoreLayersPerLaunch; ++l) {
    layers.tm_q[l] = layers.tm_q[0]; layers.tm_k[l] = layers.tm_k[0]; layers.lse_given[l] = nullptr;
  }
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  const float scale_log2 = shape->softmax_scale * 1.4426950408889634f;
  const int n_splits = score_splits((long long)plan.units * Hkv, n_layers);
  const dim3 grid((unsigned)rt.tile_cu[B], (unsigned)Hkv, (unsigned)(n_splits * n_layers));
  if (grid.x == 0) return RELAXKV_OK;
  constexpr int smem = ScoreSmem<D>::kTotal;
  static std::atomic<int> attr_done[kMaxDevices];          // per device: the opt-in to > 48 KB of dynamic shared memory
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RELAXKV_ERR_CUDA;
  auto k1 = score_sm100_kernel<D, false>;
  auto k2 = score_sm100_kernel<D, true>;
  if (!attr_done[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
        cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
      return RELAXKV_ERR_CUDA;
    attr_done[dev].store(1, std::memory_order_release);
  }
  if (need_pass1) {
    k1<<<grid, kScThreads, smem, stream>>>(layers, rt, H, Hkv, scale_log2, n_splits, plan.max_super, lse_ws, part, colpart, st);
    launch_combine_lse(n_layers, H, sum_q, n_splits * 2, part, lse_ws, stream);
  }
  k2<<<grid, kScThreads, smem, stream>>>(layers, rt, H, Hkv, scale_log2, n_splits, plan.max_super, lse_ws, part, colpart, st);
  return launch_ok();
}

template relaxkv_status launch_score_sm100<64>(const relaxkv_shape*, ReqTable, const ScorePlan&, int, const void* const*,
                                               const relaxkv_cache_view*, const float* const*, float*, float2*, float*,
                                               cudaStream_t);
template relaxkv_status launch_score_sm100<128>(const relaxkv_shape*, ReqTable, const ScorePlan&, int, const void* const*,
                                                const relaxkv_cache_view*, const float* const*, float*, float2*, float*,
                                                cudaStream_t);

}  // namespace relaxkv
