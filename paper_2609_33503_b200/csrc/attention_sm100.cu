// Sparse-context repair attention on the Blackwell tensor cores (Section 3.3; Algorithm 1, steps 16-19).
//
// One CTA owns a tile of 128 query rows = (floor(128/G) consecutive active targets) x (the G query
// heads of one KV head), so every K/V tile it stages is shared by the whole GQA group.  It walks the
// context prefix the tile can see in 128-key tiles of the materialised mixed context:
//   TMA (128B swizzle)  ->  S = Q K^T  (tcgen05.mma, fp32 accumulator in TMEM)
//   softmax warps: tcgen05.ld S, position-based causal mask on the staircase edge, online max/sum with
//                  lazy rescaling, P -> bf16 back into TMEM (over S)
//   O += P V            (tcgen05.mma, A operand = P from TMEM, B = V tile MN-major from shared memory)
// Warp roles: warps 0-3 softmax/epilogue (thread = query row = TMEM lane), warp 4 TMA producer,
// warp 5 MMA issuer and TMEM owner.  Every wait is bounded; an expired wait raises the block's abort
// flag, records RELAXKV_ERR_TIMEOUT in the device status word and the block tears down normally.
#include "attention_common.cuh"
#include "sm100_ptx.cuh"

namespace relaxkv {

using namespace ptx;

constexpr float kLog2eA = 1.4426950408889634f;
constexpr float kLn2A = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;     // log2 units: rescale O only when the row max grew by more

constexpr int kBM = 128;                      // query rows per tile (TMEM lanes)
constexpr int kBN = 128;                      // keys per context tile
constexpr int kHalfBytes = 128 * 128;         // 128 rows x 64 bf16: one 128B-swizzled half tile
constexpr int kStages = 2;
constexpr int kAttnThreads = 192;

template <int D>
struct AttnSmem {
  static constexpr int kHalves = D / 64;
  static constexpr int kTileBytes = kHalves * kHalfBytes;
  static constexpr int kQ = 0;
  static constexpr int kK = kQ + kTileBytes;
  static constexpr int kV = kK + kStages * kTileBytes;
  static constexpr int kBar = kV + kStages * kTileBytes;      // mbarriers (8 B each)
  static constexpr int kNumBars = 4 + 3 * kStages;
  static constexpr int kMisc = kBar + 8 * kNumBars;           // tmem address, abort flag
  static constexpr int kTotal = kMisc + 16;
  static constexpr int kDynamic = kTotal + 1024;              // slack to align the base to 1024 B
};

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ ReqTable rt,
                       int mode, int H, int Hkv, int tile_targets, float scale_log2,
                       const int* __restrict__ u_pos, const int* __restrict__ u_cu,
                       const int* __restrict__ r_rank, const int* __restrict__ r_cu,
                       long long n_target_rows, uint16_t* __restrict__ out, float* __restrict__ lse_out,
                       DeviceStatus* st) {
  using L = AttnSmem<D>;
  constexpr int kHalves = L::kHalves;
  constexpr uint32_t kTmemCols = (D == 128) ? 256u : 256u;   // S: 128 columns, O: D columns
  constexpr uint32_t kColS = 0, kColO = 128;

  // ---- which tile ------------------------------------------------------------------------------
  const int B = rt.n_req;
  const int G = H / Hkv;
  const int n_tiles_total = rt.tile_cu[B];
  const int hd = blockIdx.x / n_tiles_total;                  // KV head (outermost: one head's K/V stays in L2)
  const int tt = blockIdx.x - hd * n_tiles_total;
  const int b = find_segment(rt.tile_cu, B, tt);
  const int t_rev = tt - rt.tile_cu[b];
  const int nr = r_cu[b + 1] - r_cu[b];
  const int nu = u_cu[b + 1] - u_cu[b];
  const int n_tiles_true = (nr + tile_targets - 1) / tile_targets;
  if (t_rev >= n_tiles_true) return;
  if (nr > rt.bound_a[b] || (mode == RELAXKV_CTX_UNION && nu > rt.bound_b[b])) {
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SM100, nr, nu);
    return;
  }
  if (*reinterpret_cast<volatile int*>(&st->status) == RELAXKV_ERR_TIMEOUT) return;   // drain after a timeout
  const int tile = n_tiles_true - 1 - t_rev;                  // longest tiles first
  const int rho0 = tile * tile_targets;
  const int n_valid = min(tile_targets, nr - rho0);
  const long long q_row0 = (long long)(r_cu[b] - r_cu[0]) + rho0;
  const int ctx_len_b = (mode == RELAXKV_CTX_UNION) ? nu : rt.ctx_len[b];
  const long long ctx_base = (mode == RELAXKV_CTX_UNION) ? (long long)u_cu[b] : rt.ctx_cu[b];
  // causal limit of the last target of the tile -> number of context tiles
  int lim_last;
  {
    const int c = r_rank[r_cu[b] + rho0 + n_valid - 1];
    const int cc = min(max(c, 0), max(nu - 1, 0));
    lim_last = (mode == RELAXKV_CTX_UNION) ? cc : u_pos[u_cu[b] + cc];
    lim_last = min(max(lim_last, 0), ctx_len_b - 1);
  }
  const int n_kv = lim_last / kBN + 1;

  // ---- shared memory -----------------------------------------------------------------------------
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t q_smem = base + L::kQ, k_smem = base + L::kK, v_smem = base + L::kV;
  const uint32_t bar0 = base + L::kBar;
  const uint32_t bar_q = bar0, bar_sfull = bar0 + 8, bar_pfull = bar0 + 16, bar_odone = bar0 + 24;
  const uint32_t bar_kfull = bar0 + 32, bar_vfull = bar_kfull + 8 * kStages, bar_empty = bar_vfull + 8 * kStages;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::kMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::kMisc + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1); mbar_init(bar_sfull, 1); mbar_init(bar_pfull, 128); mbar_init(bar_odone, 1);
    for (int s = 0; s < kStages; ++s) { mbar_init(bar_kfull + 8 * s, 1); mbar_init(bar_vfull + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 5) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  // rows of the Q tile that no (target, head) pair fills: zero them (they feed unused MMA rows)
  {
    const int used = tile_targets * G;
    for (int i = threadIdx.x; i < (kBM - used) * 8 * kHalves; i += kAttnThreads) {
      const int row = used + (i >> 3) % (kBM - used), piece = i & 7, half = (i >> 3) / (kBM - used);
      *reinterpret_cast<uint4*>(base_ptr + L::kQ + half * kHalfBytes + row * 128 + piece * 16) = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 4) {
    // ================= TMA producer =================
    if (lane == 0) {
      prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
      mbar_expect_tx(bar_q, (uint32_t)(kHalves * tile_targets * G * 128));
      for (int hf = 0; hf < kHalves; ++hf)
        tma_load_3d(q_smem + hf * kHalfBytes, &tm_q, bar_q, hf * 64, hd * G, (int)q_row0);
      for (int j = 0; j < n_kv; ++j) {
        const int s = j % kStages;
        if (j >= kStages && !mbar_wait(bar_empty + 8 * s, ((j / kStages) - 1) & 1, abort_flag)) break;
        const int row = (int)(ctx_base + (long long)j * kBN);
        mbar_expect_tx(bar_kfull + 8 * s, L::kTileBytes);
        for (int hf = 0; hf < kHalves; ++hf)
          tma_load_3d(k_smem + s * L::kTileBytes + hf * kHalfBytes, &tm_k, bar_kfull + 8 * s, hf * 64, hd, row);
        mbar_expect_tx(bar_vfull + 8 * s, L::kTileBytes);
        for (int hf = 0; hf < kHalves; ++hf)
          tma_load_3d(v_smem + s * L::kTileBytes + hf * kHalfBytes, &tm_v, bar_vfull + 8 * s, hf * 64, hd, row);
      }
    }
  } else if (warp == 5) {
    // ================= MMA issuer =================
    if (lane == 0) {
      constexpr uint32_t idesc_qk = idesc_bf16_f32(kBM, kBN, 0);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(kBM, D, 1);
      const uint32_t t_s = tmem_base + kColS, t_o = tmem_base + kColO;
      bool ok = mbar_wait(bar_q, 0, abort_flag);
      for (int j = 0; ok && j < n_kv; ++j) {
        const int s = j % kStages;
        const uint32_t ph = (j / kStages) & 1;
        if (!(ok = mbar_wait(bar_kfull + 8 * s, ph, abort_flag))) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
          mma_ss(t_s, smem_desc_sw128(q_smem + off, 16, 1024),
                 smem_desc_sw128(k_smem + s * L::kTileBytes + off, 16, 1024), idesc_qk, kk > 0);
        }
        mma_commit(bar_sfull);
        if (!(ok = mbar_wait(bar_pfull, j & 1, abort_flag))) break;
        if (!(ok = mbar_wait(bar_vfull + 8 * s, ph, abort_flag))) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < kBN / 16; ++kk) {
          mma_ts(t_o, t_s + kk * 8, smem_desc_sw128(v_smem + s * L::kTileBytes + kk * 2048, kHalfBytes, 1024),
                 idesc_pv, (j > 0) || (kk > 0));
        }
        mma_commit(bar_empty + 8 * s);
        mma_commit(bar_odone);
      }
    }
  } else {
    // ================= softmax + epilogue: thread = query row = TMEM lane =================
    const int row = threadIdx.x;                               // 0..127
    const int t_local = row / G, j_head = row - t_local * G;
    const bool row_valid = (row < tile_targets * G) && (t_local < n_valid);
    int limit = 0;
    if (row_valid) {
      const int c = r_rank[r_cu[b] + rho0 + t_local];
      if (c < 0 || c >= nu) {
        report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SM100, c, nu);
      } else {
        limit = (mode == RELAXKV_CTX_UNION) ? c : u_pos[u_cu[b] + c];
        if (limit < 0 || limit >= ctx_len_b) { report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SM100, limit, ctx_len_b); limit = 0; }
      }
    }
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
    const uint32_t t_s = lane_base + kColS, t_o = lane_base + kColO;
    float m = -INFINITY, z = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      ok = mbar_wait(bar_sfull, j & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t s[kBN];
#pragma unroll
      for (int c = 0; c < kBN / 32; ++c) tmem_ld32(t_s + c * 32, &s[c * 32]);
      tmem_wait_ld();
      const int col0 = j * kBN;
      if (col0 + kBN - 1 > limit) {
#pragma unroll
        for (int i = 0; i < kBN; ++i)
          if (col0 + i > limit) s[i] = 0xff800000u;              // -inf
      }
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < kBN; ++i) mx = fmaxf(mx, __uint_as_float(s[i]));
      const float m_new = mx * scale_log2;
      if (j == 0) {
        m = m_new;
      } else {
        const bool need = m_new > m + kRescaleThreshold;
        if (__any_sync(0xffffffffu, need)) {
          ok = mbar_wait(bar_odone, (j - 1) & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          float alpha = 1.f;
          if (need) { alpha = fast_exp2(m - m_new); z *= alpha; m = m_new; }
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(t_o + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
            tmem_st32(t_o + c * 32, o);
          }
          tmem_wait_st();
        }
      }
      uint32_t pk[kBN / 2];
      float zs = 0.f;
#pragma unroll
      for (int i = 0; i < kBN; i += 2) {
        const float p0 = fast_exp2(fmaf(__uint_as_float(s[i]), scale_log2, -m));
        const float p1 = fast_exp2(fmaf(__uint_as_float(s[i + 1]), scale_log2, -m));
        zs += p0 + p1;
        __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
        pk[i >> 1] = *reinterpret_cast<uint32_t*>(&h2);
      }
      z += zs;
      tmem_st32(t_s, &pk[0]);
      tmem_st32(t_s + 32, &pk[32]);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_pfull);
    }
    if (ok) {
      ok = mbar_wait(bar_odone, (n_kv - 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      const float inv = 1.f / z;
      const long long orow = q_row0 + t_local;
      uint16_t* optr = out + (orow * H + hd * G + j_head) * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(t_o + c * 32, o);
        tmem_wait_ld();
        if (row_valid) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(o[i + 2 * e]) * inv,
                                                        __uint_as_float(o[i + 2 * e + 1]) * inv);
              w[e] = *reinterpret_cast<uint32_t*>(&h2);
            }
            *reinterpret_cast<uint4*>(optr + c * 32 + i) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      if (row_valid && lse_out) lse_out[(long long)(hd * G + j_head) * n_target_rows + orow] = (m + log2f(z)) * kLn2A;
    }
  }

  // ---- teardown ------------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_TIMEOUT, KID_ATTN_SM100, tile, hd);
    // give copies and MMAs still in flight time to land before shared memory and TMEM are released
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---- host side ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor [d2, d1, d0] with d0 contiguous; box {64, b1, b2}; 128-byte swizzle; out-of-range reads give zeros.
bool make_map_3d(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_bytes,
                 uint64_t stride2_bytes, uint32_t b1, uint32_t b2) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {d0, d1, d2};
  const cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
  const cuuint32_t box[3] = {64u, b1, b2};
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
static relaxkv_status launch_attention(const relaxkv_shape* shape, int mode, AttnPlan& plan, const void* q_new,
                                       const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank,
                                       const int32_t* r_cu_layer, long long n_target_rows, void* out, float* lse_out,
                                       cudaStream_t stream) {
  const int H = shape->n_q_heads, Hkv = shape->n_kv_heads, G = H / Hkv;
  const int tile_targets = kBM / G;
  const int B = shape->n_req;
  for (int b = 0; b < B; ++b)
    plan.rt.tile_cu[b + 1] = plan.rt.tile_cu[b] + (plan.rt.bound_a[b] + tile_targets - 1) / tile_targets;
  const long long grid = (long long)plan.rt.tile_cu[B] * Hkv;
  if (grid == 0) return RELAXKV_OK;
  if (grid > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  CUtensorMap tm_q, tm_k, tm_v;
  const uint64_t row_q = (uint64_t)H * D * 2, row_kv = (uint64_t)Hkv * D * 2;
  if (!make_map_3d(&tm_q, q_new, D, H, (uint64_t)n_target_rows, (uint64_t)D * 2, row_q, (uint32_t)G, (uint32_t)tile_targets) ||
      !make_map_3d(&tm_k, plan.kctx, D, Hkv, (uint64_t)plan.ctx_rows, (uint64_t)D * 2, row_kv, 1u, (uint32_t)kBN) ||
      !make_map_3d(&tm_v, plan.vctx, D, Hkv, (uint64_t)plan.ctx_rows, (uint64_t)D * 2, row_kv, 1u, (uint32_t)kBN))
    return RELAXKV_ERR_CUDA;
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  auto kern = attention_sm100_kernel<D>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<D>::kDynamic) != cudaSuccess)
    return RELAXKV_ERR_CUDA;
  kern<<<(unsigned)grid, kAttnThreads, AttnSmem<D>::kDynamic, stream>>>(
      tm_q, tm_k, tm_v, plan.rt, mode, H, Hkv, tile_targets, shape->softmax_scale * kLog2eA, u_pos, u_cu, r_rank,
      r_cu_layer, n_target_rows, static_cast<uint16_t*>(out), lse_out, st);
  return launch_ok();
}

}  // namespace relaxkv

using namespace relaxkv;

extern "C" relaxkv_status relaxkv_sparse_ctx_attention(
    const relaxkv_shape* shape, relaxkv_ctx_mode mode, const relaxkv_cache_view* cache,
    const void* q_new, const void* k_new, const void* v_new,
    const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank, const int32_t* r_cu_layer,
    int64_t n_target_rows, const int32_t* h_max_targets, const int32_t* h_max_ctx,
    void* out, float* lse_out, void* workspace, size_t workspace_bytes, relaxkv_stream stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  AttnPlan plan;
  relaxkv_status rc = prepare_attention(shape, mode, cache, q_new, k_new, v_new, u_pos, u_cu, r_rank, r_cu_layer,
                                        n_target_rows, h_max_targets, h_max_ctx, out, workspace, workspace_bytes,
                                        stream, plan);
  if (rc != RELAXKV_OK) return rc;
  if (shape->head_dim == 128)
    return launch_attention<128>(shape, mode, plan, q_new, u_pos, u_cu, r_rank, r_cu_layer, n_target_rows, out, lse_out, stream);
  return launch_attention<64>(shape, mode, plan, q_new, u_pos, u_cu, r_rank, r_cu_layer, n_target_rows, out, lse_out, stream);
}
