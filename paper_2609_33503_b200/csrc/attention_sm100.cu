// Sparse-context repair attention on the Blackwell tensor cores (Section 3.3; Algorithm 1, steps 16-19).
//
// One CTA owns a tile of 128 query rows = (floor(128/G) consecutive active targets) x (the G query
// heads of one KV head), so every K/V tile it stages is shared by the whole GQA group.  It walks the
// context prefix the tile can see in 128-key tiles of the materialised mixed context:
//   TMA (128B swizzle)  ->  S = Q K^T  (tcgen05.mma, fp32 accumulator in TMEM)
//   softmax warps: tcgen05.ld S, position-based causal mask on the staircase edge, online max/sum with
//                  lazy rescaling, P -> bf16 back into TMEM (over S)
//   O += P V            (tcgen05.mma, A operand = P from TMEM, B = V tile MN-major from shared memory)
// A CTA runs TWO such query tiles (A, B) in ping-pong: while the softmax warps of one tile work, the
// tensor pipe runs the other tile's MMAs; both tiles share every K/V tile staged in shared memory.
// Warp roles: warps 0-3 softmax/epilogue of tile A, warps 4-7 of tile B (thread = query row = TMEM
// lane), warp 8 TMA producer, warp 9 MMA issuer and TMEM owner, warp 10 a helper for cache-only calls.  K/V tiles
// move through a 5-slot ring in the order K_0 V_0 K_1 V_1 ... and are signalled in pairs (V_j, K_{j+1}) - what
// step j of the MMA warp consumes.
// When a call has too few query tiles to fill the GPU, grid.y splits every pair's context; the blocks leave
// normalised partial results that combine_splits_kernel merges by their log-sum-exp.  The K/V tensor maps
// cover either the materialised mixed context (the repair calls) or the cache itself (relaxkv_cache_attention).
// Calls over short gathered contexts (at most 128 key tiles, one split) take attention_persist_kernel below: one
// block per SM walks the same list of (tile pair, KV head) items and overlaps each turn-over with its neighbours.
// Every wait is bounded; an expired wait raises the block's abort flag, records RELAXKV_ERR_TIMEOUT in the
// device status word and the block tears down normally.
#include "attention_common.cuh"
#include "decode_attention.cuh"
#include "sm100_ptx.cuh"
#include <algorithm>
#include <atomic>

namespace relaxkv {

using namespace ptx;

constexpr float kLog2eA = 1.4426950408889634f;
constexpr float kLn2A = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;     // log2 units: rescale O only when the row max grew by more

constexpr int kBM = 128;                      // query rows per tile (TMEM lanes)
constexpr int kBN = 128;                      // keys per context tile
constexpr int kHalfBytes = 128 * 128;         // 128 rows x 64 bf16: one 128B-swizzled half tile
constexpr int kRing = 5;                      // K/V tile buffers, used in the order K0 V0 K1 V1 ...
constexpr int kPersistMaxTiles = 128;          // contexts up to this many key tiles take the persistent form
constexpr int kAttnThreads = 384;             // 2 x 4 softmax warps + a control warpgroup (TMA warp, MMA warp, 2 idle)

template <int D>
struct AttnSmem {
  static constexpr int kHalves = D / 64;
  static constexpr int kTileBytes = kHalves * kHalfBytes;
  static constexpr int kQ = 0;                                  // two query tiles
  static constexpr int kKV = kQ + 2 * kTileBytes;               // ring of kRing K/V tiles
  static constexpr int kBar = kKV + kRing * kTileBytes;         // mbarriers (8 B each)
  static constexpr int kPairBars = 3;                           // (V_j, K_{j+1}) pairs in flight: full and empty barriers
  static constexpr int kNumBars = 1 + 8 + 2 * kPairBars + 2;
  static constexpr int kMisc = kBar + 8 * kNumBars;             // tmem address, abort flag
  static constexpr int kTotal = kMisc + 16;
  static constexpr int kDynamic = kTotal + 1024;                // slack to align the base to 1024 B
};

// One step of a query row's online softmax (thread = query row = TMEM lane): S_x(j) is read from TMEM, the keys
// past the row's limit are masked on the tiles that straddle the staircase (col0 = index of the tile's first key),
// the running maximum m and sum z are updated (O_x is rescaled only when the maximum grew by more than the
// threshold), and P is written over S as bf16 in two column halves, each handed to the MMA warp (bar_p_lo,
// bar_p_hi) as soon as it is stored.
template <int D>
__device__ __forceinline__ void softmax_step(uint32_t t_s, uint32_t t_o, int col0, int limit, bool first, float scale_log2,
                                             float& m, float& z, uint32_t bar_p_lo, uint32_t bar_p_hi) {
  uint32_t s[kBN];
#pragma unroll
  for (int c = 0; c < kBN / 32; ++c) tmem_ld32(t_s + c * 32, &s[c * 32]);
  tmem_wait_ld();
  if (col0 + kBN - 1 > limit) {
#pragma unroll
    for (int i = 0; i < kBN; ++i)
      if (col0 + i > limit) s[i] = 0xff800000u;              // -inf
  }
  // row maximum: eight independent chains instead of one 128-deep dependency chain
  float mx8[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) mx8[e] = __uint_as_float(s[e]);
#pragma unroll
  for (int i = 8; i + 16 <= kBN; i += 16) {
#pragma unroll
    for (int e = 0; e < 8; ++e) mx8[e] = fmax3(mx8[e], __uint_as_float(s[i + e]), __uint_as_float(s[i + 8 + e]));
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) mx8[e] = fmaxf(mx8[e], __uint_as_float(s[kBN - 8 + e]));
  const float mx = fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])),
                         fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
  const float m_new = mx * scale_log2;
  if (first) {
    m = fmaxf(m_new, -1.0e30f);           // a row whose first tile of this split is fully masked keeps a finite reference
  } else {
    // S_x(j) is complete, hence so is O_x += P_x V_{j-1}: O_x may be rescaled here
    const bool need = m_new > m + kRescaleThreshold;
    if (__any_sync(0xffffffffu, need)) {
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
  float zs0 = 0.f, zs1 = 0.f, zs2 = 0.f, zs3 = 0.f;
  const float neg_m = -m;
#pragma unroll
  for (int c = 0; c < kBN / 32; ++c) {
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 32; i += 8) {
      // p = 2^(s * scale - m) for eight keys; the scaling and the row sums use packed fp32 pairs
      float x[8], p[8];
#pragma unroll
      for (int e = 0; e < 8; e += 2)
        fma2(x[e], x[e + 1], __uint_as_float(s[c * 32 + i + e]), __uint_as_float(s[c * 32 + i + e + 1]), scale_log2,
             scale_log2, neg_m, neg_m);
#pragma unroll
      for (int e = 0; e < 8; ++e) p[e] = fast_exp2(x[e]);
      add2(zs0, zs1, p[0], p[1]); add2(zs2, zs3, p[2], p[3]);
      add2(zs0, zs1, p[4], p[5]); add2(zs2, zs3, p[6], p[7]);
#pragma unroll
      for (int e = 0; e < 8; e += 2) {
        __nv_bfloat162 h = __floats2bfloat162_rn(p[e], p[e + 1]);
        pk[(i + e) >> 1] = *reinterpret_cast<uint32_t*>(&h);
      }
    }
    tmem_st16(t_s + c * 16, pk);
    if (c == kBN / 64 - 1) {          // first 64 keys done: hand them to the MMA warp early
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_p_lo);
    }
  }
  z += (zs0 + zs1) + (zs2 + zs3);
  tmem_wait_st();
  tc_fence_before();
  mbar_arrive(bar_p_hi);
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ ReqTable rt,
                       int mode, int allow_empty, int head_inner, int dense_ctx, int H, int Hkv, int tile_targets, float scale_log2,
                       const int* __restrict__ u_pos, const int* __restrict__ u_cu,
                       const int* __restrict__ r_rank, const int* __restrict__ r_cu,
                       long long n_target_rows, uint16_t* __restrict__ out, float* __restrict__ lse_out,
                       float* __restrict__ part_o, float* __restrict__ part_lse, DeviceStatus* st) {
  using L = AttnSmem<D>;
  constexpr int kHalves = L::kHalves;
  constexpr uint32_t kTmemCols = 512;          // S_A | S_B | O_A | O_B, 128 columns each (O uses D of them)

  // ---- which pair of query tiles ------------------------------------------------------------------
  // rt.tile_cu counts tile PAIRS per request (from the host bounds); pairs are walked from the end of
  // the target list (longest context first).  Tile A = the earlier targets, tile B = the later ones.
  const int B = rt.n_req;
  const int G = H / Hkv;
  const int n_pairs_total = rt.tile_cu[B];
  // Block order.  Large contexts: KV head outermost, so one head's K/V stays in L2 while its tiles run.
  // Contexts that fit L2 whole (head_inner): tile pair outermost, so the longest tiles of every head start first.
  const int hd = head_inner ? (int)(blockIdx.x % Hkv) : (int)(blockIdx.x / n_pairs_total);
  const int tt = head_inner ? (int)(blockIdx.x / Hkv) : (int)(blockIdx.x - hd * n_pairs_total);
  const int b = find_segment(rt.tile_cu, B, tt);
  const int p_rev = tt - rt.tile_cu[b];
  const int nr = r_cu[b + 1] - r_cu[b];
  // dense_ctx: the context is the cache itself (every position of the request), a target's limit is its position
  const int nu = dense_ctx ? rt.ctx_len[b] : (u_cu[b + 1] - u_cu[b]);
  const int pair_targets = 2 * tile_targets;
  const int n_pairs_true = (nr + pair_targets - 1) / pair_targets;
  if (p_rev >= n_pairs_true) return;
  // a true count above its host bound, or more target rows than q_new / out hold: report, touch nothing
  if (nr > rt.bound_a[b] || (mode == RELAXKV_CTX_UNION && nu > rt.bound_b[b]) ||
      (long long)(r_cu[b + 1] - r_cu[0]) > n_target_rows) {
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SM100, nr, nu);
    return;
  }
  if (*reinterpret_cast<volatile int*>(&st->status) == RELAXKV_ERR_TIMEOUT) return;   // drain after a timeout
  const int pair = n_pairs_true - 1 - p_rev;
  const int rho0 = pair * pair_targets;                       // first target of tile A
  const int ctx_len_b = (mode == RELAXKV_CTX_UNION) ? nu : rt.ctx_len[b];
  const long long ctx_base = dense_ctx ? rt.tok_off[b] : ((mode == RELAXKV_CTX_UNION) ? (long long)u_cu[b] : rt.ctx_cu[b]);
  const long long q_row_base = (long long)(r_cu[b] - r_cu[0]) + rho0;
  // valid targets and context tiles of each query tile
  int n_valid[2], n_kv[2];
#pragma unroll
  for (int x = 0; x < 2; ++x) {
    n_valid[x] = max(0, min(tile_targets, nr - rho0 - x * tile_targets));
    n_kv[x] = 0;
    if (n_valid[x] > 0) {
      const int c = r_rank[r_cu[b] + rho0 + x * tile_targets + n_valid[x] - 1];
      const int cc = min(max(c, 0), max(nu - 1, 0));
      int lim_last = (mode == RELAXKV_CTX_UNION) ? cc : u_pos[u_cu[b] + cc];
      lim_last = min(max(lim_last, 0), ctx_len_b - 1);
      n_kv[x] = lim_last / kBN + 1;
    }
  }
  const int n_kv_max = max(n_kv[0], n_kv[1]);
  // Context split (gridDim.y > 1, used when there are too few query tiles to fill the GPU): this block walks the
  // context tiles [j0, j0 + chunk) of its pair and leaves a normalised partial result + its log-sum-exp.
  const int n_splits = (int)gridDim.y, split = (int)blockIdx.y;
  const int chunk = (n_kv_max + n_splits - 1) / n_splits;
  const int j0 = split * chunk;
  int n_my[2];
#pragma unroll
  for (int x = 0; x < 2; ++x) n_my[x] = max(0, min(n_kv[x], j0 + chunk) - j0);
  const int n_my_max = max(n_my[0], n_my[1]);
  if (n_my_max == 0) {                        // nothing of this pair's context falls into this split
    if (n_splits > 1 && threadIdx.x < 2 * kBM) {
      const int x = threadIdx.x >> 7, row = threadIdx.x & 127, t_local = row / G;
      if (row < tile_targets * G && t_local < n_valid[x]) {
        const long long orow = q_row_base + x * tile_targets + t_local;
        part_lse[((long long)split * n_target_rows + orow) * H + hd * G + (row - t_local * G)] = -INFINITY;
      }
    }
    return;
  }

  // Cache-only calls read K/V tiles straight from the cache: the last tile of a request may reach past the request's
  // final token into rows that belong to nobody.  Their keys are masked, but their V rows would still meet a zero
  // probability on the tensor core (0 x NaN = NaN), so a helper warp zeroes those V rows once the tile has landed.
  const int v_fix_tile = (dense_ctx && (ctx_len_b % kBN) != 0) ? (ctx_len_b / kBN - j0) : -1;
  const bool need_v_fix = v_fix_tile >= 0 && v_fix_tile < n_my_max;

  // ---- shared memory -----------------------------------------------------------------------------
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t q_smem = base + L::kQ, kv_smem = base + L::kKV;
  const uint32_t bar0 = base + L::kBar;
  const uint32_t bar_q = bar0;
  const uint32_t bar_sfull = bar0 + 8;          // [2]
  const uint32_t bar_pfull = bar0 + 24;         // [2] first 64 keys of P ready
  const uint32_t bar_pfull_hi = bar0 + 40;      // [2] last 64 keys of P ready
  const uint32_t bar_ofinal = bar0 + 56;        // [2]
  const uint32_t bar_full = bar0 + 72;          // [kPairBars] pair p = (V_{p-1}, K_p) has landed
  const uint32_t bar_empty = bar_full + 8 * L::kPairBars;   // [kPairBars] pair p has been consumed by both tiles
  const uint32_t bar_vreq = bar_empty + 8 * L::kPairBars;   // the request's last V tile has landed (MMA warp -> helper warp)
  const uint32_t bar_vfix = bar_vreq + 8;                   // its rows past the request's end are zeroed (helper -> MMA warp)
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::kMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::kMisc + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    for (int x = 0; x < 2; ++x) { mbar_init(bar_sfull + 8 * x, 1); mbar_init(bar_pfull + 8 * x, 128); mbar_init(bar_pfull_hi + 8 * x, 128); mbar_init(bar_ofinal + 8 * x, 1); }
    for (int s = 0; s < L::kPairBars; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    mbar_init(bar_vreq, 1);
    mbar_init(bar_vfix, 32);
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 9) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  // rows of the Q tiles that no (target, head) pair fills: zero them (they feed unused MMA rows)
  {
    const int used = tile_targets * G;
    const int n_pad = kBM - used;
    for (int i = threadIdx.x; i < n_pad * 8 * kHalves * 2; i += kAttnThreads) {
      const int piece = i & 7, r = (i >> 3) % n_pad, blk = (i >> 3) / n_pad;    // blk = tile * kHalves + half
      *reinterpret_cast<uint4*>(base_ptr + L::kQ + blk * kHalfBytes + (used + r) * 128 + piece * 16) = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Register budget: the control warpgroup gives registers to the two softmax warpgroups
  // (12 warps x 168 at launch = 8 x 224 + 4 x 56).
  if (warp >= 8) {
  reg_dealloc<56>();
  if (warp == 8) {
    // ================= TMA producer =================
    if (lane == 0) {
      prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
      mbar_expect_tx(bar_q, (uint32_t)(2 * kHalves * tile_targets * G * 128));
      for (int x = 0; x < 2; ++x)
        for (int hf = 0; hf < kHalves; ++hf)
          tma_load_3d(q_smem + (x * kHalves + hf) * kHalfBytes, &tm_q, bar_q, hf * 64, hd * G,
                      (int)(q_row_base + x * tile_targets));
      // The tiles travel in the order K_0 V_0 K_1 V_1 ... through the ring slots u % kRing (u = 2j for K_j, 2j + 1
      // for V_j; j counted from j0).  They are signalled in PAIRS p = (V_{p-1}, K_p): step j of the MMA warp needs
      // exactly pair j + 1 (V_j for P V, K_{j+1} for the next Q K^T), so it waits once and frees once per step.
      auto load_tile = [&](int u, uint32_t bar) {
        const int s = u % kRing;
        const int row = (int)(ctx_base + (long long)(j0 + (u >> 1)) * kBN);
        const CUtensorMap* tm = (u & 1) ? &tm_v : &tm_k;
        for (int hf = 0; hf < kHalves; ++hf)
          tma_load_3d(kv_smem + s * L::kTileBytes + hf * kHalfBytes, tm, bar, hf * 64, hd, row);
      };
      for (int pr = 0; pr <= n_my_max; ++pr) {                  // pair pr: V_{pr-1} (if pr > 0) and K_pr (if pr < n)
        const uint32_t bar = bar_full + 8 * (pr % L::kPairBars);
        const bool has_v = pr > 0, has_k = pr < n_my_max;
        // slot of V_{pr-1} was last used by K_{pr-3} (pair pr-3), slot of K_pr by V_{pr-3} (pair pr-2)
        if (pr >= 3 && !mbar_wait(bar_empty + 8 * ((pr - 3) % L::kPairBars), (uint32_t)((pr - 3) / L::kPairBars) & 1, abort_flag)) break;
        mbar_expect_tx(bar, (uint32_t)((has_v ? L::kTileBytes : 0) + (has_k ? L::kTileBytes : 0)));
        if (has_v) load_tile(2 * pr - 1, bar);
        if (has_k) {
          if (pr >= 3 && !mbar_wait(bar_empty + 8 * ((pr - 2) % L::kPairBars), (uint32_t)((pr - 2) / L::kPairBars) & 1, abort_flag)) break;
          load_tile(2 * pr, bar);
        }
      }
    }
  } else if (warp == 9) {
    // ================= MMA issuer =================
    if (lane == 0) {
      constexpr uint32_t idesc_qk = idesc_bf16_f32(kBM, kBN, 0);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(kBM, D, 1);
      bool ok = mbar_wait(bar_q, 0, abort_flag);
      // This lane issues every MMA, and each instruction it executes in between delays the next one (measured: the
      // step got 1 % shorter when the ring-slot and barrier arithmetic below replaced a modulo and a division per
      // use).  So the positions are carried along and advanced once per step: ring slot of the step's V tile and of
      // the K tile behind it, and the pair barrier (byte offset, phase) that covers the two.
      uint32_t sv = 1, sk = 2, pk = 8, pph = 0;
      const int n0 = n_my[0], n1 = n_my[1];
      auto issue_qk = [&](int x, uint32_t slot) {                   // S_x = Q_x K^T with the K tile in `slot` -> bar_sfull[x]
        mma_ss_kloop<kHalves>(tmem_base + x * 128, desc_lo(q_smem + x * L::kTileBytes, 16),
                              desc_lo(kv_smem + slot * L::kTileBytes, 16), desc_hi_sw128(1024), idesc_qk);
        mma_commit(bar_sfull + 8 * x);
      };
      // O_x += P_x V   (P_x read from TMEM where the softmax warps left it, over S_x; V in slot sv)
      auto issue_pv = [&](int x, uint32_t par, uint32_t acc) -> bool {
        const uint32_t v_lo = desc_lo(kv_smem + sv * L::kTileBytes, kHalfBytes);
        if (!mbar_wait(bar_pfull + 8 * x, par, abort_flag)) return false;
        tc_fence_after();
        mma_ts_4steps(tmem_base + 256 + x * 128, tmem_base + x * 128, v_lo, desc_hi_sw128(1024), idesc_pv, acc);
        // the second half of P arrives while the first half is being multiplied
        if (!mbar_wait(bar_pfull_hi + 8 * x, par, abort_flag)) return false;
        tc_fence_after();
        mma_ts_4steps(tmem_base + 256 + x * 128, tmem_base + x * 128 + 32, v_lo + 512, desc_hi_sw128(1024), idesc_pv, 1u);
        return true;
      };
      // pair 0 = K_0 alone
      if (ok) ok = mbar_wait(bar_full, 0, abort_flag);
      if (ok) {
        tc_fence_after();
        if (n0 > 0) issue_qk(0, 0);
        if (n1 > 0) issue_qk(1, 0);
        mma_commit(bar_empty);
      }
      for (int j = 0; ok && j < n_my_max; ++j) {                // j counted from j0; this step consumes pair j + 1
        if (!(ok = mbar_wait(bar_full + pk, pph, abort_flag))) break;
        if (need_v_fix && j == v_fix_tile) {                    // V_j reaches past the request's end: have those rows zeroed
          mbar_arrive(bar_vreq);
          if (!(ok = mbar_wait(bar_vfix, 0, abort_flag))) break;
        }
        tc_fence_after();
        const uint32_t par = (uint32_t)j & 1u, acc = j > 0 ? 1u : 0u;
        if (j < n0) {
          if (!(ok = issue_pv(0, par, acc))) break;
          if (j == n0 - 1) mma_commit(bar_ofinal);
          if (j + 1 < n0) issue_qk(0, sk);
        }
        if (j < n1) {
          if (!(ok = issue_pv(1, par, acc))) break;
          if (j == n1 - 1) mma_commit(bar_ofinal + 8);
          if (j + 1 < n1) issue_qk(1, sk);
        }
        mma_commit(bar_empty + pk);                             // V_j and K_{j+1}: free once both tiles are through
        sv += 2; if (sv >= kRing) sv -= kRing;
        sk += 2; if (sk >= kRing) sk -= kRing;
        pk += 8; if (pk == 8 * L::kPairBars) { pk = 0; pph ^= 1u; }
      }
    }
  } else if (warp == 10 && need_v_fix) {
    // ================= helper: zero the V rows past the request's last token (cache-only calls) =================
    if (mbar_wait(bar_vreq, 0, abort_flag)) {                   // raised by the MMA warp once that tile has landed
      const int first = ctx_len_b % kBN;                        // first foreign row of the tile
      uint8_t* vt = base_ptr + L::kKV + ((2 * v_fix_tile + 1) % kRing) * L::kTileBytes;
      for (int i = lane; i < (kBN - first) * 8 * kHalves; i += 32) {
        const int piece = i & 7, r = first + ((i >> 3) % (kBN - first)), hf = (i >> 3) / (kBN - first);
        *reinterpret_cast<uint4*>(vt + hf * kHalfBytes + r * 128 + piece * 16) = make_uint4(0, 0, 0, 0);
      }
      fence_proxy_async_smem();
    }
    mbar_arrive(bar_vfix);
  }
  } else {
    reg_alloc<224>();
    // ================= softmax + epilogue: thread = query row = TMEM lane =================
    const int x = warp >> 2;                                    // 0: tile A, 1: tile B
    const int row = threadIdx.x & 127;
    const int t_local = row / G, j_head = row - t_local * G;
    const bool row_valid = (row < tile_targets * G) && (t_local < n_valid[x]);
    const int rho_t = rho0 + x * tile_targets + t_local;
    int limit = 0;
    bool row_empty = false;                                     // explicit lists: a target that sees no context entry
    if (row_valid) {
      const int c = r_rank[r_cu[b] + rho_t];
      if (c == -1 && allow_empty) {
        row_empty = true;
      } else if (c < 0 || c >= nu) {
        report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SM100, c, nu);
      } else {
        limit = (mode == RELAXKV_CTX_UNION) ? c : u_pos[u_cu[b] + c];
        if (limit < 0 || limit >= ctx_len_b) { report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SM100, limit, ctx_len_b); limit = 0; }
      }
    }
    const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t t_s = lane_base + x * 128, t_o = lane_base + 256 + x * 128;
    const uint32_t my_sfull = bar_sfull + 8 * x, my_pfull = bar_pfull + 8 * x;
    const int my_n = n_my[x];
    float m = -INFINITY, z = 0.f;
    bool ok = true;
    for (int j = 0; j < my_n; ++j) {
      ok = mbar_wait(my_sfull, j & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      softmax_step<D>(t_s, t_o, (j0 + j) * kBN, limit, j == 0, scale_log2, m, z, my_pfull, bar_pfull_hi + 8 * x);
    }
    if (ok && my_n > 0) {
      ok = mbar_wait(bar_ofinal + 8 * x, 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok && my_n > 0) {
      tc_fence_after();
      const bool none = row_empty || !(z > 0.f);                // an empty context is defined as a zero output row
      const float inv = none ? 0.f : 1.f / z;
      const float lse = none ? -INFINITY : (m + log2f(z)) * kLn2A;
      const long long orow = q_row_base + x * tile_targets + t_local;
      if (n_splits == 1) {
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
        if (row_valid && lse_out) lse_out[(long long)(hd * G + j_head) * n_target_rows + orow] = lse;
      } else {
        // partial result of this split: fp32, normalised by this split's own sum
        const long long slot = ((long long)split * n_target_rows + orow) * H + hd * G + j_head;
        float* optr = part_o + slot * D;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(t_o + c * 32, o);
          tmem_wait_ld();
          if (row_valid) {
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              *reinterpret_cast<float4*>(optr + c * 32 + i) =
                  make_float4(__uint_as_float(o[i]) * inv, __uint_as_float(o[i + 1]) * inv, __uint_as_float(o[i + 2]) * inv,
                              __uint_as_float(o[i + 3]) * inv);
          }
        }
        if (row_valid) part_lse[slot] = lse;
      }
    } else if (ok && my_n == 0 && n_splits > 1 && row_valid) {
      // this tile's context ends before the split begins (the pair's other tile still has work here)
      const long long orow = q_row_base + x * tile_targets + t_local;
      part_lse[((long long)split * n_target_rows + orow) * H + hd * G + j_head] = -INFINITY;
    }
  }

  // ---- teardown ------------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_TIMEOUT, KID_ATTN_SM100, pair, hd);
    // give copies and MMAs still in flight time to land before shared memory and TMEM are released
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------------------------------
// Persistent form of the kernel above, for calls whose blocks are short (a context of at most 128 tiles): one block
// per SM walks work items (pair of query tiles x KV head, the same list in the same longest-first order) that its
// producer lane claims from a global counter a few steps before the current item ends.  Barriers, tensor memory and
// the K/V ring live across items; the next item's first K tile travels with the current item's last V tile, its Q
// tiles are loaded as soon as the current item's last Q K^T has completed, and its first Q K^T is issued right behind
// the current item's last P V, so a block turn-over costs about 5 k clk instead of about 14 k.  Items reach the other
// roles as 64-byte records in a two-slot mailbox in shared memory.  One split only, gathered contexts only (the
// cache-only calls keep the kernel above).  Same arithmetic per row, hence the same bits.
// ---------------------------------------------------------------------------------------------------------------------
template <int D>
struct PersistSmem {
  static constexpr int kHalves = D / 64;
  static constexpr int kTileBytes = kHalves * kHalfBytes;
  static constexpr int kQ = 0;
  static constexpr int kKV = kQ + 2 * kTileBytes;
  static constexpr int kBar = kKV + kRing * kTileBytes;
  static constexpr int kPairBars = 3;
  // q | s, p, p_hi, ofinal x2 | pairs full/empty | qfree | odrained x2 | item full x2 | item free x2
  static constexpr int kNumBars = 1 + 8 + 2 * kPairBars + 1 + 2 + 2 + 2;
  static constexpr int kMisc = kBar + 8 * kNumBars;                     // tmem address, abort flag, two item records
  static constexpr int kTotal = kMisc + 8 + 2 * 64;
  static constexpr int kDynamic = kTotal + 1024;
};

// One work item as every role needs it; 16 ints so that it travels through shared memory as four 16-byte pieces.
struct WorkItem {
  int work;            // 1: work, -1: the list is exhausted
  int n_max, n_my0, n_my1;
  int n_valid0, n_valid1, hd, q_row_base;
  int nu, ctx_len_b, r_base, rho0;      // r_base = r_cu[b]
  int u_base, ctx_base, b, pad;         // u_base = u_cu[b]
  __device__ __forceinline__ int n_valid(int x) const { return x ? n_valid1 : n_valid0; }
  __device__ __forceinline__ int n_my(int x) const { return x ? n_my1 : n_my0; }
};
__device__ __forceinline__ void item_store(int4* rec, const WorkItem& it) {
  rec[0] = make_int4(it.work, it.n_max, it.n_my0, it.n_my1);
  rec[1] = make_int4(it.n_valid0, it.n_valid1, it.hd, it.q_row_base);
  rec[2] = make_int4(it.nu, it.ctx_len_b, it.r_base, it.rho0);
  rec[3] = make_int4(it.u_base, it.ctx_base, it.b, 0);
}
__device__ __forceinline__ void item_load_head(const int4* rec, WorkItem& it) {      // what the MMA issuer needs
  const int4 a = rec[0];
  it.work = a.x; it.n_max = a.y; it.n_my0 = a.z; it.n_my1 = a.w;
}
__device__ __forceinline__ void item_load(const int4* rec, WorkItem& it) {
  item_load_head(rec, it);
  const int4 b = rec[1], c = rec[2], d = rec[3];
  it.n_valid0 = b.x; it.n_valid1 = b.y; it.hd = b.z; it.q_row_base = b.w;
  it.nu = c.x; it.ctx_len_b = c.y; it.r_base = c.z; it.rho0 = c.w;
  it.u_base = d.x; it.ctx_base = d.y; it.b = d.z; it.pad = 0;
}

__device__ __forceinline__ WorkItem decode_item(int id, const ReqTable& rt, int head_inner, int Hkv, int mode, int tile_targets,
                                                const int* __restrict__ u_pos, const int* __restrict__ u_cu,
                                                const int* __restrict__ r_rank, const int* __restrict__ r_cu,
                                                long long n_target_rows, DeviceStatus* st) {
  WorkItem it;
  it.work = 0; it.pad = 0;
  const int B = rt.n_req;
  const int n_pairs_total = rt.tile_cu[B];
  it.hd = head_inner ? (id % Hkv) : (id / n_pairs_total);
  const int tt = head_inner ? (id / Hkv) : (id - it.hd * n_pairs_total);
  const int b = find_segment(rt.tile_cu, B, tt);
  it.b = b;
  const int p_rev = tt - rt.tile_cu[b];
  it.r_base = r_cu[b]; it.u_base = u_cu[b];
  const int nr = r_cu[b + 1] - it.r_base;
  const int nu = u_cu[b + 1] - it.u_base;
  it.nu = nu;
  const int pair_targets = 2 * tile_targets;
  const int n_pairs_true = (nr + pair_targets - 1) / pair_targets;
  it.n_max = 0; it.n_my0 = it.n_my1 = 0; it.n_valid0 = it.n_valid1 = 0;
  it.rho0 = 0; it.ctx_len_b = 0; it.ctx_base = 0; it.q_row_base = 0;
  if (p_rev >= n_pairs_true) return it;
  if (nr > rt.bound_a[b] || (mode == RELAXKV_CTX_UNION && nu > rt.bound_b[b]) || (long long)(r_cu[b + 1] - r_cu[0]) > n_target_rows) {
    report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SM100, nr, nu);
    return it;
  }
  const int pair = n_pairs_true - 1 - p_rev;
  it.rho0 = pair * pair_targets;
  it.ctx_len_b = (mode == RELAXKV_CTX_UNION) ? nu : rt.ctx_len[b];
  it.ctx_base = (int)((mode == RELAXKV_CTX_UNION) ? (long long)it.u_base : rt.ctx_cu[b]);
  it.q_row_base = (it.r_base - r_cu[0]) + it.rho0;
  int nm[2] = {0, 0}, nv[2] = {0, 0};
#pragma unroll
  for (int x = 0; x < 2; ++x) {
    nv[x] = max(0, min(tile_targets, nr - it.rho0 - x * tile_targets));
    if (nv[x] > 0) {
      const int c = r_rank[it.r_base + it.rho0 + x * tile_targets + nv[x] - 1];
      const int cc = min(max(c, 0), max(nu - 1, 0));
      int lim_last = (mode == RELAXKV_CTX_UNION) ? cc : u_pos[it.u_base + cc];
      lim_last = min(max(lim_last, 0), it.ctx_len_b - 1);
      nm[x] = lim_last / kBN + 1;
    }
  }
  it.n_valid0 = nv[0]; it.n_valid1 = nv[1]; it.n_my0 = nm[0]; it.n_my1 = nm[1];
  it.n_max = max(nm[0], nm[1]);
  it.work = it.n_max > 0;
  return it;
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_persist_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                         const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ ReqTable rt,
                         int mode, int allow_empty, int head_inner, int H, int Hkv, int tile_targets, float scale_log2,
                         const int* __restrict__ u_pos, const int* __restrict__ u_cu,
                         const int* __restrict__ r_rank, const int* __restrict__ r_cu,
                         long long n_target_rows, uint16_t* __restrict__ out, float* __restrict__ lse_out,
                         int total_items, int* __restrict__ work_counter, DeviceStatus* st) {
  using L = PersistSmem<D>;
  constexpr int kHalves = L::kHalves;
  constexpr uint32_t kTmemCols = 512;
  const int G = H / Hkv;
  if (*reinterpret_cast<volatile int*>(&st->status) == RELAXKV_ERR_TIMEOUT) return;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t q_smem = base + L::kQ, kv_smem = base + L::kKV;
  const uint32_t bar0 = base + L::kBar;
  const uint32_t bar_q = bar0;
  const uint32_t bar_sfull = bar0 + 8, bar_pfull = bar0 + 24, bar_pfull_hi = bar0 + 40, bar_ofinal = bar0 + 56;
  const uint32_t bar_full = bar0 + 72, bar_empty = bar_full + 8 * L::kPairBars;
  const uint32_t bar_qfree = bar_empty + 8 * L::kPairBars;
  const uint32_t bar_odrained = bar_qfree + 8;          // [2]
  const uint32_t bar_item = bar_odrained + 16;          // [2]
  const uint32_t bar_itemfree = bar_item + 16;          // [2]
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::kMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::kMisc + 4);
  int4* item_rec = reinterpret_cast<int4*>(base_ptr + L::kMisc + 8 + 8);   // two records of 64 bytes, 16-byte aligned
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    for (int x = 0; x < 2; ++x) { mbar_init(bar_sfull + 8 * x, 1); mbar_init(bar_pfull + 8 * x, 128); mbar_init(bar_pfull_hi + 8 * x, 128); mbar_init(bar_ofinal + 8 * x, 1); }
    for (int s = 0; s < L::kPairBars; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    mbar_init(bar_qfree, 1);
    for (int x = 0; x < 2; ++x) { mbar_init(bar_odrained + 8 * x, 128); mbar_init(bar_item + 8 * x, 1); mbar_init(bar_itemfree + 8 * x, 2 * kBM + 1); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 9) { tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols); tmem_relinquish(); }
  {
    const int used = tile_targets * G;
    const int n_pad = kBM - used;
    for (int i = threadIdx.x; i < n_pad * 8 * kHalves * 2; i += kAttnThreads) {
      const int piece = i & 7, r = (i >> 3) % n_pad, blk = (i >> 3) / n_pad;
      *reinterpret_cast<uint4*>(base_ptr + L::kQ + blk * kHalfBytes + (used + r) * 128 + piece * 16) = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // The k-th published record sits in slot k & 1 (phase k >> 1).  A reader copies it and arrives on the slot's
  // "free" barrier; the producer overwrites a slot only after all 257 readers of its previous record have done so.
  auto read_item = [&](int k, WorkItem& it, bool head_only) -> bool {
    if (!mbar_wait(bar_item + 8 * (k & 1), (uint32_t)(k >> 1) & 1, abort_flag)) return false;
    if (head_only) item_load_head(item_rec + 4 * (k & 1), it); else item_load(item_rec + 4 * (k & 1), it);
    mbar_arrive(bar_itemfree + 8 * (k & 1));
    return true;
  };

  if (warp >= 8) {
  reg_dealloc<56>();
  if (warp == 8) {
    // ================= producer: work items, Q tiles, K/V tiles =================
    if (lane == 0) {
      prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
      int n_fetched = 0, n_pub = 0;
      bool ok = true;
      auto fetch_work = [&](WorkItem& it) -> bool {          // next item that has work; false when the list is exhausted
        for (;;) {
          const int id = (n_fetched == 0) ? (int)blockIdx.x : (int)gridDim.x + atomicAdd(work_counter, 1);
          ++n_fetched;
          if (id >= total_items) { it.work = -1; return false; }
          it = decode_item(id, rt, head_inner, Hkv, mode, tile_targets, u_pos, u_cu, r_rank, r_cu, n_target_rows, st);
          if (it.work) return true;
        }
      };
      auto publish = [&](const WorkItem& it) -> bool {
        const int k = n_pub;
        if (k >= 2 && !mbar_wait(bar_itemfree + 8 * (k & 1), (uint32_t)((k - 2) >> 1) & 1, abort_flag)) return false;
        item_store(item_rec + 4 * (k & 1), it);
        mbar_arrive(bar_item + 8 * (k & 1));
        ++n_pub;
        return true;
      };
      auto load_q = [&](const WorkItem& it) {
        mbar_expect_tx(bar_q, (uint32_t)(2 * kHalves * tile_targets * G * 128));
        for (int x = 0; x < 2; ++x)
          for (int hf = 0; hf < kHalves; ++hf)
            tma_load_3d(q_smem + (x * kHalves + hf) * kHalfBytes, &tm_q, bar_q, hf * 64, it.hd * G, it.q_row_base + x * tile_targets);
      };
      auto load_tile = [&](int u, const WorkItem& it, int j, uint32_t bar) {      // u = 2 g for K of global tile g, 2 g + 1 for V
        const int s = u % kRing;
        const int row = it.ctx_base + j * kBN;
        const CUtensorMap* tm = (u & 1) ? &tm_v : &tm_k;
        for (int hf = 0; hf < kHalves; ++hf) tma_load_3d(kv_smem + s * L::kTileBytes + hf * kHalfBytes, tm, bar, hf * 64, it.hd, row);
      };
      WorkItem cur, nxt;
      fetch_work(cur);
      ok = publish(cur);
      if (ok && cur.work > 0) {
        load_q(cur);
        int Gt = 0;                                                  // tile index, counted over the items, of cur's tile 0
        int cw = 0;                                                  // work items done so far
        for (;;) {
          bool have_nxt = false, fetched = false;
          for (int j = 0; ok && j <= cur.n_max; ++j) {               // pair g = (V_{g-1}, K_g)
            if (!fetched && j >= cur.n_max - 2) {                    // claim the next item late (the list balances the SMs
                                                                     // only if nobody holds work long before starting it),
                                                                     // yet a few steps before the readers ask for it
              have_nxt = fetch_work(nxt);
              fetched = true;
              if (!(ok = publish(nxt))) break;
            }
            if (j == 0 && cw > 0) continue;                          // loaded as the trailing pair of the previous item
            const int g = Gt + j;
            const bool has_v = j > 0;
            const bool has_k = (j < cur.n_max) || have_nxt;
            if (!has_v && !has_k) continue;
            const uint32_t bar = bar_full + 8 * (uint32_t)(g % L::kPairBars);
            if (g >= 3 && !(ok = mbar_wait(bar_empty + 8 * (uint32_t)((g - 3) % L::kPairBars), (uint32_t)((g - 3) / L::kPairBars) & 1, abort_flag))) break;
            mbar_expect_tx(bar, (uint32_t)((has_v ? L::kTileBytes : 0) + (has_k ? L::kTileBytes : 0)));
            if (has_v) load_tile(2 * g - 1, cur, j - 1, bar);
            if (has_k) {
              if (g >= 3 && !(ok = mbar_wait(bar_empty + 8 * (uint32_t)((g - 2) % L::kPairBars), (uint32_t)((g - 2) / L::kPairBars) & 1, abort_flag))) break;
              if (j < cur.n_max) load_tile(2 * g, cur, j, bar); else load_tile(2 * g, nxt, 0, bar);
            }
          }
          if (!ok || !have_nxt) break;
          // every Q K^T of cur has completed: the Q tiles may be replaced
          if (!(ok = mbar_wait(bar_qfree, (uint32_t)cw & 1, abort_flag))) break;
          load_q(nxt);
          Gt += cur.n_max; cur = nxt; ++cw;
        }
      }
    }
  } else if (warp == 9) {
    // ================= MMA issuer =================
    // One lane issues every MMA; each of its instructions delays the next one, so the loop over an item's inner steps
    // holds nothing but the waits and the issues, and the item's first and last step (which also look at the previous
    // item's epilogue and at the next item) run through a separate, general copy of the step.
    if (lane == 0) {
      constexpr uint32_t idesc_qk = idesc_bf16_f32(kBM, kBN, 0);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(kBM, D, 1);
      bool ok = true;
      uint32_t k = 0;                       // index of the current item
      uint32_t sp0 = 0, sp1 = 0;            // parity of each tile's next P (its S / P barriers complete once per step)
      uint32_t op0 = 0, op1 = 0;            // epilogues of each tile so far (parity of its "O drained" barrier)
      // running positions, advanced once per step: ring slot of the step's V tile and of the K tile behind it, and the
      // pair barrier (offset, phase) that covers the two
      uint32_t sv = 1, sk = 2, pk = 8;
      uint32_t pph = 0;
      auto issue_qk = [&](int x, uint32_t slot) {                   // S_x = Q_x K^T with the K tile in `slot`
        mma_ss_kloop<kHalves>(tmem_base + x * 128, desc_lo(q_smem + x * L::kTileBytes, 16), desc_lo(kv_smem + slot * L::kTileBytes, 16),
                              desc_hi_sw128(1024), idesc_qk);
        mma_commit(bar_sfull + 8 * x);
      };
      auto issue_pv = [&](int x, uint32_t par, uint32_t acc) -> bool {   // O_x (+)= P_x V with the V tile in slot sv
        const uint32_t v_lo = desc_lo(kv_smem + sv * L::kTileBytes, kHalfBytes);
        if (!mbar_wait(bar_pfull + 8 * x, par, abort_flag)) return false;
        tc_fence_after();
        mma_ts_4steps(tmem_base + 256 + x * 128, tmem_base + x * 128, v_lo, desc_hi_sw128(1024), idesc_pv, acc);
        if (!mbar_wait(bar_pfull_hi + 8 * x, par, abort_flag)) return false;
        tc_fence_after();
        mma_ts_4steps(tmem_base + 256 + x * 128, tmem_base + x * 128 + 32, v_lo + 512, desc_hi_sw128(1024), idesc_pv, 1u);
        return true;
      };
      auto advance = [&]() {
        mma_commit(bar_empty + pk);
        sv += 2; if (sv >= kRing) sv -= kRing;
        sk += 2; if (sk >= kRing) sk -= kRing;
        pk += 8; if (pk == 8 * L::kPairBars) { pk = 0; pph ^= 1u; }
      };
      WorkItem cur, nxt;
      cur.work = 0; nxt.work = 0; nxt.n_max = nxt.n_my0 = nxt.n_my1 = 0;
      ok = read_item(0, cur, true);
      if (ok && cur.work > 0) {
        ok = mbar_wait(bar_q, 0, abort_flag);
        if (ok) ok = mbar_wait(bar_full, 0, abort_flag);
        if (ok) {
          tc_fence_after();
          if (cur.n_my0 > 0) issue_qk(0, 0);
          if (cur.n_my1 > 0) issue_qk(1, 0);
          if (cur.n_max == 1) mma_commit(bar_qfree);
          mma_commit(bar_empty);
        }
        while (ok) {
          const int n0 = cur.n_my0, n1 = cur.n_my1, n_max = cur.n_max;
          bool have_nxt = false;
          // the general step: j = 0 and j = n_max - 1
          auto edge_step = [&](int j) -> bool {
            if (!mbar_wait(bar_full + pk, pph, abort_flag)) return false;
            const bool last = (j == n_max - 1);
            if (last) {                                             // the next item's record: shown early in cur
              if (!read_item((int)k + 1, nxt, true)) return false;
              have_nxt = nxt.work > 0;
            }
            tc_fence_after();
            bool q_ready = false;
            if (j < n0) {
              if (j == 0 && op0 > 0) {                              // O_0 of the previous item must have been read out
                if (!mbar_wait(bar_odrained, (op0 - 1) & 1u, abort_flag)) return false;
                tc_fence_after();
              }
              if (!issue_pv(0, (sp0 + (uint32_t)j) & 1u, j > 0 ? 1u : 0u)) return false;
              if (j == n0 - 1) mma_commit(bar_ofinal);
              if (j + 1 < n0) issue_qk(0, sk);
            }
            if (last && have_nxt && mbar_try_wait(bar_q, (k + 1) & 1u)) {   // the next item's Q tiles have landed already
              q_ready = true;
              tc_fence_after();
              if (nxt.n_my0 > 0) issue_qk(0, sk);
            }
            if (j < n1) {
              if (j == 0 && op1 > 0) {
                if (!mbar_wait(bar_odrained + 8, (op1 - 1) & 1u, abort_flag)) return false;
                tc_fence_after();
              }
              if (!issue_pv(1, (sp1 + (uint32_t)j) & 1u, j > 0 ? 1u : 0u)) return false;
              if (j == n1 - 1) mma_commit(bar_ofinal + 8);
              if (j + 1 < n1) issue_qk(1, sk);
            }
            if (last && have_nxt) {
              if (!q_ready) {
                if (!mbar_wait(bar_q, (k + 1) & 1u, abort_flag)) return false;
                tc_fence_after();
                if (nxt.n_my0 > 0) issue_qk(0, sk);
              }
              if (nxt.n_my1 > 0) issue_qk(1, sk);
              if (nxt.n_max == 1) mma_commit(bar_qfree);
            }
            advance();
            return true;
          };
          if (!(ok = edge_step(0))) break;
          // inner steps 1 .. n_max - 2
          for (int j = 1; j < n_max - 1; ++j) {
            if (!(ok = mbar_wait(bar_full + pk, pph, abort_flag))) break;
            tc_fence_after();
            if (j < n0) {
              if (!(ok = issue_pv(0, (sp0 + (uint32_t)j) & 1u, 1u))) break;
              if (j == n0 - 1) mma_commit(bar_ofinal);
              if (j + 1 < n0) issue_qk(0, sk);
            }
            if (j < n1) {
              if (!(ok = issue_pv(1, (sp1 + (uint32_t)j) & 1u, 1u))) break;
              if (j == n1 - 1) mma_commit(bar_ofinal + 8);
              if (j + 1 < n1) issue_qk(1, sk);
            }
            advance();
          }
          if (!ok) break;
          if (n_max >= 2) {
            mma_commit(bar_qfree);                                  // the last Q K^T of cur has been issued
            if (!(ok = edge_step(n_max - 1))) break;
          }
          sp0 += (uint32_t)n0; sp1 += (uint32_t)n1;
          op0 += (n0 > 0) ? 1u : 0u; op1 += (n1 > 0) ? 1u : 0u;
          if (!have_nxt) break;
          cur = nxt; ++k;
        }
      }
    }
  }
  } else {
    reg_alloc<224>();
    // ================= softmax + epilogue =================
    const int x = warp >> 2;
    const int row = threadIdx.x & 127;
    const int t_local = row / G, j_head = row - t_local * G;
    const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t t_s = lane_base + x * 128, t_o = lane_base + 256 + x * 128;
    const uint32_t my_sfull = bar_sfull + 8 * x, my_pfull = bar_pfull + 8 * x;
    const uint32_t rec_smem = smem_u32(item_rec);
    // One register of phase state: bit 0 = parity of this tile's next S, bit 1 = parity of its next final O,
    // bits 2.. = index of the current item.  The item's record stays in shared memory (its slot is released only
    // after the epilogue), so that little of it has to live in registers across the key loop.
    uint32_t ph = 0;
    auto rec_ld = [&](uint32_t k, int piece) -> int4 {
      int4 v;
      asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(rec_smem + (k & 1u) * 64u + piece * 16u));
      return v;
    };
    auto wait_rec = [&](uint32_t k) -> bool { return mbar_wait(bar_item + 8 * (k & 1u), (k >> 1) & 1u, abort_flag); };
    // this thread's row of item k: validity and the load of its context rank
    auto row_rank = [&](uint32_t k, bool& valid) -> int {
      const int4 a = rec_ld(k, 0), b = rec_ld(k, 1), cc = rec_ld(k, 2);
      valid = a.x > 0 && (row < tile_targets * G) && (t_local < (x ? b.y : b.x));
      return valid ? r_rank[cc.z + cc.w + x * tile_targets + t_local] : 0;
    };
    bool ok = wait_rec(0);
    bool row_valid = false;
    int c = ok ? row_rank(0, row_valid) : 0;
    while (ok) {
      const uint32_t k = ph >> 2;
      int limit = 0, my_n;
      bool row_empty = false;
      {
        const int4 a = rec_ld(k, 0);
        if (a.x <= 0) { mbar_arrive(bar_itemfree + 8 * (k & 1u)); break; }
        my_n = x ? a.w : a.z;
        if (row_valid) {
          const int4 cc = rec_ld(k, 2), d = rec_ld(k, 3);
          const int nu = cc.x, ctx_len_b = cc.y;
          if (c == -1 && allow_empty) {
            row_empty = true;
          } else if (c < 0 || c >= nu) {
            report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SM100, c, nu);
          } else {
            limit = (mode == RELAXKV_CTX_UNION) ? c : u_pos[d.x + c];
            if (limit < 0 || limit >= ctx_len_b) { report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SM100, limit, ctx_len_b); limit = 0; }
          }
        }
      }
      float m = -INFINITY, z = 0.f;
      for (int j = 0; j < my_n; ++j) {
        ok = mbar_wait(my_sfull, (ph + (uint32_t)j) & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        softmax_step<D>(t_s, t_o, j * kBN, limit, j == 0, scale_log2, m, z, my_pfull, bar_pfull_hi + 8 * x);
      }
      if (!ok) break;
      // the next item's record (shown long ago) and this thread's row of it: the load travels under the epilogue
      ok = wait_rec(k + 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      bool nrow_valid;
      const int nc = row_rank(k + 1, nrow_valid);
      if (my_n > 0) {
        ok = mbar_wait(bar_ofinal + 8 * x, (ph >> 1) & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const bool none = row_empty || !(z > 0.f);
        const float inv = none ? 0.f : 1.f / z;
        const float lse = none ? -INFINITY : (m + log2f(z)) * kLn2A;
        const int4 b = rec_ld(k, 1);
        const int hd = b.z;
        const long long orow = (long long)b.w + x * tile_targets + t_local;
        uint16_t* optr = out + (orow * H + hd * G + j_head) * D;
#pragma unroll
        for (int cc = 0; cc < D / 32; ++cc) {
          uint32_t o[32];
          tmem_ld32(t_o + cc * 32, o);
          tmem_wait_ld();
          if (row_valid) {
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint32_t w[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(o[i + 2 * e]) * inv, __uint_as_float(o[i + 2 * e + 1]) * inv);
                w[e] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(optr + cc * 32 + i) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
        if (row_valid && lse_out) lse_out[(long long)(hd * G + j_head) * n_target_rows + orow] = lse;
        tc_fence_before();
        mbar_arrive(bar_odrained + 8 * x);
        ph ^= 2u;
      }
      mbar_arrive(bar_itemfree + 8 * (k & 1u));                     // this thread is through with item k's record
      ph = ((ph + (uint32_t)my_n) & 1u) | (ph & 2u) | ((k + 1) << 2);
      c = nc; row_valid = nrow_valid;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_TIMEOUT, KID_ATTN_SM100, (int)blockIdx.x, -2);
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 9) { tc_fence_after(); tmem_dealloc(tmem_base, kTmemCols); }
}

// Explicit lists (the paper's controlled configurations): per target the index of the last context entry
// at or before its position (-1: none), per context entry the row of the fresh K/V that replaces it (-1:
// cached).  rt.tile_cu = prefix of the host bounds on the target counts, rt.bound_b = bounds on the context.
__global__ void build_list_maps_kernel(ReqTable rt, const int* __restrict__ ctx_pos, const int* __restrict__ ctx_cu,
                                       const int* __restrict__ tgt_pos, const int* __restrict__ tgt_cu,
                                       long long ctx_bound_total, int* __restrict__ limit, int* __restrict__ fresh_row,
                                       DeviceStatus* st) {
  const int B = rt.n_req;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long n_tgt_slots = rt.tile_cu[B];
  if (i < n_tgt_slots) {
    const int b = find_segment(rt.tile_cu, B, (int)i);
    const int rho = (int)i - rt.tile_cu[b];
    const int t0 = tgt_cu[b], nt = tgt_cu[b + 1] - t0;
    if (rho == 0 && (nt > rt.bound_a[b] || tgt_cu[0] != 0)) report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SM100, nt, tgt_cu[0]);
    if (rho < nt) {
      const int p = tgt_pos[t0 + rho];
      const int c0 = ctx_cu[b], nc = ctx_cu[b + 1] - c0;
      int lo = 0, hi = nc;                                   // first context entry with position > p
      while (lo < hi) { const int mid = (lo + hi) >> 1; if (ctx_pos[c0 + mid] <= p) lo = mid + 1; else hi = mid; }
      if (p < 0 || p >= rt.ctx_len[b]) { report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SM100, p, rt.ctx_len[b]); lo = 1; }
      limit[t0 + rho] = lo - 1;
    }
  } else if (i < n_tgt_slots + ctx_bound_total) {
    const long long x = i - n_tgt_slots;
    if (x < ctx_cu[B]) {
      int b = 0;
      while (b + 1 < B && x >= ctx_cu[b + 1]) ++b;
      const int p = ctx_pos[x];
      const int t0 = tgt_cu[b], nt = tgt_cu[b + 1] - t0;
      int lo = 0, hi = nt;
      while (lo < hi) { const int mid = (lo + hi) >> 1; if (tgt_pos[t0 + mid] < p) lo = mid + 1; else hi = mid; }
      fresh_row[x] = (lo < nt && tgt_pos[t0 + lo] == p) ? (t0 + lo) : -1;
    }
  }
}

// Test utility: one thread waits (bounded) on an mbarrier that nothing ever completes.  Exercises the
// give-up path of every kernel's waits without hanging anything: the wait expires after the limit,
// the abort flag is raised and RELAXKV_ERR_TIMEOUT lands in the device status word.
__global__ void wait_timeout_probe_kernel(DeviceStatus* st) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ volatile int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    fence_barrier_init();
    const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag);
    if (!ok && abort_flag) report(st, RELAXKV_ERR_TIMEOUT, KID_ATTN_SM100, -1, -1);
  }
}

constexpr int kCombineThreads = 128;
constexpr int kMaxCombineSplits = 1024;       // four warps x 4 KB of weights

// Merges the partial results of a context split: out = sum_s w_s O_s / sum_s w_s with w_s = exp(lse_s - max lse).
// One warp per (target row, query head); rows past the true target count are left alone.
__global__ void __launch_bounds__(kCombineThreads)
combine_splits_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse, int n_splits,
                      long long n_target_rows, int H, int D, const int* __restrict__ r_cu, int n_req,
                      uint16_t* __restrict__ out, float* __restrict__ lse_out) {
  // the splits' weights of this warp's (row, head): the lanes fetch the log-sum-exps side by side (a serial walk over
  // the splits would pay one memory latency per split), the sums below still run in split order
  __shared__ float wgt_s[kCombineThreads / 32][kMaxCombineSplits];
  const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long w = (long long)blockIdx.x * (kCombineThreads / 32) + wib;
  griddep_launch();
  griddep_wait();                               // the partial results come from the kernel before
  const long long rows_true = min((long long)(r_cu[n_req] - r_cu[0]), n_target_rows);
  if (w >= rows_true * H) return;
  const long long row = w / H;
  const int h = (int)(w - row * H);
  float mx = -INFINITY;
  for (int sp = lane; sp < n_splits; sp += 32) {
    const float l = part_lse[((long long)sp * n_target_rows + row) * H + h];
    wgt_s[wib][sp] = l;
    mx = fmaxf(mx, l);
  }
  mx = warp_reduce_max(mx);
  __syncwarp();
  for (int sp = lane; sp < n_splits; sp += 32) {
    const float l = wgt_s[wib][sp];
    wgt_s[wib][sp] = (l == -INFINITY || mx == -INFINITY) ? 0.f : __expf(l - mx);
  }
  __syncwarp();
  const int per = D / 32;                       // 2 or 4 consecutive floats per lane
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  float den = 0.f;
  const float* o = part_o + (row * H + h) * D + lane * per;
  const long long sp_stride = n_target_rows * H * D;
#pragma unroll 8
  for (int sp = 0; sp < n_splits; ++sp) {       // fixed order: reproducible
    const float wgt = wgt_s[wib][sp];
    den += wgt;
    const bool live = wgt > 0.f;                  // an empty split wrote no partial output: whatever is there is ignored
    if (per == 4) {
      const float4 v = *reinterpret_cast<const float4*>(o + sp * sp_stride);
      acc[0] = fmaf(wgt, live ? v.x : 0.f, acc[0]); acc[1] = fmaf(wgt, live ? v.y : 0.f, acc[1]);
      acc[2] = fmaf(wgt, live ? v.z : 0.f, acc[2]); acc[3] = fmaf(wgt, live ? v.w : 0.f, acc[3]);
    } else {
      const float2 v = *reinterpret_cast<const float2*>(o + sp * sp_stride);
      acc[0] = fmaf(wgt, live ? v.x : 0.f, acc[0]); acc[1] = fmaf(wgt, live ? v.y : 0.f, acc[1]);
    }
  }
  const float inv = den > 0.f ? 1.f / den : 0.f;
  uint16_t* optr = out + (row * H + h) * D + lane * per;
  for (int e = 0; e < per; e += 2) {
    __nv_bfloat162 h2 = __floats2bfloat162_rn(acc[e] * inv, acc[e + 1] * inv);
    *reinterpret_cast<uint32_t*>(optr + e) = *reinterpret_cast<uint32_t*>(&h2);
  }
  if (lane == 0 && lse_out) lse_out[(long long)h * n_target_rows + row] = den > 0.f ? mx + logf(den) : -INFINITY;
}

relaxkv_status launch_combine_splits(const float* part_o, const float* part_lse, int n_splits, long long n_target_rows, int H,
                                     int D, const int32_t* r_cu, int n_req, long long rows_bound, void* out, float* lse_out,
                                     cudaStream_t stream) {
  const long long warps = rows_bound * H;
  if (warps <= 0) return RELAXKV_OK;
  if (n_splits > kMaxCombineSplits) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  constexpr int wpb = kCombineThreads / 32;
  return cuda_ok(launch_chained(n_target_rows <= kChainedMaxRows, combine_splits_kernel, (unsigned)((warps + wpb - 1) / wpb), kCombineThreads, 0, stream, part_o,
                                part_lse, n_splits, (long long)n_target_rows, H, D, r_cu, n_req, static_cast<uint16_t*>(out), lse_out));
}

// ---- host side ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static std::atomic<EncodeTiledFn> cached{nullptr};
  EncodeTiledFn fn = cached.load(std::memory_order_acquire);
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess) {
      fn = reinterpret_cast<EncodeTiledFn>(p);
      cached.store(fn, std::memory_order_release);
    }
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
                                       cudaStream_t stream, int allow_empty = 0) {
  const int H = shape->n_q_heads, Hkv = shape->n_kv_heads, G = H / Hkv;
  const int tile_targets = kBM / G;
  const int B = shape->n_req;
  for (int b = 0; b < B; ++b)     // tile_cu counts the launch units per request: PAIRS of query tiles
    plan.rt.tile_cu[b + 1] = plan.rt.tile_cu[b] + (plan.rt.bound_a[b] + 2 * tile_targets - 1) / (2 * tile_targets);
  const long long grid = (long long)plan.rt.tile_cu[B] * Hkv;
  if (grid == 0) return RELAXKV_OK;
  if (grid > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  CUtensorMap tm_q, tm_k, tm_v;
  const uint64_t row_q = (uint64_t)H * D * 2, row_kv = (uint64_t)Hkv * D * 2;
  if (!make_map_3d(&tm_q, q_new, D, H, (uint64_t)n_target_rows, (uint64_t)D * 2, row_q, (uint32_t)G, (uint32_t)tile_targets) ||
      !make_map_3d(&tm_k, plan.k_base, D, Hkv, (uint64_t)plan.ctx_rows, plan.kv_head_stride_bytes, plan.kv_token_stride_bytes, 1u,
                   (uint32_t)kBN) ||
      !make_map_3d(&tm_v, plan.v_base, D, Hkv, (uint64_t)plan.ctx_rows, plan.kv_head_stride_bytes, plan.kv_token_stride_bytes, 1u,
                   (uint32_t)kBN))
    return RELAXKV_ERR_CUDA;
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  // the materialised context (K and V, all heads) against the 126 MB L2
  long long ctx_rows_used = 0;
  for (int b = 0; b < B; ++b) ctx_rows_used += plan.rt.bound_b[b];
  const int head_inner = (ctx_rows_used * (long long)row_kv * 2 <= (40ll << 20)) ? 1 : 0;
  const int sms = sm_count_of_current_device();
  if (sms <= 0) return RELAXKV_ERR_CUDA;
  // Context split.  A block's work is its pair's context length; with fewer blocks than a few waves of SMs (a query
  // prefill, a decode step, a layer with few targets, a short context) the longest pairs would run alone at the end,
  // so every pair's context is cut into pieces of at least four tiles until the launch has about four blocks per SM.
  long long max_tiles = 1;
  for (int b = 0; b < B; ++b) max_tiles = std::max<long long>(max_tiles, (plan.rt.bound_b[b] + kBN - 1) / kBN);
  long long n_splits = 1;
  const int forced = (shape->h_tuning && shape->h_tuning->attention_ctx_splits > 0) ? shape->h_tuning->attention_ctx_splits : 0;
  if (forced > 0) {
    n_splits = forced;
  } else if (grid < 4ll * sms) {
    n_splits = std::min<long long>(std::max<long long>(1, (grid < sms ? sms : 4ll * sms) / grid), std::max<long long>(1, max_tiles / 4));
  }
  n_splits = std::min<long long>(n_splits, kMaxCtxSplits);
  n_splits = std::min<long long>(n_splits, kSplitRowsCap / n_target_rows);   // partial slots: [split][row of the call]
  if (n_splits < 1) n_splits = 1;
  auto kern = attention_sm100_kernel<D>;
  static std::atomic<int> attr_done[kMaxDevices];          // per device: the opt-in to > 48 KB of dynamic shared memory
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RELAXKV_ERR_CUDA;
  if (!attr_done[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<D>::kDynamic) != cudaSuccess)
      return RELAXKV_ERR_CUDA;
    attr_done[dev].store(1, std::memory_order_release);
  }
  // Persistent form: where a block's work is short the turn-over between blocks is what there is to save (measured
  // 3 % at an 8K context; nothing at 32K, where the chip runs at its power cap either way).
  const relaxkv_tuning* tun = shape->h_tuning;
  const int want_persist = tun ? tun->attention_persistent : 0;
  if (n_splits == 1 && !plan.dense_ctx && (want_persist == 1 || (want_persist == 0 && max_tiles <= kPersistMaxTiles && grid > sms))) {
    auto pk = attention_persist_kernel<D>;
    static std::atomic<int> pattr_done[kMaxDevices];
    if (!pattr_done[dev].load(std::memory_order_acquire)) {
      if (cudaFuncSetAttribute(pk, cudaFuncAttributeMaxDynamicSharedMemorySize, PersistSmem<D>::kDynamic) != cudaSuccess)
        return RELAXKV_ERR_CUDA;
      pattr_done[dev].store(1, std::memory_order_release);
    }
    int* counter = reinterpret_cast<int*>(plan.split_lse);          // unused by a one-split call: the work counter
    if (cudaMemsetAsync(counter, 0, sizeof(int), stream) != cudaSuccess) return RELAXKV_ERR_CUDA;
    long long pgrid = std::min<long long>(grid, sms);
    if (tun && tun->attention_grid_blocks > 0) pgrid = std::min<long long>(grid, tun->attention_grid_blocks);
    RELAXKV_RANGE("attention_persist_kernel");
    pk<<<(unsigned)pgrid, kAttnThreads, PersistSmem<D>::kDynamic, stream>>>(
        tm_q, tm_k, tm_v, plan.rt, mode, allow_empty, head_inner, H, Hkv, tile_targets, shape->softmax_scale * kLog2eA,
        u_pos, u_cu, r_rank, r_cu_layer, n_target_rows, static_cast<uint16_t*>(out), lse_out, (int)grid, counter, st);
    return launch_ok();
  }
  RELAXKV_RANGE("attention_sm100_kernel");
  kern<<<dim3((unsigned)grid, (unsigned)n_splits), kAttnThreads, AttnSmem<D>::kDynamic, stream>>>(
      tm_q, tm_k, tm_v, plan.rt, mode, allow_empty, head_inner, plan.dense_ctx, H, Hkv, tile_targets, shape->softmax_scale * kLog2eA,
      u_pos, u_cu, r_rank, r_cu_layer, n_target_rows, static_cast<uint16_t*>(out), lse_out, plan.split_o, plan.split_lse, st);
  relaxkv_status rc = launch_ok();
  if (rc != RELAXKV_OK || n_splits == 1) return rc;
  return launch_combine_splits(plan.split_o, plan.split_lse, (int)n_splits, n_target_rows, H, D, r_cu_layer, B, plan.sum_targets,
                               out, lse_out, stream);
}

}  // namespace relaxkv

using namespace relaxkv;

extern "C" relaxkv_status relaxkv_sparse_ctx_attention(
    const relaxkv_shape* shape, relaxkv_ctx_mode mode, const relaxkv_cache_view* cache,
    const void* q_new, const void* k_new, const void* v_new,
    const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank, const int32_t* r_cu_layer,
    int64_t n_target_rows, const int32_t* h_max_targets, const int32_t* h_max_ctx,
    void* out, float* lse_out, void* workspace, size_t workspace_bytes, relaxkv_stream stream_) {
  RELAXKV_RANGE("relaxkv_sparse_ctx_attention");
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

extern "C" relaxkv_status relaxkv_debug_wait_timeout(relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_debug_wait_timeout");
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  wait_timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(st);
  return launch_ok();
}

extern "C" relaxkv_status relaxkv_list_attention(
    const relaxkv_shape* shape, const relaxkv_cache_view* cache,
    const void* q_new, const void* k_new, const void* v_new,
    const int32_t* ctx_pos, const int32_t* ctx_cu, const int32_t* tgt_pos, const int32_t* tgt_cu,
    int64_t n_target_rows, const int32_t* h_max_targets, const int32_t* h_max_ctx,
    void* out, float* lse_out, void* workspace, size_t workspace_bytes, relaxkv_stream stream_) {
  RELAXKV_RANGE("relaxkv_list_attention");
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if (!ctx_pos || !ctx_cu || !tgt_pos || !tgt_cu || !h_max_targets || !h_max_ctx || !workspace)
    return RELAXKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return RELAXKV_ERR_INVALID_ARG;
  const WsLayout ws = ws_layout(shape, 1);
  if (workspace_bytes < ws.total) return RELAXKV_ERR_WORKSPACE_TOO_SMALL;
  int* limit = reinterpret_cast<int*>(static_cast<char*>(workspace) + ws.list_limit);
  int* fresh = reinterpret_cast<int*>(static_cast<char*>(workspace) + ws.list_fresh);
  // 1. the two maps
  ReqTable rt;
  fill_req_table(rt, shape, nullptr, nullptr);
  long long tgt_total = 0, ctx_total = 0;
  for (int b = 0; b < shape->n_req; ++b) {
    if (h_max_targets[b] < 0 || h_max_targets[b] > shape->h_ctx_len[b] || h_max_ctx[b] < 0 ||
        h_max_ctx[b] > shape->h_ctx_len[b])
      return RELAXKV_ERR_INVALID_ARG;
    rt.bound_a[b] = h_max_targets[b];
    rt.bound_b[b] = h_max_ctx[b];
    tgt_total += h_max_targets[b];
    ctx_total += h_max_ctx[b];
    rt.tile_cu[b + 1] = (int)tgt_total;
  }
  if (tgt_total + ctx_total > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  if (tgt_total + ctx_total > 0) {
    const long long n = tgt_total + ctx_total;
    build_list_maps_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(rt, ctx_pos, ctx_cu, tgt_pos, tgt_cu, ctx_total,
                                                                          limit, fresh, st);
    if ((rc = launch_ok()) != RELAXKV_OK) return rc;
  }
  // 2. gather (fresh rows resolved through the map) and 3. the attention kernel with the limits as "ranks"
  AttnPlan plan;
  rc = prepare_attention(shape, RELAXKV_CTX_UNION, cache, q_new, k_new, v_new, ctx_pos, ctx_cu, limit, tgt_cu, n_target_rows,
                         h_max_targets, h_max_ctx, out, workspace, workspace_bytes, stream, plan, fresh);
  if (rc != RELAXKV_OK) return rc;
  if (shape->head_dim == 128)
    return launch_attention<128>(shape, RELAXKV_CTX_UNION, plan, q_new, ctx_pos, ctx_cu, limit, tgt_cu, n_target_rows, out,
                                 lse_out, stream, 1);
  return launch_attention<64>(shape, RELAXKV_CTX_UNION, plan, q_new, ctx_pos, ctx_cu, limit, tgt_cu, n_target_rows, out,
                              lse_out, stream, 1);
}

// Attention of given token positions over the cache's own causal prefix (cache only, no gather): the tensor maps
// cover the cache, a target's causal limit is its position.
extern "C" relaxkv_status relaxkv_cache_attention(
    const relaxkv_shape* shape, const relaxkv_cache_view* cache, const void* q_new,
    const int32_t* tgt_pos, const int32_t* tgt_cu, int64_t n_target_rows, const int32_t* h_max_targets,
    void* out, float* lse_out, void* workspace, size_t workspace_bytes, relaxkv_stream stream_) {
  RELAXKV_RANGE("relaxkv_cache_attention");
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if ((rc = check_cache(shape, cache, true)) != RELAXKV_OK) return rc;
  if (!q_new || !out || !tgt_pos || !tgt_cu || !h_max_targets || !workspace) return RELAXKV_ERR_INVALID_ARG;
  if (!aligned16(q_new) || !aligned16(out) || n_target_rows < 1) return RELAXKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return RELAXKV_ERR_INVALID_ARG;
  const WsLayout ws = ws_layout(shape, 1);
  if (workspace_bytes < ws.total) return RELAXKV_ERR_WORKSPACE_TOO_SMALL;
  AttnPlan plan;
  fill_req_table(plan.rt, shape, cache, nullptr);
  plan.sum_targets = 0;
  long long cache_rows = 0;
  for (int b = 0; b < shape->n_req; ++b) {
    if (h_max_targets[b] < 0 || h_max_targets[b] > shape->h_ctx_len[b]) return RELAXKV_ERR_INVALID_ARG;
    plan.rt.bound_a[b] = h_max_targets[b];
    plan.rt.bound_b[b] = shape->h_ctx_len[b];
    plan.sum_targets += h_max_targets[b];
    cache_rows = std::max<long long>(cache_rows, (long long)cache->h_req_token_offset[b] + shape->h_ctx_len[b]);
  }
  if (plan.sum_targets > 0x7fffffffLL || cache_rows > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  char* base = static_cast<char*>(workspace);
  plan.kctx = nullptr; plan.vctx = nullptr;
  plan.split_o = reinterpret_cast<float*>(base + ws.split_o);
  plan.split_lse = reinterpret_cast<float*>(base + ws.split_lse);
  plan.k_base = cache->k; plan.v_base = cache->v;
  plan.kv_head_stride_bytes = (unsigned long long)cache->head_stride * 2;
  plan.kv_token_stride_bytes = (unsigned long long)cache->token_stride * 2;
  plan.ctx_rows = cache_rows;
  plan.dense_ctx = 1;
  // one target per request at most (a decode step): the streaming kernel
  bool one_each = true;
  for (int b = 0; b < shape->n_req; ++b) one_each = one_each && h_max_targets[b] <= 1;
  if (one_each) return launch_decode_attention(shape, plan, q_new, tgt_pos, tgt_cu, n_target_rows, out, lse_out, stream);
  // lists: targets by position (their "rank" in the dense context), counts from tgt_cu; u_pos / u_cu are not read
  if (shape->head_dim == 128)
    return launch_attention<128>(shape, RELAXKV_CTX_UNION, plan, q_new, nullptr, nullptr, tgt_pos, tgt_cu, n_target_rows, out,
                                 lse_out, stream);
  return launch_attention<64>(shape, RELAXKV_CTX_UNION, plan, q_new, nullptr, nullptr, tgt_pos, tgt_cu, n_target_rows, out,
                              lse_out, stream);
}
