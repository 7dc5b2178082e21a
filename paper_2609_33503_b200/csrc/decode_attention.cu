// Attention of ONE token per request over the cache's causal prefix: the decode step that follows the repair loop in the
// paper's time-to-first-token region (reproducibility appendix).  The work is reading the request's K and V rows once
// (every cached byte meets G multiply-adds, G = query heads per KV head <= 16), so this is a streaming kernel: a block
// owns (request, KV head, a range of 128-key tiles), a producer lane streams the K and V tiles through a three-stage
// ring in shared memory by TMA (the cache's own tensor maps, 128-byte swizzle, this CTA only), and each of the eight
// consumer warps takes 16 keys of a tile.  With so few query rows the 128-row tcgen05 tile would be 4 % full and its
// per-step hand-overs would set the pace; a warp-level mma.sync.m16n8k16 holds the G rows in one 16-row fragment and
// keeps the loop at a few hundred instructions per 32 keys, which is all this HBM-bound step needs from the tensor
// cores: S = Q K^T (K fragments by ldmatrix from the swizzled tile), online softmax on the accumulator fragments,
// P (bf16) re-used as the A fragment, O += P V (V fragments by ldmatrix.trans).  The blocks of a (request, head) leave
// normalised partial results and their log-sum-exp; combine_splits_kernel (the same merge the tcgen05 kernel uses)
// adds them in a fixed order.  Every wait is bounded.
#include "attention_common.cuh"
#include "decode_attention.cuh"
#include "sm100_ptx.cuh"
#include <algorithm>
#include <atomic>

namespace relaxkv {

using namespace ptx;

bool make_map_3d(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_bytes,
                 uint64_t stride2_bytes, uint32_t b1, uint32_t b2);          // attention_sm100.cu

constexpr int kDecConsumers = 8;                      // consumer warps
constexpr int kDecThreads = (kDecConsumers + 1) * 32;
constexpr int kDecTile = 128;                         // keys per tile
constexpr int kDecKeysPerWarp = kDecTile / kDecConsumers;   // 16: two 8-key column tiles of S, one 16-key step of P V
constexpr int kDecStages = 3;
constexpr float kLog2eD = 1.4426950408889634f;
constexpr float kLn2D = 0.6931471805599453f;

template <int D>
struct DecSmem {
  static constexpr int kHalves = D / 64;
  static constexpr int kHalfBytes = kDecTile * 128;                   // 128 rows x 64 bf16, 128-byte swizzled
  static constexpr int kTileBytes = kHalves * kHalfBytes;
  static constexpr int kStageBytes = 2 * kTileBytes;                  // K tile | V tile
  static constexpr int kBar = kDecStages * kStageBytes;               // full[stages], empty[stages]
  static constexpr int kMisc = kBar + 16 * kDecStages;                // abort flag
  static constexpr int kTotal = kMisc + 16;
  static constexpr int kDynamic = kTotal + 1024;
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t* r, uint32_t smem_addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t* r, uint32_t smem_addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr) : "memory");
}
// D (16 x 8, fp32) += A (16 x 16 bf16, row) * B (16 x 8 bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int D, int GMAX>
__global__ void __launch_bounds__(kDecThreads, 1)
decode_attention_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                        const __grid_constant__ ReqTable rt, const uint16_t* __restrict__ q,
                        const int* __restrict__ tgt_pos, const int* __restrict__ tgt_cu, long long n_target_rows, int H, int Hkv,
                        float scale_log2, uint16_t* __restrict__ out, float* __restrict__ lse_out, float* __restrict__ part_o,
                        float* __restrict__ part_lse, DeviceStatus* st) {
  using L = DecSmem<D>;
  const int G = H / Hkv;
  const int b = blockIdx.z, hd = blockIdx.y, split = blockIdx.x, n_splits = gridDim.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  griddep_launch();
  griddep_wait();                          // q, the lists and the newest cache row come from the kernels before
  const int nr = tgt_cu[b + 1] - tgt_cu[b];
  if (nr <= 0) return;
  const long long row = (long long)tgt_cu[b] - tgt_cu[0];
  if (nr > rt.bound_a[b] || nr > 1 || row >= n_target_rows) {      // more targets than the host bound (one): touch nothing
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SIMT, nr, (int)row);
    return;
  }
  const int pos = tgt_pos[tgt_cu[b]];
  if (pos < 0 || pos >= rt.ctx_len[b]) {
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_BAD_INDEX, KID_ATTN_SIMT, pos, rt.ctx_len[b]);
    return;
  }
  if (*reinterpret_cast<volatile int*>(&st->status) == RELAXKV_ERR_TIMEOUT) return;   // drain after a timeout
  const int n_keys = pos + 1;
  const int n_tiles = (n_keys + kDecTile - 1) / kDecTile;
  const int per = (n_tiles + n_splits - 1) / n_splits;
  const int t0 = split * per, t1 = min(n_tiles, t0 + per);            // this block's tiles

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_full = base + L::kBar, bar_empty = bar_full + 8 * kDecStages;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::kMisc);
  __shared__ __align__(16) float q_s[GMAX][D];                      // the query heads of this KV head
  __shared__ float m_s[kDecConsumers][GMAX], z_s[kDecConsumers][GMAX];
  // the warps' partial outputs for the merge take the ring's place once every tile has been consumed
  float (*o_s)[GMAX][D] = reinterpret_cast<float (*)[GMAX][D]>(base_ptr);
  static_assert(kDecConsumers * GMAX * D * 4 <= kDecStages * DecSmem<D>::kStageBytes, "merge buffer fits the ring");
  if (threadIdx.x == 0) {
    for (int s = 0; s < kDecStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, kDecConsumers); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  for (int i = threadIdx.x; i < GMAX * D; i += kDecThreads) {
    const int g = i / D, d = i - g * D;
    q_s[g][d] = (g < G) ? bf16_bits_to_float(q[(row * H + hd * G + g) * D + d]) : 0.f;     // exact; the scale goes on S
  }
  __syncthreads();

  float frag_m[2] = {-INFINITY, -INFINITY}, frag_z[2] = {0.f, 0.f}, frag_o[D / 8][4];     // a consumer warp's result (fragment layout)
#pragma unroll
  for (int d = 0; d < D / 8; ++d) { frag_o[d][0] = frag_o[d][1] = frag_o[d][2] = frag_o[d][3] = 0.f; }
  if (warp == kDecConsumers) {
    // ================= producer =================
    if (lane == 0) {
      prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
      const int row0 = (int)rt.tok_off[b];
      for (int t = t0, it = 0; t < t1; ++t, ++it) {
        const int s = it % kDecStages;
        if (it >= kDecStages && !mbar_wait(bar_empty + 8 * s, (uint32_t)((it / kDecStages) - 1) & 1, abort_flag)) break;
        mbar_expect_tx(bar_full + 8 * s, L::kStageBytes);
        const uint32_t dst = base + s * L::kStageBytes;
        for (int hf = 0; hf < L::kHalves; ++hf) {
          tma_load_3d(dst + hf * L::kHalfBytes, &tm_k, bar_full + 8 * s, hf * 64, hd, row0 + t * kDecTile);
          tma_load_3d(dst + L::kTileBytes + hf * L::kHalfBytes, &tm_v, bar_full + 8 * s, hf * 64, hd, row0 + t * kDecTile);
        }
      }
    }
  } else {
    // ================= consumers =================
    const int gid = lane >> 2, tig = lane & 3;                        // fragment coordinates: row gid (and gid + 8), column pair tig
    // Q as A fragments, one per 16 dims: rows = the G query heads (zero beyond)
    uint32_t qa[D / 16][4];
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {                                // columns ks*16 + tig*2 (+8 for h2 = 1)
        const int col = ks * 16 + h2 * 8 + tig * 2;
        const __nv_bfloat162 lo = __floats2bfloat162_rn(q_s[gid % GMAX][col] * (gid < GMAX ? 1.f : 0.f), q_s[gid % GMAX][col + 1] * (gid < GMAX ? 1.f : 0.f));
        const __nv_bfloat162 hi = (GMAX > 8) ? __floats2bfloat162_rn(q_s[(gid + 8) % GMAX][col], q_s[(gid + 8) % GMAX][col + 1])
                                             : __floats2bfloat162_rn(0.f, 0.f);
        qa[ks][h2 * 2] = *reinterpret_cast<const uint32_t*>(&lo);
        qa[ks][h2 * 2 + 1] = *reinterpret_cast<const uint32_t*>(&hi);
      }
    }
    float m_r[2] = {-INFINITY, -INFINITY}, z_r[2] = {0.f, 0.f};       // rows gid and gid + 8
    float oacc[D / 8][4];
#pragma unroll
    for (int d = 0; d < D / 8; ++d) { oacc[d][0] = oacc[d][1] = oacc[d][2] = oacc[d][3] = 0.f; }
    bool ok = true;
    for (int t = t0, it = 0; t < t1 && ok; ++t, ++it) {
      const int s = it % kDecStages;
      ok = mbar_wait(bar_full + 8 * s, (uint32_t)(it / kDecStages) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const uint32_t kt = base + s * L::kStageBytes, vt = kt + L::kTileBytes;
      constexpr int KPW = kDecKeysPerWarp;
      const int c = t * kDecTile + warp * KPW;                        // first key of this warp's share of the tile
      const int n_here = min(KPW, n_keys - c);                        // its keys inside the causal prefix
      if (n_here > 0) {
        if (n_here < KPW) {
          // V rows past the prefix belong to nobody (they may hold NaN, and 0 x NaN = NaN on the tensor core): zero them
          uint8_t* vrows = base_ptr + s * L::kStageBytes + L::kTileBytes;
          for (int i = lane; i < (KPW - n_here) * (D / 8); i += 32) {
            const int r = warp * KPW + n_here + i / (D / 8), c16 = i % (D / 8);
            *reinterpret_cast<uint4*>(vrows + (c16 >> 3) * L::kHalfBytes + r * 128 + (((c16 & 7) ^ (r & 7)) << 4)) = make_uint4(0, 0, 0, 0);
          }
          __syncwarp();
        }
        // ---- S = Q K^T: 8-key column tiles ----
        float sacc[KPW / 8][4];
#pragma unroll
        for (int j = 0; j < KPW / 8; ++j) {
          sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f;
          const int r = warp * KPW + j * 8 + (lane & 7);               // the key row whose address this lane supplies
#pragma unroll
          for (int q4 = 0; q4 < D / 32; ++q4) {
            const int c16 = 4 * q4 + (lane >> 3);                     // dims [32 q4 + 8 (lane / 8), + 8)
            uint32_t kb[4];
            ldmatrix_x4(kb, kt + (c16 >> 3) * L::kHalfBytes + r * 128 + (((c16 & 7) ^ (r & 7)) << 4));
            mma_bf16_16816(sacc[j], qa[2 * q4], kb[0], kb[1]);
            mma_bf16_16816(sacc[j], qa[2 * q4 + 1], kb[2], kb[3]);
          }
        }
        // ---- online softmax on the fragments: this lane holds, of rows gid and gid + 8, keys 8 j + 2 tig (+1) ----
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < KPW / 8; ++j) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int key = j * 8 + tig * 2 + (e & 1);
            sacc[j][e] = (key < n_here) ? sacc[j][e] * scale_log2 : -INFINITY;
            mx[e >> 1] = fmaxf(mx[e >> 1], sacc[j][e]);
          }
        }
        float alpha[2];
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
          mx[rr] = fmaxf(mx[rr], __shfl_xor_sync(0xffffffffu, mx[rr], 1));
          mx[rr] = fmaxf(mx[rr], __shfl_xor_sync(0xffffffffu, mx[rr], 2));
          const float m_new = fmaxf(m_r[rr], mx[rr]);                  // finite: key 0 of the chunk is inside the prefix
          alpha[rr] = exp2f(m_r[rr] - m_new);                          // 0 on the first chunk
          m_r[rr] = m_new;
          z_r[rr] *= alpha[rr];
        }
        uint32_t pa[KPW / 16][4];                                      // P as A fragments, 16 keys each
#pragma unroll
        for (int j = 0; j < KPW / 8; ++j) {
          float p[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            p[e] = exp2f(sacc[j][e] - m_r[e >> 1]);
            z_r[e >> 1] += p[e];                                       // this lane's keys; the quad is added up at the end
          }
          const __nv_bfloat162 p01 = __floats2bfloat162_rn(p[0], p[1]), p23 = __floats2bfloat162_rn(p[2], p[3]);
          pa[j >> 1][(j & 1) * 2] = *reinterpret_cast<const uint32_t*>(&p01);
          pa[j >> 1][(j & 1) * 2 + 1] = *reinterpret_cast<const uint32_t*>(&p23);
        }
#pragma unroll
        for (int d = 0; d < D / 8; ++d) { oacc[d][0] *= alpha[0]; oacc[d][1] *= alpha[0]; oacc[d][2] *= alpha[1]; oacc[d][3] *= alpha[1]; }
        // ---- O += P V: V fragments transposed out of the tile, two 8-dim column tiles per load ----
#pragma unroll
        for (int ks = 0; ks < KPW / 16; ++ks) {
          const int r = warp * KPW + ks * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
          for (int dp = 0; dp < D / 16; ++dp) {
            const int c16 = 2 * dp + (lane >> 4);
            uint32_t vb[4];
            ldmatrix_x4_trans(vb, vt + (c16 >> 3) * L::kHalfBytes + r * 128 + (((c16 & 7) ^ (r & 7)) << 4));
            mma_bf16_16816(oacc[2 * dp], pa[ks], vb[0], vb[1]);
            mma_bf16_16816(oacc[2 * dp + 1], pa[ks], vb[2], vb[3]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty + 8 * s);                  // this warp is through with the stage
    }
    // hand the rows' results to the merge in the form the code below expects: m[g], z[g] per lane-0 value, o per (g, d)
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      z_r[rr] += __shfl_xor_sync(0xffffffffu, z_r[rr], 1);
      z_r[rr] += __shfl_xor_sync(0xffffffffu, z_r[rr], 2);
    }
    frag_m[0] = m_r[0]; frag_m[1] = m_r[1]; frag_z[0] = z_r[0]; frag_z[1] = z_r[1];
#pragma unroll
    for (int d = 0; d < D / 8; ++d) { frag_o[d][0] = oacc[d][0]; frag_o[d][1] = oacc[d][1]; frag_o[d][2] = oacc[d][2]; frag_o[d][3] = oacc[d][3]; }
  }
  __syncthreads();                                                    // every tile consumed: the ring is free
  if (warp < kDecConsumers && !*abort_flag) {
    // ---- this warp's result for the merge: rows gid (and gid + 8) of the fragments are query heads ----
    const int gid = lane >> 2, tig = lane & 3;
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int g = gid + 8 * rr;
      if (g < G) {
        if (tig == 0) { m_s[warp][g] = frag_m[rr]; z_s[warp][g] = frag_z[rr]; }
#pragma unroll
        for (int d = 0; d < D / 8; ++d) {
          o_s[warp][g][d * 8 + tig * 2] = frag_o[d][2 * rr];
          o_s[warp][g][d * 8 + tig * 2 + 1] = frag_o[d][2 * rr + 1];
        }
      }
    }
  }
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_TIMEOUT, KID_ATTN_SIMT, (int)blockIdx.x, (int)blockIdx.y);
    const uint64_t tw = global_timer_ns();                            // copies still in flight: let them land
    while (global_timer_ns() - tw < 200000ull) __nanosleep(1000);
    return;
  }
  for (int i = threadIdx.x; i < G * D; i += kDecThreads) {
    const int g = i / D, d = i - g * D;
    float mb = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecConsumers; ++w) mb = fmaxf(mb, m_s[w][g]);
    float acc = 0.f, zb = 0.f;
    if (mb > -INFINITY) {
#pragma unroll
      for (int w = 0; w < kDecConsumers; ++w) {                        // fixed order
        const float wgt = (m_s[w][g] > -INFINITY) ? exp2f(m_s[w][g] - mb) : 0.f;
        acc = fmaf(o_s[w][g][d], wgt, acc);
        zb = fmaf(z_s[w][g], wgt, zb);
      }
    }
    const bool none = !(zb > 0.f);                                     // this block's key range is empty
    const float val = none ? 0.f : acc / zb;
    const float lse = none ? -INFINITY : (mb + log2f(zb)) * kLn2D;
    const int h = hd * G + g;
    if (n_splits == 1) {
      const __nv_bfloat16 hv = __float2bfloat16(val);
      out[(row * H + h) * D + d] = *reinterpret_cast<const uint16_t*>(&hv);
      if (d == 0 && lse_out) lse_out[(long long)h * n_target_rows + row] = lse;
    } else {
      const long long slot = ((long long)split * n_target_rows + row) * H + h;
      part_o[slot * D + d] = val;
      if (d == 0) part_lse[slot] = lse;
    }
  }
}

template <int D, int GMAX>
static relaxkv_status launch_g(const CUtensorMap& tm_k, const CUtensorMap& tm_v, const AttnPlan& plan, dim3 grid, const void* q,
                               const int32_t* tgt_pos, const int32_t* tgt_cu, int64_t n_target_rows, int H, int Hkv, float scale_log2,
                               void* out, float* lse_out, DeviceStatus* st, cudaStream_t stream) {
  static std::atomic<int> attr_done[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RELAXKV_ERR_CUDA;
  auto kern = decode_attention_kernel<D, GMAX>;
  if (!attr_done[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, DecSmem<D>::kDynamic) != cudaSuccess) return RELAXKV_ERR_CUDA;
    attr_done[dev].store(1, std::memory_order_release);
  }
  return cuda_ok(launch_chained(true, kern, grid, kDecThreads, DecSmem<D>::kDynamic, stream, tm_k, tm_v, plan.rt,
                                static_cast<const uint16_t*>(q), tgt_pos, tgt_cu, (long long)n_target_rows, H, Hkv, scale_log2,
                                static_cast<uint16_t*>(out), lse_out, plan.split_o, plan.split_lse, st));
}

template <int D>
static relaxkv_status launch_d(const relaxkv_shape* shape, const AttnPlan& plan, const void* q, const int32_t* tgt_pos,
                               const int32_t* tgt_cu, int64_t n_target_rows, void* out, float* lse_out, cudaStream_t stream) {
  const int H = shape->n_q_heads, Hkv = shape->n_kv_heads, G = H / Hkv, B = shape->n_req;
  const int sms = sm_count_of_current_device();
  if (sms <= 0) return RELAXKV_ERR_CUDA;
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  CUtensorMap tm_k, tm_v;
  if (!make_map_3d(&tm_k, plan.k_base, D, Hkv, (uint64_t)plan.ctx_rows, plan.kv_head_stride_bytes, plan.kv_token_stride_bytes, 1u,
                   (uint32_t)kDecTile) ||
      !make_map_3d(&tm_v, plan.v_base, D, Hkv, (uint64_t)plan.ctx_rows, plan.kv_head_stride_bytes, plan.kv_token_stride_bytes, 1u,
                   (uint32_t)kDecTile))
    return RELAXKV_ERR_CUDA;
  int max_ctx = 1;
  for (int b = 0; b < B; ++b) max_ctx = std::max(max_ctx, shape->h_ctx_len[b]);
  const int max_tiles = (max_ctx + kDecTile - 1) / kDecTile;
  // one block per SM (the ring takes its shared memory): one wave of blocks, at least two tiles each, as many
  // splits as the split workspace has slots for
  long long n_splits = std::max<long long>(1, sms / std::max(1, B * Hkv));
  n_splits = std::min<long long>(n_splits, std::max(1, max_tiles / 2));
  if (shape->h_tuning && shape->h_tuning->attention_ctx_splits > 0) n_splits = shape->h_tuning->attention_ctx_splits;
  n_splits = std::min<long long>(n_splits, kSplitRowsCap / std::max<long long>(1, n_target_rows));
  n_splits = std::max<long long>(1, std::min<long long>(n_splits, 1024));
  RELAXKV_RANGE("decode_attention_kernel");
  const dim3 grid((unsigned)n_splits, (unsigned)Hkv, (unsigned)B);
  const float scale_log2 = shape->softmax_scale * kLog2eD;
  relaxkv_status rc;
  if (G <= 4) rc = launch_g<D, 4>(tm_k, tm_v, plan, grid, q, tgt_pos, tgt_cu, n_target_rows, H, Hkv, scale_log2, out, lse_out, st, stream);
  else if (G <= 8) rc = launch_g<D, 8>(tm_k, tm_v, plan, grid, q, tgt_pos, tgt_cu, n_target_rows, H, Hkv, scale_log2, out, lse_out, st, stream);
  else rc = launch_g<D, 16>(tm_k, tm_v, plan, grid, q, tgt_pos, tgt_cu, n_target_rows, H, Hkv, scale_log2, out, lse_out, st, stream);
  if (rc != RELAXKV_OK || n_splits == 1) return rc;
  return launch_combine_splits(plan.split_o, plan.split_lse, (int)n_splits, n_target_rows, H, shape->head_dim, tgt_cu, B,
                               plan.sum_targets, out, lse_out, stream);
}

relaxkv_status launch_decode_attention(const relaxkv_shape* shape, const AttnPlan& plan, const void* q, const int32_t* tgt_pos,
                                       const int32_t* tgt_cu, int64_t n_target_rows, void* out, float* lse_out,
                                       cudaStream_t stream) {
  if (shape->head_dim == 128) return launch_d<128>(shape, plan, q, tgt_pos, tgt_cu, n_target_rows, out, lse_out, stream);
  return launch_d<64>(shape, plan, q, tgt_pos, tgt_cu, n_target_rows, out, lse_out, stream);
}

}  // namespace relaxkv
