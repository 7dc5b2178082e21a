// y = x W^T (+ residual) on the Blackwell tensor cores: the projections of the active targets' block work
// (Algorithm 1, steps 16 and 20).  x [M, K], W [N, K] (the [out, in] layout), y [M, N], bf16 with fp32
// accumulation in TMEM.  Persistent kernel, one CTA per SM: CTA tile 128 x 256, K blocks of 64 through a
// 4-stage TMA ring (128-byte swizzle) that runs on across tiles, one MMA issuer thread (tcgen05.mma M=128,
// N=256, K=16), two 256-column accumulators in TMEM so that the four epilogue warps (thread = row = TMEM
// lane) drain tile i while the tensor pipe works on tile i+1.  Tiles are walked in groups of 16 row tiles so
// that a wave's working set (x rows + W rows) stays in L2.
#include "common.cuh"
#include "gemm_skinny.cuh"
#include "gemv.cuh"
#include "sm100_ptx.cuh"
#include <algorithm>

namespace relaxkv {

using namespace ptx;

bool make_map_3d(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_bytes,
                 uint64_t stride2_bytes, uint32_t b1, uint32_t b2);          // attention_sm100.cu

constexpr int kGemmBM = 128, kGemmBN = 256, kGemmBK = 64, kGemmStages = 4, kGemmThreads = 192, kGemmGroupM = 16;
constexpr int kGemmABytes = kGemmBM * kGemmBK * 2, kGemmBBytes = kGemmBN * kGemmBK * 2;
constexpr int kGemmStageBytes = kGemmABytes + kGemmBBytes;
constexpr int kGemmBars = 2 * kGemmStages + 4;           // full, empty per stage; accumulator full, empty x 2
constexpr int kGemmSmem = kGemmStages * kGemmStageBytes + 8 * kGemmBars + 16 + 1024;

// Output columns split into up to three buffers of their own (the stacked Q/K/V projection): segment i = columns
// [col0[i], col0[i + 1]) goes to the row-major buffer y[i] of that width.  n == 0: one buffer (the kernel's y).  The
// boundaries are multiples of 32, the width of an epilogue chunk.
struct GemmSegs {
  uint16_t* y[3];
  int col0[4];
  int n;
};
// where the 32-column chunk that starts at output column col0 of `row` goes: base pointer of its first element
__device__ __forceinline__ uint16_t* chunk_ptr(const GemmSegs& segs, uint16_t* y, long long row, int N, int col0) {
  if (segs.n == 0) return y + row * N + col0;
  int sg = 0;
  while (sg + 1 < segs.n && col0 >= segs.col0[sg + 1]) ++sg;
  return segs.y[sg] + row * (segs.col0[sg + 1] - segs.col0[sg]) + (col0 - segs.col0[sg]);
}

__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_sm100_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                  long long M, int N, int K, uint16_t* __restrict__ y, const uint16_t* __restrict__ residual,
                  int swiglu, const __grid_constant__ GemmSegs segs, DeviceStatus* st) {
  const int tiles_m = (int)((M + kGemmBM - 1) / kGemmBM), tiles_n = (N + kGemmBN - 1) / kGemmBN;
  const long long n_tiles = (long long)tiles_m * tiles_n;
  if (*reinterpret_cast<volatile int*>(&st->status) == RELAXKV_ERR_TIMEOUT) return;
  // tile t of the grouped order: kGemmGroupM row tiles x all column tiles at a time
  auto tile_of = [&](long long t, int& tm, int& tn) {
    const int per_group = kGemmGroupM * tiles_n;
    const int group = (int)(t / per_group), first_m = group * kGemmGroupM;
    const int group_m = min(tiles_m - first_m, kGemmGroupM);
    const int r = (int)(t - (long long)group * per_group);
    tm = first_m + r % group_m;
    tn = r / group_m;
  };

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar0 = base + kGemmStages * kGemmStageBytes;
  const uint32_t bar_full = bar0, bar_empty = bar0 + 8 * kGemmStages;
  const uint32_t bar_acc_full = bar0 + 16 * kGemmStages, bar_acc_empty = bar_acc_full + 16;     // [2] each
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kGemmStages * kGemmStageBytes + 8 * kGemmBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(const_cast<uint32_t*>(tmem_slot) + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kGemmStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bar_acc_full + 8 * a, 1); mbar_init(bar_acc_empty + 8 * a, 128); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 5) { tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int n_k = (K + kGemmBK - 1) / kGemmBK;

  if (warp == 4) {
    // ---- TMA producer: the ring index runs on from tile to tile ----
    if (lane == 0) {
      prefetch_tensormap(&tm_a); prefetch_tensormap(&tm_b);
      long long it = 0;
      for (long long t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        int tm, tn;
        tile_of(t, tm, tn);
        bool ok = true;
        for (int kt = 0; kt < n_k; ++kt, ++it) {
          const int s = (int)(it % kGemmStages);
          if (it >= kGemmStages && !(ok = mbar_wait(bar_empty + 8 * s, (uint32_t)((it / kGemmStages) - 1) & 1, abort_flag))) break;
          mbar_expect_tx(bar_full + 8 * s, kGemmStageBytes);
          tma_load_3d(base + s * kGemmStageBytes, &tm_a, bar_full + 8 * s, kt * kGemmBK, tm * kGemmBM, 0);
          tma_load_3d(base + s * kGemmStageBytes + kGemmABytes, &tm_b, bar_full + 8 * s, kt * kGemmBK, tn * kGemmBN, 0);
        }
        if (!ok) break;
      }
    }
  } else if (warp == 5) {
    // ---- MMA issuer: accumulator i & 1 for the CTA's i-th tile ----
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(kGemmBM, kGemmBN, 0);
      bool ok = true;
      long long it = 0;
      int i = 0;
      for (long long t = blockIdx.x; ok && t < n_tiles; t += gridDim.x, ++i) {
        const int a = i & 1;
        if (i >= 2 && !(ok = mbar_wait(bar_acc_empty + 8 * a, (uint32_t)((i >> 1) - 1) & 1, abort_flag))) break;
        tc_fence_after();
        for (int kt = 0; kt < n_k; ++kt, ++it) {
          const int s = (int)(it % kGemmStages);
          if (!(ok = mbar_wait(bar_full + 8 * s, (uint32_t)(it / kGemmStages) & 1, abort_flag))) break;
          tc_fence_after();
          const uint32_t sa = base + s * kGemmStageBytes;
          mma_ss_4steps(tmem_base + a * kGemmBN, desc_lo(sa, 16), desc_lo(sa + kGemmABytes, 16), desc_hi_sw128(1024), idesc,
                        kt > 0 ? 1u : 0u);
          mma_commit(bar_empty + 8 * s);
        }
        if (ok) mma_commit(bar_acc_full + 8 * a);
      }
    }
  } else {
    // ---- epilogue: thread = output row = TMEM lane ----
    int i = 0;
    for (long long t = blockIdx.x; t < n_tiles; t += gridDim.x, ++i) {
      const int a = i & 1;
      int tm, tn;
      tile_of(t, tm, tn);
      bool ok = mbar_wait(bar_acc_full + 8 * a, (uint32_t)(i >> 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const long long row = (long long)tm * kGemmBM + warp * 32 + lane;
      const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16) + a * kGemmBN;
      if (swiglu) {
        // the tile's columns are [128 gate | 128 up] of the same 128 intermediate features (weight rows arranged so
        // by the caller): out[row, tn * 128 + j] = silu(gate_j) * up_j, fp32, one rounding to bf16
        const int n_inter = N / 2;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t g[32], u[32];
          tmem_ld32(t_lane + c * 32, g);
          tmem_ld32(t_lane + 128 + c * 32, u);
          tmem_wait_ld();
          const int col0 = tn * 128 + c * 32;
          if (row < M && col0 < n_inter) {
            const long long off = row * n_inter + col0;
#pragma unroll
            for (int i8 = 0; i8 < 32; i8 += 8) {
              uint32_t w[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float g0 = __uint_as_float(g[i8 + 2 * e]), g1 = __uint_as_float(g[i8 + 2 * e + 1]);
                __nv_bfloat162 h2 = __floats2bfloat162_rn(g0 / (1.f + __expf(-g0)) * __uint_as_float(u[i8 + 2 * e]),
                                                          g1 / (1.f + __expf(-g1)) * __uint_as_float(u[i8 + 2 * e + 1]));
                w[e] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(y + off + i8) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      } else
#pragma unroll 1
      for (int c = 0; c < kGemmBN / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(t_lane + c * 32, v);
        tmem_wait_ld();
        const int col0 = tn * kGemmBN + c * 32;
        if (row < M && col0 < N) {
          const long long off = row * N + col0;
          uint16_t* yc = chunk_ptr(segs, y, row, N, col0);
#pragma unroll
          for (int i8 = 0; i8 < 32; i8 += 8) {
            if (col0 + i8 < N) {                                 // N is a multiple of 8
              float f[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[i8 + e]);
              if (residual != nullptr) {
                const uint4 r = __ldg(reinterpret_cast<const uint4*>(residual + off + i8));
                const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) { f[2 * e] += __uint_as_float(rw[e] << 16); f[2 * e + 1] += __uint_as_float(rw[e] & 0xffff0000u); }
              }
              uint32_t w[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                __nv_bfloat162 h2 = __floats2bfloat162_rn(f[2 * e], f[2 * e + 1]);
                w[e] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(yc + i8) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      }
      // the accumulator has been read out: the MMA warp may overwrite it
      tc_fence_before();
      mbar_arrive(bar_acc_empty + 8 * a);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_TIMEOUT, KID_GEMM_SM100, (int)blockIdx.x, 0);
    const uint64_t tw = global_timer_ns();
    while (global_timer_ns() - tw < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 5) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

// ---- the same GEMM on SM pairs (cta_group::2): 256 x 256 tiles per cluster, each CTA stages its 128 A rows and 128 of
// the tile's 256 B rows per K block (32 KB: six stages), one MMA instruction stream drives both tensor cores ----
constexpr int kPairStages = 6;
constexpr int kPairStageBytes = kGemmABytes + kGemmBBytes / 2;
constexpr int kPairBarsTotal = 2 * kPairStages + 4;
constexpr int kPairSmem = kPairStages * kPairStageBytes + 8 * kPairBarsTotal + 16 + 1024;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
gemm_pair_sm100_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                  long long M, int N, int K, uint16_t* __restrict__ y, const uint16_t* __restrict__ residual,
                  int swiglu, const __grid_constant__ GemmSegs segs, DeviceStatus* st) {
  // a cluster of two CTAs computes 256 x 256 output tiles: CTA rank r holds rows [128 r, 128 r + 128) of the tile's A
  // rows and of its B rows (= output columns), the leader's MMA thread drives both SMs (M = 256), every CTA drains
  // its own 128 x 256 accumulator.  tiles_m counts 256-row tiles here.  (No early exit after a timeout: the two
  // CTAs of a cluster must leave together.)
  const uint32_t cr = cluster_ctarank();
  const int tiles_m = (int)((M + 2 * kGemmBM - 1) / (2 * kGemmBM)), tiles_n = (N + kGemmBN - 1) / kGemmBN;
  const long long n_tiles = (long long)tiles_m * tiles_n;
  const long long first_tile = blockIdx.x >> 1, tile_step = gridDim.x >> 1;
  // tile t of the grouped order: kGemmGroupM row tiles x all column tiles at a time
  auto tile_of = [&](long long t, int& tm, int& tn) {
    const int per_group = kGemmGroupM * tiles_n;
    const int group = (int)(t / per_group), first_m = group * kGemmGroupM;
    const int group_m = min(tiles_m - first_m, kGemmGroupM);
    const int r = (int)(t - (long long)group * per_group);
    tm = first_m + r % group_m;
    tn = r / group_m;
  };

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar0 = base + kPairStages * kPairStageBytes;
  const uint32_t bar_full = bar0, bar_empty = bar0 + 8 * kPairStages;
  const uint32_t bar_acc_full = bar0 + 16 * kPairStages, bar_acc_empty = bar_acc_full + 16;     // [2] each
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kPairStages * kPairStageBytes + 8 * kPairBarsTotal);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(const_cast<uint32_t*>(tmem_slot) + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    // the leader's "landed" barriers also count one arrival relayed from the peer, its "accumulator drained" barriers
    // the epilogue threads of both CTAs
    const uint32_t n_cta = (cr == 0) ? 2u : 1u;
    for (int s = 0; s < kPairStages; ++s) { mbar_init(bar_full + 8 * s, n_cta); mbar_init(bar_empty + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(bar_acc_full + 8 * a, 1); mbar_init(bar_acc_empty + 8 * a, 256); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 5) { tmem_alloc2(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512); tmem_relinquish2(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int n_k = (K + kGemmBK - 1) / kGemmBK;

  if (warp == 4) {
    // ---- TMA producer: the ring index runs on from tile to tile ----
    if (lane == 0) {
      prefetch_tensormap(&tm_a); prefetch_tensormap(&tm_b);
      long long it = 0;
      for (long long t = first_tile; t < n_tiles; t += tile_step) {
        int tm, tn;
        tile_of(t, tm, tn);
        bool ok = true;
        for (int kt = 0; kt < n_k; ++kt, ++it) {
          const int s = (int)(it % kPairStages);
          if (it >= kPairStages && !(ok = mbar_wait(bar_empty + 8 * s, (uint32_t)((it / kPairStages) - 1) & 1, abort_flag))) break;
          mbar_expect_tx(bar_full + 8 * s, kPairStageBytes);
          tma_load_3d(base + s * kPairStageBytes, &tm_a, bar_full + 8 * s, kt * kGemmBK, (2 * tm + (int)cr) * kGemmBM, 0);
          tma_load_3d(base + s * kPairStageBytes + kGemmABytes, &tm_b, bar_full + 8 * s, kt * kGemmBK,
                      tn * kGemmBN + (int)cr * (kGemmBN / 2), 0);
        }
        if (!ok) break;
      }
    }
  } else if (warp == 5) {
    // ---- leader: MMA issuer for both SMs (accumulator i & 1 for the cluster's i-th tile); peer: relays "stage landed" ----
    if (lane == 0 && cr != 0) {
      bool ok = true;
      long long it = 0;
      for (long long t = first_tile; ok && t < n_tiles; t += tile_step) {
        for (int kt = 0; kt < n_k; ++kt, ++it) {
          const int s = (int)(it % kPairStages);
          if (!(ok = mbar_wait(bar_full + 8 * s, (uint32_t)(it / kPairStages) & 1, abort_flag))) break;
          mbar_arrive_remote(mapa_shared(bar_full + 8 * s, 0));
        }
      }
    }
    if (lane == 0 && cr == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(2 * kGemmBM, kGemmBN, 0);
      bool ok = true;
      long long it = 0;
      int i = 0;
      for (long long t = first_tile; ok && t < n_tiles; t += tile_step, ++i) {
        const int a = i & 1;
        if (i >= 2 && !(ok = mbar_wait_cluster(bar_acc_empty + 8 * a, (uint32_t)((i >> 1) - 1) & 1, abort_flag))) break;
        tc_fence_after();
        for (int kt = 0; kt < n_k; ++kt, ++it) {
          const int s = (int)(it % kPairStages);
          if (!(ok = mbar_wait_cluster(bar_full + 8 * s, (uint32_t)(it / kPairStages) & 1, abort_flag))) break;
          tc_fence_after();
          const uint32_t sa = base + s * kPairStageBytes;
          mma2_ss_4steps(tmem_base + a * kGemmBN, desc_lo(sa, 16), desc_lo(sa + kGemmABytes, 16), desc_hi_sw128(1024), idesc,
                         kt > 0 ? 1u : 0u);
          mma_commit2_mc(bar_empty + 8 * s, 3);
        }
        if (ok) mma_commit2_mc(bar_acc_full + 8 * a, 3);
      }
    }
  } else {
    // ---- epilogue: thread = output row = TMEM lane ----
    int i = 0;
    for (long long t = first_tile; t < n_tiles; t += tile_step, ++i) {
      const int a = i & 1;
      int tm, tn;
      tile_of(t, tm, tn);
      bool ok = mbar_wait(bar_acc_full + 8 * a, (uint32_t)(i >> 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const long long row = (long long)(2 * tm + (int)cr) * kGemmBM + warp * 32 + lane;
      const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16) + a * kGemmBN;
      if (swiglu) {
        // the tile's columns are [128 gate | 128 up] of the same 128 intermediate features (weight rows arranged so
        // by the caller): out[row, tn * 128 + j] = silu(gate_j) * up_j, fp32, one rounding to bf16
        const int n_inter = N / 2;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t g[32], u[32];
          tmem_ld32(t_lane + c * 32, g);
          tmem_ld32(t_lane + 128 + c * 32, u);
          tmem_wait_ld();
          const int col0 = tn * 128 + c * 32;
          if (row < M && col0 < n_inter) {
            const long long off = row * n_inter + col0;
#pragma unroll
            for (int i8 = 0; i8 < 32; i8 += 8) {
              uint32_t w[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float g0 = __uint_as_float(g[i8 + 2 * e]), g1 = __uint_as_float(g[i8 + 2 * e + 1]);
                __nv_bfloat162 h2 = __floats2bfloat162_rn(g0 / (1.f + __expf(-g0)) * __uint_as_float(u[i8 + 2 * e]),
                                                          g1 / (1.f + __expf(-g1)) * __uint_as_float(u[i8 + 2 * e + 1]));
                w[e] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(y + off + i8) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      } else
#pragma unroll 1
      for (int c = 0; c < kGemmBN / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(t_lane + c * 32, v);
        tmem_wait_ld();
        const int col0 = tn * kGemmBN + c * 32;
        if (row < M && col0 < N) {
          const long long off = row * N + col0;
          uint16_t* yc = chunk_ptr(segs, y, row, N, col0);
#pragma unroll
          for (int i8 = 0; i8 < 32; i8 += 8) {
            if (col0 + i8 < N) {                                 // N is a multiple of 8
              float f[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[i8 + e]);
              if (residual != nullptr) {
                const uint4 r = __ldg(reinterpret_cast<const uint4*>(residual + off + i8));
                const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) { f[2 * e] += __uint_as_float(rw[e] << 16); f[2 * e + 1] += __uint_as_float(rw[e] & 0xffff0000u); }
              }
              uint32_t w[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                __nv_bfloat162 h2 = __floats2bfloat162_rn(f[2 * e], f[2 * e + 1]);
                w[e] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(yc + i8) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      }
      // the accumulator has been read out: the MMA warp may overwrite it
      tc_fence_before();
      mbar_arrive_remote(mapa_shared(bar_acc_empty + 8 * a, 0));
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_TIMEOUT, KID_GEMM_SM100, (int)blockIdx.x, 0);
    const uint64_t tw = global_timer_ns();
    while (global_timer_ns() - tw < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  cluster_sync();                             // the peer's shared memory is an operand of the leader's MMAs
  if (warp == 5) { tc_fence_after(); tmem_dealloc2(tmem_base, 512); }
}

}  // namespace relaxkv

using namespace relaxkv;

static relaxkv_status launch_gemm(const void* x, const void* weight, const void* residual, void* y, int64_t n_rows,
                                  int32_t n_out, int32_t n_in, int swiglu, relaxkv_stream stream_,
                                  const GemmSegs* segs_in = nullptr) {
  GemmSegs segs = {};
  if (segs_in) segs = *segs_in;
  if (!x || !weight || !y || !aligned16(x) || !aligned16(weight) || !aligned16(y) || (residual && !aligned16(residual)))
    return RELAXKV_ERR_INVALID_ARG;
  if (n_rows < 0 || n_out < 8 || n_in < 8 || (n_out % 8) || (n_in % 8)) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (swiglu && ((n_out % 256) || residual)) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (n_rows == 0) return RELAXKV_OK;
  if (n_rows <= kGemvMaxRows)       // a decode token: stream the weights once, no 128-row tiles
    return launch_gemv(x, weight, residual, y, (int)n_rows, n_out, n_in, swiglu, static_cast<cudaStream_t>(stream_));
  if (n_rows <= kSkinnyMaxRows && !swiglu && skinny_tiles(n_out) <= sm_count_of_current_device()) {
    // one row tile and no more column tiles than SMs (the query's tokens through a 5120-wide projection): 128 x 128
    // tiles, K split over a cluster so that about all SMs stream weights.  (The fused gate/up projection has 272 such
    // tiles at the model shapes and keeps the large kernel.)
    SkinnyOut outs = {};
    outs.y[0] = static_cast<uint16_t*>(y);
    outs.residual[0] = static_cast<const uint16_t*>(residual);
    outs.col0[0] = 0; outs.col0[1] = n_out;
    outs.n = 1;
    return launch_gemm_skinny(x, weight, outs, (int)n_rows, n_out, n_in, static_cast<cudaStream_t>(stream_));
  }
  // SM pairs (256-row tiles) unless that would leave a large share of the last tile row empty: with an odd number of
  // 128-row tiles, seven at most, the second block of the last pair would compute padding only (>= 1/8 of the work),
  // and the single-block kernel (128 x 256 tiles) is used.
  const long long tiles_128 = (n_rows + kGemmBM - 1) / kGemmBM;
  const bool use_pair = !((tiles_128 & 1) && tiles_128 <= 7);
  CUtensorMap tm_a, tm_b;
  if (!make_map_3d(&tm_a, x, (uint64_t)n_in, (uint64_t)n_rows, 1, (uint64_t)n_in * 2, (uint64_t)n_in * 2 * (uint64_t)n_rows, kGemmBM, 1) ||
      !make_map_3d(&tm_b, weight, (uint64_t)n_in, (uint64_t)n_out, 1, (uint64_t)n_in * 2, (uint64_t)n_in * 2 * (uint64_t)n_out,
                   use_pair ? kGemmBN / 2 : kGemmBN, 1))
    return RELAXKV_ERR_CUDA;
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  static std::atomic<int> attr_done[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RELAXKV_ERR_CUDA;
  if (!attr_done[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(gemm_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_pair_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmem) != cudaSuccess)
      return RELAXKV_ERR_CUDA;
    attr_done[dev].store(1, std::memory_order_release);
  }
  const int sms = sm_count_of_current_device();
  if (sms <= 0) return RELAXKV_ERR_CUDA;
  const long long tiles_n = (n_out + kGemmBN - 1) / kGemmBN;
  if (use_pair) {
    const long long tiles_m2 = (n_rows + 2 * kGemmBM - 1) / (2 * kGemmBM);
    if (tiles_m2 * tiles_n > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
    // persistent: as many clusters as can be resident at once (fewer than SMs / 2 where a GPC has an odd SM left over)
    static std::atomic<int> max_clusters[kMaxDevices];
    int n_clusters = max_clusters[dev].load(std::memory_order_acquire);
    if (n_clusters == 0) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)sms);
      cfg.blockDim = dim3(kGemmThreads);
      cfg.dynamicSmemBytes = kPairSmem;
      cudaLaunchAttribute attr;
      attr.id = cudaLaunchAttributeClusterDimension;
      attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
      cfg.attrs = &attr;
      cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, gemm_pair_sm100_kernel, &cfg) != cudaSuccess || n < 1) n = std::max(1, sms / 2 - 8);
      n_clusters = n;
      max_clusters[dev].store(n, std::memory_order_release);
    }
    const long long clusters = std::min<long long>(tiles_m2 * tiles_n, n_clusters);
    gemm_pair_sm100_kernel<<<(unsigned)(2 * clusters), kGemmThreads, kPairSmem, static_cast<cudaStream_t>(stream_)>>>(
        tm_a, tm_b, n_rows, n_out, n_in, static_cast<uint16_t*>(y), static_cast<const uint16_t*>(residual), swiglu, segs, st);
    return launch_ok();
  }
  const long long tiles_m = (n_rows + kGemmBM - 1) / kGemmBM;
  if (tiles_m * tiles_n > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  const long long grid = std::min<long long>(tiles_m * tiles_n, sms);     // persistent: one CTA per SM
  gemm_sm100_kernel<<<(unsigned)grid, kGemmThreads, kGemmSmem, static_cast<cudaStream_t>(stream_)>>>(
      tm_a, tm_b, n_rows, n_out, n_in, static_cast<uint16_t*>(y), static_cast<const uint16_t*>(residual), swiglu, segs, st);
  return launch_ok();
}

extern "C" relaxkv_status relaxkv_linear(const void* x, const void* weight, const void* residual, void* y,
                                         int64_t n_rows, int32_t n_out, int32_t n_in, relaxkv_stream stream_) {
  RELAXKV_RANGE("relaxkv_linear");
  return launch_gemm(x, weight, residual, y, n_rows, n_out, n_in, 0, stream_);
}

extern "C" relaxkv_status relaxkv_linear_qkv(const void* x, const void* w_qkv, void* q, void* k, void* v, int64_t n_rows,
                                             int32_t n_q, int32_t n_kv, int32_t n_in, relaxkv_stream stream_) {
  RELAXKV_RANGE("relaxkv_linear_qkv");
  if (!x || !w_qkv || !q || !k || !v || !aligned16(x) || !aligned16(w_qkv) || !aligned16(q) || !aligned16(k) || !aligned16(v))
    return RELAXKV_ERR_INVALID_ARG;
  if (n_rows < 0 || n_q < 8 || n_kv < 8 || n_in < 8 || (n_q % 8) || (n_kv % 8) || (n_in % 8)) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (n_rows == 0) return RELAXKV_OK;
  const int n_out = n_q + 2 * n_kv;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (n_rows <= kGemvMaxRows) {
    GemvOut outs = {};
    outs.y[0] = static_cast<uint16_t*>(q); outs.y[1] = static_cast<uint16_t*>(k); outs.y[2] = static_cast<uint16_t*>(v);
    outs.col0[0] = 0; outs.col0[1] = n_q; outs.col0[2] = n_q + n_kv; outs.col0[3] = n_out;
    outs.n = 3;
    return launch_gemv_segments(x, w_qkv, outs, (int)n_rows, n_out, n_in, stream);
  }
  if (n_rows <= kSkinnyMaxRows && skinny_tiles(n_out) <= sm_count_of_current_device()) {
    SkinnyOut outs = {};
    outs.y[0] = static_cast<uint16_t*>(q); outs.y[1] = static_cast<uint16_t*>(k); outs.y[2] = static_cast<uint16_t*>(v);
    outs.col0[0] = 0; outs.col0[1] = n_q; outs.col0[2] = n_q + n_kv; outs.col0[3] = n_out;
    outs.n = 3;
    return launch_gemm_skinny(x, w_qkv, outs, (int)n_rows, n_out, n_in, stream);
  }
  // many rows: one GEMM over the stacked matrix whose epilogue writes the three buffers (the K and V projections alone
  // have four 256-column tiles each and leave the last wave of SM pairs half empty) ...
  if (n_q % 32 == 0 && n_kv % 32 == 0) {
    GemmSegs segs = {};
    segs.y[0] = static_cast<uint16_t*>(q); segs.y[1] = static_cast<uint16_t*>(k); segs.y[2] = static_cast<uint16_t*>(v);
    segs.col0[0] = 0; segs.col0[1] = n_q; segs.col0[2] = n_q + n_kv; segs.col0[3] = n_out;
    segs.n = 3;
    return launch_gemm(x, w_qkv, nullptr, q, n_rows, n_out, n_in, 0, stream_, &segs);
  }
  // ... unless a boundary falls inside a 32-column chunk of the epilogue: then the three projections one after the other
  const uint16_t* w = static_cast<const uint16_t*>(w_qkv);
  relaxkv_status rc = launch_gemm(x, w, nullptr, q, n_rows, n_q, n_in, 0, stream_);
  if (rc == RELAXKV_OK) rc = launch_gemm(x, w + (size_t)n_q * n_in, nullptr, k, n_rows, n_kv, n_in, 0, stream_);
  if (rc == RELAXKV_OK) rc = launch_gemm(x, w + (size_t)(n_q + n_kv) * n_in, nullptr, v, n_rows, n_kv, n_in, 0, stream_);
  return rc;
}

extern "C" relaxkv_status relaxkv_linear_swiglu(const void* x, const void* weight_tiled, void* y, int64_t n_rows,
                                                int32_t n_inter, int32_t n_in, relaxkv_stream stream_) {
  RELAXKV_RANGE("relaxkv_linear_swiglu");
  if (n_inter < 128 || (n_inter % 128)) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  return launch_gemm(x, weight_tiled, nullptr, y, n_rows, 2 * n_inter, n_in, 1, stream_);
}
