// y = x W^T (+ residual) for at most 128 rows of x (the query's own tokens going through the block, Section 2 of the
// paper: the query pass that yields the scores, and the query prefill that closes the time-to-first-token region).
// With one row tile the 128 x 256 tiling of the large GEMM leaves most SMs without work (a 5120-wide projection is 20
// tiles) and the time is the weight matrix streaming through those few SMs.  Here the tile is 128 x 128 and a
// thread-block CLUSTER of S blocks (S = 1..8, chosen so that the launch is one wave of about all SMs) shares it and
// splits K: block r multiplies K blocks [r n_k / S, (r + 1) n_k / S) into its own TMEM accumulator (six-stage TMA
// ring, tcgen05.mma M=128 N=128 K=16), writes the partial tile into its own shared memory, and after a cluster
// barrier every block sums, for the 8-column groups it owns (group g belongs to block g mod S), the S partials in rank
// order - its own from local, the others' through distributed shared memory - adds the residual and writes bf16.
// A fixed order: results do not depend on timing.  No scratch in global memory.
// Up to three output segments (column ranges going to different buffers) serve the fused Q/K/V projection.
// The cluster barriers have no time limit, so every thread executes all of them whatever its (bounded) waits on the
// mbarriers have returned, and no block leaves before its peers have read its partial tile.
#include "common.cuh"
#include "gemm_skinny.cuh"
#include "sm100_ptx.cuh"
#include <algorithm>
#include <atomic>

namespace relaxkv {

using namespace ptx;

bool make_map_3d(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_bytes,
                 uint64_t stride2_bytes, uint32_t b1, uint32_t b2);          // attention_sm100.cu

constexpr int kSkBM = 128, kSkBN = 128, kSkBK = 64, kSkStages = 6, kSkThreads = 192;
constexpr int kSkABytes = kSkBM * kSkBK * 2, kSkBBytes = kSkBN * kSkBK * 2;
constexpr int kSkStageBytes = kSkABytes + kSkBBytes;                       // 32 KB
constexpr int kSkBars = 2 * kSkStages + 1;                                 // full, empty per stage; accumulator full
constexpr int kSkSmem = kSkStages * kSkStageBytes + 8 * kSkBars + 16 + 1024;
static_assert(kSkBM * kSkBN * 4 <= kSkStages * kSkStageBytes, "the partial tile reuses the TMA ring");

__device__ __forceinline__ float ld_cluster_f32(uint32_t cluster_addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(cluster_addr) : "memory");
  return v;
}

template <int S>
__global__ void __launch_bounds__(kSkThreads, 1)
gemm_skinny_sm100_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                         int M, int N, int K, const __grid_constant__ SkinnyOut outs, DeviceStatus* st) {
  const uint32_t rank = (S > 1) ? cluster_ctarank() : 0u;
  const int tn = (int)(blockIdx.x / S);
  const int n_k = (K + kSkBK - 1) / kSkBK;
  const int k0 = (int)((long long)rank * n_k / S), k1 = (int)((long long)(rank + 1) * n_k / S);
  // after an expired wait elsewhere the tensor-core kernels move nothing until the status word has been read; here
  // that means: run through the barriers (a block must not leave its cluster waiting), compute nothing
  const bool drained = *reinterpret_cast<volatile int*>(&st->status) == RELAXKV_ERR_TIMEOUT;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar0 = base + kSkStages * kSkStageBytes;
  const uint32_t bar_full = bar0, bar_empty = bar0 + 8 * kSkStages, bar_acc = bar0 + 16 * kSkStages;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kSkStages * kSkStageBytes + 8 * kSkBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(const_cast<uint32_t*>(tmem_slot) + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSkStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    mbar_init(bar_acc, 1);
    *abort_flag = drained ? 1 : 0;
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 5) { tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kSkBN); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  bool ok = !*abort_flag;
  if (warp == 4) {
    // ---- TMA producer ----
    if (lane == 0 && ok) {
      prefetch_tensormap(&tm_a); prefetch_tensormap(&tm_b);
      for (int kt = k0, it = 0; kt < k1; ++kt, ++it) {
        const int s = it % kSkStages;
        if (it >= kSkStages && !mbar_wait(bar_empty + 8 * s, (uint32_t)((it / kSkStages) - 1) & 1, abort_flag)) break;
        mbar_expect_tx(bar_full + 8 * s, kSkStageBytes);
        tma_load_3d(base + s * kSkStageBytes, &tm_a, bar_full + 8 * s, kt * kSkBK, 0, 0);
        tma_load_3d(base + s * kSkStageBytes + kSkABytes, &tm_b, bar_full + 8 * s, kt * kSkBK, tn * kSkBN, 0);
      }
    }
  } else if (warp == 5) {
    // ---- MMA issuer ----
    if (lane == 0 && ok) {
      constexpr uint32_t idesc = idesc_bf16_f32(kSkBM, kSkBN, 0);
      bool go = true;
      for (int kt = k0, it = 0; kt < k1; ++kt, ++it) {
        const int s = it % kSkStages;
        if (!(go = mbar_wait(bar_full + 8 * s, (uint32_t)(it / kSkStages) & 1, abort_flag))) break;
        tc_fence_after();
        const uint32_t sa = base + s * kSkStageBytes;
        mma_ss_4steps(tmem_base, desc_lo(sa, 16), desc_lo(sa + kSkABytes, 16), desc_hi_sw128(1024), idesc, it > 0 ? 1u : 0u);
        mma_commit(bar_empty + 8 * s);
      }
      if (go) mma_commit(bar_acc);
    }
  } else {
    // ---- epilogue warps (thread = row = TMEM lane): this block's partial tile -> its own shared memory, [column][row]
    // fp32 (the lanes of a warp hold consecutive rows: every store below writes 128 consecutive bytes).  The MMAs have
    // completed by then, so the TMA ring is free to hold it. ----
    if (ok) ok = mbar_wait(bar_acc, 0, abort_flag);
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    if (ok) {
      const int row = warp * 32 + lane;
      const uint32_t t_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
      float* stage = reinterpret_cast<float*>(base_ptr);
#pragma unroll 1
      for (int c = 0; c < kSkBN / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(t_lane + c * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) stage[(c * 32 + i) * kSkBM + row] = __uint_as_float(v[i]);
      }
    }
  }
  // every block's partial tile is in place
  __syncthreads();
  if (S > 1) cluster_sync();
  ok = !*abort_flag;

  if (warp < 4 && ok) {
    const int row = warp * 32 + lane;
    const uint32_t stage_addr = base + (uint32_t)row * 4u;
    uint32_t peer[S];
#pragma unroll
    for (int src = 0; src < S; ++src) peer[src] = (S > 1) ? mapa_shared(stage_addr, (uint32_t)src) : stage_addr;
    // 8-column groups g = rank, rank + S, ... of the tile
#pragma unroll 1
    for (int g = (int)rank; g < kSkBN / 8; g += S) {
      const int col0 = tn * kSkBN + g * 8;
      if (col0 >= N) break;
      float f[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] = 0.f;
#pragma unroll
      for (int src = 0; src < S; ++src) {                        // rank order: the same sum whatever the timing
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = ld_cluster_f32(peer[src] + (uint32_t)((g * 8 + e) * kSkBM) * 4u);
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] += v[e];
      }
      if (row < M) {
        // which output buffer these 8 columns go to (segment boundaries are multiples of 8 columns)
        int sg = 0;
        while (sg + 1 < outs.n && col0 >= outs.col0[sg + 1]) ++sg;
        const int width = outs.col0[sg + 1] - outs.col0[sg];
        const long long off = (long long)row * width + (col0 - outs.col0[sg]);
        const uint16_t* res = outs.residual[sg];
        if (res != nullptr) {
          const uint4 r = __ldg(reinterpret_cast<const uint4*>(res + off));
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
        *reinterpret_cast<uint4*>(outs.y[sg] + off) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
  }
  // nobody leaves while a peer may still read its partial tile
  tc_fence_before();
  __syncthreads();
  if (S > 1) cluster_sync();
  if (*abort_flag && !drained) {
    if (threadIdx.x == 0) report(st, RELAXKV_ERR_TIMEOUT, KID_GEMM_SM100, (int)blockIdx.x, 1);
    const uint64_t tw = global_timer_ns();
    while (global_timer_ns() - tw < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 5) { tc_fence_after(); tmem_dealloc(tmem_base, kSkBN); }
}

// Largest number of S-block clusters of this kernel that can be resident at once (per device, looked up once).
template <int S>
static int max_clusters(int dev, int sms) {
  static std::atomic<int> cached[kMaxDevices];
  int n = cached[dev].load(std::memory_order_acquire);
  if (n == 0) {
    if (S == 1) {
      n = sms;
    } else {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)(sms / S * S));
      cfg.blockDim = dim3(kSkThreads);
      cfg.dynamicSmemBytes = kSkSmem;
      cudaLaunchAttribute attr;
      attr.id = cudaLaunchAttributeClusterDimension;
      attr.val.clusterDim.x = (unsigned)S; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
      cfg.attrs = &attr;
      cfg.numAttrs = 1;
      if (cudaOccupancyMaxActiveClusters(&n, gemm_skinny_sm100_kernel<S>, &cfg) != cudaSuccess || n < 1) n = std::max(1, sms / S / 2);
    }
    cached[dev].store(n, std::memory_order_release);
  }
  return n;
}

template <int S>
static bool prepare_s(int dev, int sms, int* n_clusters) {
  static std::atomic<int> attr_done[kMaxDevices];
  if (!attr_done[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(gemm_skinny_sm100_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSkSmem) != cudaSuccess)
      return false;
    attr_done[dev].store(1, std::memory_order_release);
  }
  *n_clusters = max_clusters<S>(dev, sms);
  return true;
}

template <int S>
static relaxkv_status launch_s(const CUtensorMap& tm_a, const CUtensorMap& tm_b, const SkinnyOut& outs, int n_rows, int n_out,
                               int n_in, int tiles_n, DeviceStatus* st, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(tiles_n * S));
  cfg.blockDim = dim3(kSkThreads);
  cfg.dynamicSmemBytes = kSkSmem;
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = (unsigned)S; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, gemm_skinny_sm100_kernel<S>, tm_a, tm_b, n_rows, n_out, n_in, outs, st) != cudaSuccess)
    return RELAXKV_ERR_CUDA;
  return launch_ok();
}

int skinny_tiles(int n_out) { return (n_out + kSkBN - 1) / kSkBN; }

relaxkv_status launch_gemm_skinny(const void* x, const void* weight, const SkinnyOut& outs, int n_rows, int n_out, int n_in,
                                  cudaStream_t stream) {
  RELAXKV_RANGE("gemm_skinny_sm100_kernel");
  CUtensorMap tm_a, tm_b;
  if (!make_map_3d(&tm_a, x, (uint64_t)n_in, (uint64_t)n_rows, 1, (uint64_t)n_in * 2, (uint64_t)n_in * 2 * (uint64_t)n_rows, kSkBM, 1) ||
      !make_map_3d(&tm_b, weight, (uint64_t)n_in, (uint64_t)n_out, 1, (uint64_t)n_in * 2, (uint64_t)n_in * 2 * (uint64_t)n_out, kSkBN, 1))
    return RELAXKV_ERR_CUDA;
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RELAXKV_ERR_CUDA;
  const int sms = sm_count_of_current_device();
  if (sms <= 0) return RELAXKV_ERR_CUDA;
  const int tiles_n = skinny_tiles(n_out);
  const int n_k = (n_in + kSkBK - 1) / kSkBK;
  // the largest cluster whose launch is still one wave (all its clusters resident at once) and leaves every block at
  // least two K blocks
#define RELAXKV_TRY_S(SV)                                                                           \
  if (n_k >= 2 * SV) {                                                                              \
    int nc = 0;                                                                                     \
    if (!prepare_s<SV>(dev, sms, &nc)) return RELAXKV_ERR_CUDA;                                      \
    if (tiles_n <= nc) return launch_s<SV>(tm_a, tm_b, outs, n_rows, n_out, n_in, tiles_n, st, stream); \
  }
  RELAXKV_TRY_S(8) RELAXKV_TRY_S(7) RELAXKV_TRY_S(6) RELAXKV_TRY_S(5) RELAXKV_TRY_S(4) RELAXKV_TRY_S(3) RELAXKV_TRY_S(2)
#undef RELAXKV_TRY_S
  int nc = 0;
  if (!prepare_s<1>(dev, sms, &nc)) return RELAXKV_ERR_CUDA;
  return launch_s<1>(tm_a, tm_b, outs, n_rows, n_out, n_in, tiles_n, st, stream);
}

}  // namespace relaxkv
