// Projections of a handful of rows (a decode token, the last query row going through the output head): y = x W^T with
// at most kGemvMaxRows rows of x.  The work is reading W once (HBM-bound: every weight byte meets one to four
// multiply-adds), so this is a plain streaming kernel, not the 128-row tensor-core GEMM: each warp owns two output
// features (16 per block: a 5120-wide projection is 320 blocks, all resident at once), its lanes stride over K in
// 16-byte pieces with eight independent weight loads in flight per lane, x stays in L1, and a shuffle tree sums the
// lanes' partial dot products in a fixed order.  (Algorithm 1 runs the model's
// own block unchanged; after the repair loop the same block serves the decode step of the TTFT region.)
#include "common.cuh"
#include "gemv.cuh"

namespace relaxkv {

constexpr int kGemvThreads = 256;
constexpr int kGemvFeatPerWarp = 2;        // few features per warp: many blocks, so that enough bytes are in flight
constexpr int kGemvFeatPerBlock = (kGemvThreads / 32) * kGemvFeatPerWarp;
constexpr int kGemvPrefetchElems = 1024;   // weights per row and warp requested into L2 before the dependency wait

__device__ __forceinline__ void unpack8_gemv(const uint4& v, float* f) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) { f[2 * e] = __uint_as_float(w[e] << 16); f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u); }
}

// SWIGLU = 0: y[m, n] = sum_k x[m, k] w[n, k] (+ residual[m, n])          w [n_out, K]
// SWIGLU = 1: y[m, f] = silu(sum_k x w[g(f), k]) * (sum_k x w[g(f) + 128, k])   with g(f) = (f / 128) * 256 + f % 128
//             (the gate rows of every block of 128 features are followed by its up rows); n_out counts the features f
// SEG = 1: the features are the rows of several stacked weight matrices (the fused Q/K/V projection) and segment i,
//          features [col0[i], col0[i + 1]), is written to its own buffer outs.y[i] of that width; y is unused.
// KS > 1: KS warps share a warp's features and split K among them (partial sums added through shared memory in a
//         fixed order): a matrix of a few tens of MB then has four times as many, four times shorter dependent load
//         chains, which is what bounds such a launch (not bandwidth).
template <int M, int SWIGLU, int SEG, int KS>
__global__ void __launch_bounds__(kGemvThreads)
gemv_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ w, const uint16_t* __restrict__ residual,
            uint16_t* __restrict__ y, int n_out, int K, const GemvOut outs) {
  constexpr int kWarps = kGemvThreads / 32, kGroups = kWarps / KS;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grp = warp / KS, kp = warp % KS;
  const int f0 = (blockIdx.x * kGroups + grp) * kGemvFeatPerWarp;
  constexpr int R = SWIGLU ? 2 * kGemvFeatPerWarp : kGemvFeatPerWarp;      // weight rows this warp streams
  const uint16_t* wr[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int f = min(f0 + (r % kGemvFeatPerWarp), n_out - 1);              // the tail warp re-reads the last feature
    const long long row = SWIGLU ? ((long long)(f / 128) * 256 + (f % 128) + (r >= kGemvFeatPerWarp ? 128 : 0)) : f;
    wr[r] = w + row * K;
  }
  float acc[R][M];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int m = 0; m < M; ++m) acc[r][m] = 0.f;
  const int k_part = (KS == 1) ? K : ((K + KS * 256 - 1) / (KS * 256)) * 256;      // this warp's share of K
  const int k_lo = kp * k_part, k_hi = min(K, k_lo + k_part);
  // Chained launch: the weights depend on no earlier kernel, so the head of this warp's rows is requested into L2
  // while the kernel before this one is still finishing; x (and the residual) are read after the wait.
  {
    const int kpre = k_lo + lane * 64;                                      // one 128-byte line per lane
    if (kpre < min(k_hi, k_lo + kGemvPrefetchElems)) {
#pragma unroll
      for (int r = 0; r < R; ++r) asm volatile("prefetch.global.L2 [%0];" ::"l"(wr[r] + kpre));
    }
  }
  griddep_wait();
#pragma unroll 4
  for (int k = k_lo + lane * 8; k < k_hi; k += 32 * 8) {
    uint4 wv[R];
#pragma unroll
    for (int r = 0; r < R; ++r) wv[r] = __ldg(reinterpret_cast<const uint4*>(wr[r] + k));     // all loads first
    float xf[M][8];
#pragma unroll
    for (int m = 0; m < M; ++m) unpack8_gemv(__ldg(reinterpret_cast<const uint4*>(x + (long long)m * K + k)), xf[m]);
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float wf[8];
      unpack8_gemv(wv[r], wf);
#pragma unroll
      for (int m = 0; m < M; ++m)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[r][m] = fmaf(xf[m][e], wf[e], acc[r][m]);
    }
  }
  // the next kernel may become resident now, not earlier: its blocks would hold this kernel's later blocks' places and
  // its prefetches would compete with this kernel's stream (measured: triggering at the top costs a 40-layer decode
  // step with 350 MB gate/up matrices 7 %, triggering here gains 5 %)
  griddep_launch();
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int m = 0; m < M; ++m) acc[r][m] = warp_reduce_sum(acc[r][m]);
  if (KS > 1) {
    __shared__ float part[kWarps][R][M];
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int m = 0; m < M; ++m) part[warp][r][m] = acc[r][m];
    }
    __syncthreads();
    if (kp != 0) return;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int m = 0; m < M; ++m) {
        float v = 0.f;
#pragma unroll
        for (int q = 0; q < KS; ++q) v += part[grp * KS + q][r][m];          // fixed order
        acc[r][m] = v;
      }
  }
  if (lane < kGemvFeatPerWarp) {
    const int f = f0 + lane;
    if (f < n_out) {
#pragma unroll
      for (int m = 0; m < M; ++m) {
        float v = 0.f;
#pragma unroll
        for (int r = 0; r < kGemvFeatPerWarp; ++r) {          // static indexing keeps the accumulators in registers
          if (r == lane) {
            if (SWIGLU) {                                     // one rounding, after the activation
              const float g = acc[r][m], u = acc[r + (SWIGLU ? kGemvFeatPerWarp : 0)][m];
              v = g / (1.f + __expf(-g)) * u;
            } else {
              v = acc[r][m];
            }
          }
        }
        const __nv_bfloat16 h = __float2bfloat16((!SWIGLU && !SEG && residual) ? v + bf16_bits_to_float(residual[(long long)m * n_out + f]) : v);
        if (SEG) {
          int sg = 0;
          while (sg + 1 < outs.n && f >= outs.col0[sg + 1]) ++sg;
          outs.y[sg][(long long)m * (outs.col0[sg + 1] - outs.col0[sg]) + (f - outs.col0[sg])] = *reinterpret_cast<const uint16_t*>(&h);
        } else {
          y[(long long)m * n_out + f] = *reinterpret_cast<const uint16_t*>(&h);
        }
      }
    }
  }
}

constexpr long long kGemvSplitKBelowBytes = 256ll << 20;     // matrices below this size split K over four warps

template <int SWIGLU, int SEG, int KS>
static relaxkv_status launch_mk(const uint16_t* x, const uint16_t* w, const uint16_t* residual, uint16_t* y, int n_rows,
                                int n_out, int K, const GemvOut& outs, cudaStream_t stream) {
  constexpr int feat_per_block = kGemvFeatPerBlock / KS;
  const unsigned blocks = (unsigned)((n_out + feat_per_block - 1) / feat_per_block);
  cudaError_t e = cudaSuccess;
  switch (n_rows) {
    case 1: e = launch_chained(true, gemv_kernel<1, SWIGLU, SEG, KS>, blocks, kGemvThreads, 0, stream, x, w, residual, y, n_out, K, outs); break;
    case 2: e = launch_chained(true, gemv_kernel<2, SWIGLU, SEG, KS>, blocks, kGemvThreads, 0, stream, x, w, residual, y, n_out, K, outs); break;
    case 3: e = launch_chained(true, gemv_kernel<3, SWIGLU, SEG, KS>, blocks, kGemvThreads, 0, stream, x, w, residual, y, n_out, K, outs); break;
    case 4: e = launch_chained(true, gemv_kernel<4, SWIGLU, SEG, KS>, blocks, kGemvThreads, 0, stream, x, w, residual, y, n_out, K, outs); break;
    default: return RELAXKV_ERR_INVALID_ARG;
  }
  return cuda_ok(e);
}

template <int SWIGLU, int SEG>
static relaxkv_status launch_m(const uint16_t* x, const uint16_t* w, const uint16_t* residual, uint16_t* y, int n_rows,
                               int n_out, int K, const GemvOut& outs, cudaStream_t stream) {
  const long long bytes = (long long)(SWIGLU ? 2 : 1) * n_out * K * 2;
  if (bytes < kGemvSplitKBelowBytes && K >= 4 * 256)
    return launch_mk<SWIGLU, SEG, 4>(x, w, residual, y, n_rows, n_out, K, outs, stream);
  return launch_mk<SWIGLU, SEG, 1>(x, w, residual, y, n_rows, n_out, K, outs, stream);
}

relaxkv_status launch_gemv(const void* x, const void* weight, const void* residual, void* y, int n_rows, int n_out,
                           int n_in, int swiglu, cudaStream_t stream) {
  RELAXKV_RANGE("gemv_kernel");
  const GemvOut none = {};
  if (swiglu)
    return launch_m<1, 0>(static_cast<const uint16_t*>(x), static_cast<const uint16_t*>(weight), nullptr,
                          static_cast<uint16_t*>(y), n_rows, n_out / 2, n_in, none, stream);
  return launch_m<0, 0>(static_cast<const uint16_t*>(x), static_cast<const uint16_t*>(weight),
                        static_cast<const uint16_t*>(residual), static_cast<uint16_t*>(y), n_rows, n_out, n_in, none, stream);
}

relaxkv_status launch_gemv_segments(const void* x, const void* weight, const GemvOut& outs, int n_rows, int n_out, int n_in,
                                    cudaStream_t stream) {
  RELAXKV_RANGE("gemv_kernel");
  return launch_m<0, 1>(static_cast<const uint16_t*>(x), static_cast<const uint16_t*>(weight), nullptr, nullptr, n_rows, n_out,
                        n_in, outs, stream);
}

}  // namespace relaxkv
