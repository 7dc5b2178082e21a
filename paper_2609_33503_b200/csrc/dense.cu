// The small row-wise kernels of the active targets' block work (Algorithm 1, steps 14, 16, 20): RMSNorm, rotary
// embedding at the tokens' ORIGINAL positions (Section 3.3), SwiGLU, and the carry of the hidden rows that stay
// active from layer l to l+1 (R_{l+1} is a subset of R_l).  All HBM-bound, 16-byte accesses.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace relaxkv {

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) { f[2 * e] = __uint_as_float(w[e] << 16); f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u); }
}
__device__ __forceinline__ uint4 pack8(const float* f) {
  uint32_t w[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    __nv_bfloat162 h2 = __floats2bfloat162_rn(f[2 * e], f[2 * e + 1]);
    w[e] = *reinterpret_cast<uint32_t*>(&h2);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// y = x / sqrt(mean(x^2) + eps) * w ; one block per row, C a multiple of 8.
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ w, uint16_t* __restrict__ y, int C, float eps) {
  const long long row = blockIdx.x;
  const uint16_t* xr = x + row * C;
  float ss = 0.f;
  griddep_launch();
  griddep_wait();
  for (int i = threadIdx.x * 8; i < C; i += 256 * 8) {
    float f[8];
    unpack8(__ldg(reinterpret_cast<const uint4*>(xr + i)), f);
#pragma unroll
    for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
  }
  __shared__ float red[8];
  ss = warp_reduce_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += red[i];                 // fixed order: reproducible
  const float inv = rsqrtf(tot / (float)C + eps);
  for (int i = threadIdx.x * 8; i < C; i += 256 * 8) {
    float f[8], g[8];
    unpack8(__ldg(reinterpret_cast<const uint4*>(xr + i)), f);
    unpack8(__ldg(reinterpret_cast<const uint4*>(w + i)), g);
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = f[e] * inv * g[e];
    *reinterpret_cast<uint4*>(y + row * C + i) = pack8(f);
  }
}

// Short rows (a head vector: C <= 256): one warp per row, each lane 8 elements, so the per-head Q/K norm of a
// [rows, heads, D] tensor is one pass over it.  In place (y == x) is fine: a lane writes what it alone read.
__global__ void __launch_bounds__(256)
rmsnorm_short_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ w, uint16_t* __restrict__ y, long long rows,
                     int C, float eps) {
  const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  griddep_launch();
  griddep_wait();
  if (row >= rows) return;
  const bool mine = lane * 8 < C;
  float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (mine) unpack8(*reinterpret_cast<const uint4*>(x + row * C + lane * 8), f);
  float ss = 0.f;
#pragma unroll
  for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
  ss = warp_reduce_sum(ss);
  const float inv = rsqrtf(ss / (float)C + eps);
  if (mine) {
    float g[8];
    unpack8(__ldg(reinterpret_cast<const uint4*>(w + lane * 8)), g);
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = f[e] * inv * g[e];
    *reinterpret_cast<uint4*>(y + row * C + lane * 8) = pack8(f);
  }
}

// Rotate-half rotary embedding in place on x [rows, heads, D]; one thread per (row, 8 pairs): the eight
// (cos, sin) pairs are computed once and applied to every head of the row.
__global__ void rope_kernel(uint16_t* __restrict__ x, long long rows, int heads, int D, const int* __restrict__ positions,
                            double log2_theta) {
  const int half = D / 2, groups = half / 8;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * groups) return;
  const int gi = (int)(idx % groups);
  const long long row = idx / groups;
  const double pos = (double)positions[row];
  float cs[8], sn[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const int i = gi * 8 + e;
    // angle = pos * theta^(-2i/D), reduced in double so that positions of tens of thousands keep their phase
    const double inv_freq = exp2(-log2_theta * (2.0 * i / D));
    double ang = pos * inv_freq;
    ang -= 6.283185307179586 * floor(ang * 0.15915494309189535);
    sincosf((float)ang, &sn[e], &cs[e]);
  }
  for (int h = 0; h < heads; ++h) {
    uint16_t* v = x + (row * heads + h) * D;
    float a[8], b[8];
    unpack8(*reinterpret_cast<const uint4*>(v + gi * 8), a);
    unpack8(*reinterpret_cast<const uint4*>(v + half + gi * 8), b);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float x1 = a[e], x2 = b[e];
      a[e] = x1 * cs[e] - x2 * sn[e];
      b[e] = x2 * cs[e] + x1 * sn[e];
    }
    *reinterpret_cast<uint4*>(v + gi * 8) = pack8(a);
    *reinterpret_cast<uint4*>(v + half + gi * 8) = pack8(b);
  }
}

// Per-head RMSNorm (optional) and rotary embedding of the projected queries and keys of a few rows in ONE launch
// (the query's own tokens, a decode token: four launches of a few microseconds otherwise; for the repair loop's many
// rows: one pass over q and k instead of two).  One block per (row, four heads): the first D/2 threads compute the
// row's (cos, sin) table, then every warp takes one head (query heads first, then KV
// heads); a lane holds D/32 consecutive dims, its rotation partner sits 16 lanes away.  Grid: (rows, groups of heads):
// four heads per block for a few rows (all warps busy at once), all heads in one block for many rows (the table's
// double-precision arithmetic, about 3 k clk per block, is then paid once per row).  Between the two steps the
// values are rounded to bf16, as they would be if the normalised heads had been stored and read back.
template <int D>
__global__ void __launch_bounds__(128)
head_norm_rope_kernel(uint16_t* __restrict__ q, uint16_t* __restrict__ k, int Hq, int Hkv, int heads_per_block, const uint16_t* __restrict__ wq,
                      const uint16_t* __restrict__ wk, float eps, const int* __restrict__ positions, double log2_theta) {
  constexpr int DPL = D / 32, half = D / 2;
  constexpr int U = 4;                                        // heads a warp has in flight at once
  __shared__ float cs_s[half], sn_s[half];
  const long long row = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int d0 = lane * DPL;                                  // this lane's dims d0 .. d0 + DPL - 1
  const bool low = d0 < half;                                 // first half of the head vector: partner is + D/2
  // heads of this block: [blockIdx.y * heads_per_block, + heads_per_block); warp w takes every fourth one from w on,
  // U at a time: their loads are issued together (one 8-byte load per lane and head is too little in flight to keep
  // HBM busy when a block walks all heads of a row), the first batch before the table below is computed
  const int h_end = min(Hq + Hkv, ((int)blockIdx.y + 1) * heads_per_block);
  const int h_first = blockIdx.y * heads_per_block + warp;
  auto head_ptr = [&](int h) -> uint16_t* { return (h < Hq) ? q + (row * Hq + h) * D : k + (row * Hkv + (h - Hq)) * D; };
  auto load_batch = [&](int hb, uint2* raw) {
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int h = hb + 4 * u;
      raw[u] = make_uint2(0u, 0u);
      if (h < h_end) {
        if constexpr (DPL == 4) raw[u] = *reinterpret_cast<const uint2*>(head_ptr(h) + d0);     // one 8-byte access per lane
        else raw[u].x = *reinterpret_cast<const uint32_t*>(head_ptr(h) + d0);
      }
    }
  };
  auto process_batch = [&](int hb, const uint2* raw) {
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int h = hb + 4 * u;
      if (h >= h_end) break;                                    // uniform over the warp
      uint16_t* v = head_ptr(h);
      const uint16_t* w = (h < Hq) ? wq : wk;
      float f[DPL];
      f[0] = __uint_as_float(raw[u].x << 16); f[1] = __uint_as_float(raw[u].x & 0xffff0000u);
      if constexpr (DPL == 4) { f[2] = __uint_as_float(raw[u].y << 16); f[3] = __uint_as_float(raw[u].y & 0xffff0000u); }
      if (w != nullptr) {
        float ss = 0.f;
#pragma unroll
        for (int e = 0; e < DPL; ++e) ss = fmaf(f[e], f[e], ss);
        ss = warp_reduce_sum(ss);
        const float inv = rsqrtf(ss / (float)D + eps);
#pragma unroll
        for (int e = 0; e < DPL; ++e) f[e] = __bfloat162float(__float2bfloat16(f[e] * inv * bf16_bits_to_float(w[d0 + e])));
      }
      float r[DPL];
#pragma unroll
      for (int e = 0; e < DPL; ++e) {
        const float other = __shfl_xor_sync(0xffffffffu, f[e], 16);        // dim d0 + e -/+ D/2
        const int i = (d0 + e) % half;
        r[e] = low ? f[e] * cs_s[i] - other * sn_s[i] : f[e] * cs_s[i] + other * sn_s[i];
      }
      __nv_bfloat162 h01 = __floats2bfloat162_rn(r[0], r[1]);
      if constexpr (DPL == 4) {
        __nv_bfloat162 h23 = __floats2bfloat162_rn(r[2], r[3]);
        *reinterpret_cast<uint2*>(v + d0) = make_uint2(*reinterpret_cast<uint32_t*>(&h01), *reinterpret_cast<uint32_t*>(&h23));
      } else {
        *reinterpret_cast<uint32_t*>(v + d0) = *reinterpret_cast<uint32_t*>(&h01);
      }
    }
  };
  griddep_launch();
  griddep_wait();                                             // q, k and the positions may come from the kernels before
  uint2 raw[U];
  load_batch(h_first, raw);
  if (threadIdx.x < half) {
    const int i = threadIdx.x;
    const double inv_freq = exp2(-log2_theta * (2.0 * i / D));
    double ang = (double)positions[row] * inv_freq;
    ang -= 6.283185307179586 * floor(ang * 0.15915494309189535);
    sincosf((float)ang, &sn_s[i], &cs_s[i]);
  }
  __syncthreads();
  for (int hb = h_first; hb < h_end; hb += 4 * U) {
    uint2 next[U];
    load_batch(hb + 4 * U, next);                             // the next batch travels while this one is worked on
    process_batch(hb, raw);
#pragma unroll
    for (int u = 0; u < U; ++u) raw[u] = next[u];
  }
}

// ---- many rows: whole rows through shared memory with bulk asynchronous copies -------------------------------------
// The repair loop normalises and rotates tens of thousands of rows per layer.  With plain loads a warp has a few
// hundred bytes in flight and these kernels stop at 0.55-0.65 of the HBM copy bandwidth; here every warp owns one row,
// one lane asks the copy engine for the whole row (10 KB at 5120 columns), the lanes work on it in shared memory and
// one lane sends it back, so a block of four warps keeps 40-48 KB in flight without holding a byte in registers (the
// scheme of the gather and cache-update kernels).  This GPU's memory only, never multicast; every wait is bounded.
using namespace ptx;
constexpr int kRowWarps = 4;
constexpr int kRowBulkMinRows = 4096;        // fewer rows: the latency-oriented kernels above (equal at 2048 rows)
constexpr int kRowBulkMaxBytes = 16 * 1024;  // per row (and warp) of shared memory

__device__ __forceinline__ void row_wait_failed(DeviceStatus* st, long long row) {
  if ((threadIdx.x & 31) == 0) {
    report(st, RELAXKV_ERR_TIMEOUT, KID_DENSE, (int)row, -1);
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);    // copies still in flight may land before the block leaves
  }
  __syncwarp();
}

// y = x / sqrt(mean(x^2) + eps) * w, one warp per row of C columns (C * 2 bytes a multiple of 16).
__global__ void __launch_bounds__(kRowWarps * 32)
rmsnorm_rows_bulk_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ w, uint16_t* __restrict__ y, long long n_rows,
                         int C, float eps, DeviceStatus* st) {
  extern __shared__ __align__(128) uint8_t row_stage[];      // [warp][C] bf16
  __shared__ __align__(8) unsigned long long bars[kRowWarps];
  __shared__ volatile int gave_up[kRowWarps];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * kRowWarps + warp;
  if (row >= n_rows) return;
  const uint32_t row_bytes = (uint32_t)C * 2;
  uint8_t* mine = row_stage + (size_t)warp * row_bytes;
  const uint32_t bar = smem_u32(&bars[warp]), dst = smem_u32(mine);
  if (lane == 0) {
    gave_up[warp] = 0;
    mbar_init(bar, 1);
    fence_barrier_init();
    mbar_expect_tx(bar, row_bytes);
    bulk_load(dst, x + row * C, row_bytes, bar);
  }
  __syncwarp();
  bool ok = true;
  if (lane == 0) ok = mbar_wait(bar, 0, &gave_up[warp]);
  ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
  if (!ok) { row_wait_failed(st, row); return; }
  float ss = 0.f;
  for (int i = lane * 8; i < C; i += 32 * 8) {
    float f[8];
    unpack8(*reinterpret_cast<const uint4*>(mine + i * 2), f);
#pragma unroll
    for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
  }
  ss = warp_reduce_sum(ss);
  const float inv = rsqrtf(ss / (float)C + eps);
  for (int i = lane * 8; i < C; i += 32 * 8) {
    float f[8], g[8];
    unpack8(*reinterpret_cast<const uint4*>(mine + i * 2), f);
    unpack8(__ldg(reinterpret_cast<const uint4*>(w + i)), g);
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = f[e] * inv * g[e];
    *reinterpret_cast<uint4*>(mine + i * 2) = pack8(f);
  }
  fence_proxy_async_smem();                                   // the lanes' writes, before the copy engine reads them
  __syncwarp();
  if (lane == 0) {
    bulk_store(y + row * C, dst, row_bytes);
    bulk_store_commit_and_drain();                            // shared memory must outlive the copy that reads it
  }
}

// Per-head RMSNorm (optional) + rotary embedding of one row of q [Hq, D] and k [Hkv, D] per warp, in place.  One head
// per half-warp: a lane holds D/32 consecutive dims of the first half of the head vector and the same dims of the
// second half (both members of its rotation pairs), their cos / sin (computed by the lane itself, angle reduced in
// double) and norm weights in registers for all heads of the row.
template <int D>
__global__ void __launch_bounds__(kRowWarps * 32)
head_norm_rope_rows_bulk_kernel(uint16_t* __restrict__ q, uint16_t* __restrict__ k, long long n_rows, int Hq, int Hkv,
                                const uint16_t* __restrict__ wq, const uint16_t* __restrict__ wk, float eps,
                                const int* __restrict__ positions, double log2_theta, DeviceStatus* st) {
  constexpr int P = D / 32, half = D / 2;
  extern __shared__ __align__(128) uint8_t row_stage[];      // [warp][Hq + Hkv][D] bf16
  __shared__ __align__(8) unsigned long long bars[kRowWarps];
  __shared__ volatile int gave_up[kRowWarps];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * kRowWarps + warp;
  if (row >= n_rows) return;
  const uint32_t q_bytes = (uint32_t)Hq * D * 2, k_bytes = (uint32_t)Hkv * D * 2;
  uint8_t* mine = row_stage + (size_t)warp * (q_bytes + k_bytes);
  const uint32_t bar = smem_u32(&bars[warp]), dst = smem_u32(mine);
  if (lane == 0) {
    gave_up[warp] = 0;
    mbar_init(bar, 1);
    fence_barrier_init();
    mbar_expect_tx(bar, q_bytes + k_bytes);
    bulk_load(dst, q + row * Hq * D, q_bytes, bar);
    bulk_load(dst + q_bytes, k + row * Hkv * D, k_bytes, bar);
  }
  __syncwarp();
  // while the row travels: this lane's cos / sin and norm weights
  const int d0 = (lane & 15) * P;
  float cs[P], sn[P], wq_lo[P], wq_hi[P], wk_lo[P], wk_hi[P];
  {
    const double pos = (double)positions[row];
#pragma unroll
    for (int e = 0; e < P; ++e) {
      const double inv_freq = exp2(-log2_theta * (2.0 * (d0 + e) / D));
      double ang = pos * inv_freq;
      ang -= 6.283185307179586 * floor(ang * 0.15915494309189535);
      sincosf((float)ang, &sn[e], &cs[e]);
      wq_lo[e] = wq_hi[e] = wk_lo[e] = wk_hi[e] = 1.f;
    }
    if (wq != nullptr) {
#pragma unroll
      for (int e = 0; e < P; ++e) {
        wq_lo[e] = bf16_bits_to_float(wq[d0 + e]); wq_hi[e] = bf16_bits_to_float(wq[half + d0 + e]);
        wk_lo[e] = bf16_bits_to_float(wk[d0 + e]); wk_hi[e] = bf16_bits_to_float(wk[half + d0 + e]);
      }
    }
  }
  bool ok = true;
  if (lane == 0) ok = mbar_wait(bar, 0, &gave_up[warp]);
  ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
  if (!ok) { row_wait_failed(st, row); return; }
  const int n_heads = Hq + Hkv;
  for (int h0 = 0; h0 < n_heads; h0 += 2) {                   // both half-warps stay in step for the shuffles
    const int h = h0 + (lane >> 4);
    const bool live = h < n_heads;
    uint8_t* v = mine + (size_t)(live ? h : h0) * D * 2;      // q heads first, then the k heads: contiguous in the stage
    float lo[P], hi[P];
    if constexpr (P == 4) {
      const uint2 a = *reinterpret_cast<const uint2*>(v + d0 * 2), b = *reinterpret_cast<const uint2*>(v + (half + d0) * 2);
      lo[0] = __uint_as_float(a.x << 16); lo[1] = __uint_as_float(a.x & 0xffff0000u);
      lo[2] = __uint_as_float(a.y << 16); lo[3] = __uint_as_float(a.y & 0xffff0000u);
      hi[0] = __uint_as_float(b.x << 16); hi[1] = __uint_as_float(b.x & 0xffff0000u);
      hi[2] = __uint_as_float(b.y << 16); hi[3] = __uint_as_float(b.y & 0xffff0000u);
    } else {
      const uint32_t a = *reinterpret_cast<const uint32_t*>(v + d0 * 2), b = *reinterpret_cast<const uint32_t*>(v + (half + d0) * 2);
      lo[0] = __uint_as_float(a << 16); lo[1] = __uint_as_float(a & 0xffff0000u);
      hi[0] = __uint_as_float(b << 16); hi[1] = __uint_as_float(b & 0xffff0000u);
    }
    if (wq != nullptr) {
      float ss = 0.f;
#pragma unroll
      for (int e = 0; e < P; ++e) { ss = fmaf(lo[e], lo[e], ss); ss = fmaf(hi[e], hi[e], ss); }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);         // over the half-warp of this head
      const bool is_q = h < Hq;
      const float inv = rsqrtf(ss / (float)D + eps);
#pragma unroll
      for (int e = 0; e < P; ++e) {
        lo[e] = __bfloat162float(__float2bfloat16(lo[e] * inv * (is_q ? wq_lo[e] : wk_lo[e])));
        hi[e] = __bfloat162float(__float2bfloat16(hi[e] * inv * (is_q ? wq_hi[e] : wk_hi[e])));
      }
    }
    if (live) {
      float rl[P], rh[P];
#pragma unroll
      for (int e = 0; e < P; ++e) {
        rl[e] = lo[e] * cs[e] - hi[e] * sn[e];
        rh[e] = hi[e] * cs[e] + lo[e] * sn[e];
      }
      const __nv_bfloat162 l01 = __floats2bfloat162_rn(rl[0], rl[1]), h01 = __floats2bfloat162_rn(rh[0], rh[1]);
      if constexpr (P == 4) {
        const __nv_bfloat162 l23 = __floats2bfloat162_rn(rl[2], rl[3]), h23 = __floats2bfloat162_rn(rh[2], rh[3]);
        *reinterpret_cast<uint2*>(v + d0 * 2) = make_uint2(*reinterpret_cast<const uint32_t*>(&l01), *reinterpret_cast<const uint32_t*>(&l23));
        *reinterpret_cast<uint2*>(v + (half + d0) * 2) = make_uint2(*reinterpret_cast<const uint32_t*>(&h01), *reinterpret_cast<const uint32_t*>(&h23));
      } else {
        *reinterpret_cast<uint32_t*>(v + d0 * 2) = *reinterpret_cast<const uint32_t*>(&l01);
        *reinterpret_cast<uint32_t*>(v + (half + d0) * 2) = *reinterpret_cast<const uint32_t*>(&h01);
      }
    }
  }
  fence_proxy_async_smem();
  __syncwarp();
  if (lane == 0) {
    bulk_store(q + row * Hq * D, dst, q_bytes);
    bulk_store(k + row * Hkv * D, dst + q_bytes, k_bytes);
    bulk_store_commit_and_drain();
  }
}

// out[r, i] = silu(gu[r, i]) * gu[r, I + i]
__global__ void swiglu_kernel(const uint16_t* __restrict__ gu, uint16_t* __restrict__ out, long long rows, int I) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int per_row = I / 8;
  if (idx >= rows * per_row) return;
  const long long r = idx / per_row;
  const int i = (int)(idx - r * per_row) * 8;
  float g[8], u[8];
  unpack8(__ldg(reinterpret_cast<const uint4*>(gu + r * 2 * I + i)), g);
  unpack8(__ldg(reinterpret_cast<const uint4*>(gu + r * 2 * I + I + i)), u);
#pragma unroll
  for (int e = 0; e < 8; ++e) g[e] = g[e] / (1.f + __expf(-g[e])) * u[e];
  *reinterpret_cast<uint4*>(out + r * I + i) = pack8(g);
}

// positions of the layer's active targets: pos[row] = u_pos[u_cu[b] + r_rank[r_cu[b] + rho]]
__global__ void target_positions_kernel(ReqTable rt, const int* __restrict__ u_pos, const int* __restrict__ u_cu,
                                        const int* __restrict__ r_rank, const int* __restrict__ r_cu, int* __restrict__ pos,
                                        DeviceStatus* st) {
  const int B = rt.n_req;
  const int y = blockIdx.x * blockDim.x + threadIdx.x;
  if (y >= rt.tile_cu[B]) return;
  const int b = find_segment(rt.tile_cu, B, y);
  const int rho = y - rt.tile_cu[b];
  const int nr = r_cu[b + 1] - r_cu[b];
  if (rho >= nr) return;
  const int c = r_rank[r_cu[b] + rho];
  const int nu = u_cu[b + 1] - u_cu[b];
  if (c < 0 || c >= nu) { report(st, RELAXKV_ERR_BAD_INDEX, KID_DENSE, c, nu); return; }
  pos[r_cu[b] - r_cu[0] + rho] = u_pos[u_cu[b] + c];
}

// Hidden rows that stay active: for each target of layer l+1 (rank c), its row among layer l's targets.
// One block copies one row (C a multiple of 8).
__global__ void __launch_bounds__(128)
carry_rows_kernel(ReqTable rt, const uint16_t* __restrict__ h_in, uint16_t* __restrict__ h_out, int C,
                  const int* __restrict__ r_rank, const int* __restrict__ r_cu_l, const int* __restrict__ r_cu_next,
                  DeviceStatus* st) {
  const int B = rt.n_req;
  __shared__ long long src_row;
  const int y = blockIdx.x;
  const int b = find_segment(rt.tile_cu, B, y);
  const int rho = y - rt.tile_cu[b];
  const int n_next = r_cu_next[b + 1] - r_cu_next[b];
  if (rho >= n_next) return;
  if (threadIdx.x == 0) {
    const int c = r_rank[r_cu_next[b] + rho];
    const int* list = r_rank + r_cu_l[b];
    const int n_l = r_cu_l[b + 1] - r_cu_l[b];
    int lo = 0, hi = n_l;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (list[mid] < c) lo = mid + 1; else hi = mid; }
    if (lo >= n_l || list[lo] != c) { report(st, RELAXKV_ERR_BAD_INDEX, KID_DENSE, c, lo); src_row = -1; }
    else src_row = (long long)(r_cu_l[b] - r_cu_l[0]) + lo;
  }
  __syncthreads();
  if (src_row < 0) return;
  const long long dst_row = (long long)(r_cu_next[b] - r_cu_next[0]) + rho;
  for (int i = threadIdx.x * 8; i < C; i += 128 * 8)
    *reinterpret_cast<uint4*>(h_out + dst_row * C + i) = __ldg(reinterpret_cast<const uint4*>(h_in + src_row * C + i));
}

// The same for many rows: one warp per row, the row travels through shared memory by bulk copies (see above).
__global__ void __launch_bounds__(kRowWarps * 32)
carry_rows_bulk_kernel(ReqTable rt, const uint16_t* __restrict__ h_in, uint16_t* __restrict__ h_out, int C,
                       const int* __restrict__ r_rank, const int* __restrict__ r_cu_l, const int* __restrict__ r_cu_next,
                       DeviceStatus* st) {
  extern __shared__ __align__(128) uint8_t row_stage[];      // [warp][C] bf16
  __shared__ __align__(8) unsigned long long bars[kRowWarps];
  __shared__ volatile int gave_up[kRowWarps];
  const int B = rt.n_req;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long y = (long long)blockIdx.x * kRowWarps + warp;
  if (y >= rt.tile_cu[B] || lane != 0) return;                // one lane per row does everything: search, load, store
  const int b = find_segment(rt.tile_cu, B, (int)y);
  const int rho = (int)y - rt.tile_cu[b];
  const int n_next = r_cu_next[b + 1] - r_cu_next[b];
  if (rho >= n_next) return;
  const int c = r_rank[r_cu_next[b] + rho];
  const int* list = r_rank + r_cu_l[b];
  const int n_l = r_cu_l[b + 1] - r_cu_l[b];
  int lo = 0, hi = n_l;
  while (lo < hi) { const int mid = (lo + hi) >> 1; if (list[mid] < c) lo = mid + 1; else hi = mid; }
  if (lo >= n_l || list[lo] != c) { report(st, RELAXKV_ERR_BAD_INDEX, KID_DENSE, c, lo); return; }
  const long long src_row = (long long)(r_cu_l[b] - r_cu_l[0]) + lo;
  const long long dst_row = (long long)(r_cu_next[b] - r_cu_next[0]) + rho;
  const uint32_t row_bytes = (uint32_t)C * 2;
  const uint32_t bar = smem_u32(&bars[warp]), stage = smem_u32(row_stage + (size_t)warp * row_bytes);
  gave_up[warp] = 0;
  mbar_init(bar, 1);
  fence_barrier_init();
  mbar_expect_tx(bar, row_bytes);
  bulk_load(stage, h_in + src_row * C, row_bytes, bar);
  if (!mbar_wait(bar, 0, &gave_up[warp])) {
    report(st, RELAXKV_ERR_TIMEOUT, KID_DENSE, (int)y, -1);
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    return;
  }
  bulk_store(h_out + dst_row * C, stage, row_bytes);
  bulk_store_commit_and_drain();
}

}  // namespace relaxkv

using namespace relaxkv;

extern "C" relaxkv_status relaxkv_rmsnorm(const void* x, const void* weight, void* y, int64_t n_rows, int32_t n_cols,
                                          float eps, relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_rmsnorm");
  if (!x || !weight || !y || !aligned16(x) || !aligned16(weight) || !aligned16(y) || !(eps >= 0.f)) return RELAXKV_ERR_INVALID_ARG;
  if (n_rows < 0 || n_cols < 8 || (n_cols % 8)) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (n_rows == 0) return RELAXKV_OK;
  if (n_cols <= 256) {
    const long long blocks = (n_rows * 32 + 255) / 256;
    if (blocks > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
    return cuda_ok(launch_chained(n_rows <= kChainedMaxRows, rmsnorm_short_kernel, (unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream),
                                  static_cast<const uint16_t*>(x), static_cast<const uint16_t*>(weight),
                                  static_cast<uint16_t*>(y), (long long)n_rows, n_cols, eps));
  }
  if (n_rows > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (n_rows >= kRowBulkMinRows && n_cols * 2 <= kRowBulkMaxBytes) {
    DeviceStatus* st = status_word();
    if (!st) return RELAXKV_ERR_CUDA;
    const size_t smem = (size_t)kRowWarps * n_cols * 2;
    if (smem > 48 * 1024 - 256 &&
        cudaFuncSetAttribute(rmsnorm_rows_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return RELAXKV_ERR_CUDA;
    rmsnorm_rows_bulk_kernel<<<(unsigned)((n_rows + kRowWarps - 1) / kRowWarps), kRowWarps * 32, smem, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint16_t*>(x), static_cast<const uint16_t*>(weight), static_cast<uint16_t*>(y), (long long)n_rows, n_cols, eps, st);
    return launch_ok();
  }
  return cuda_ok(launch_chained(n_rows <= kChainedMaxRows, rmsnorm_kernel, (unsigned)n_rows, 256, 0, static_cast<cudaStream_t>(stream),
                                static_cast<const uint16_t*>(x), static_cast<const uint16_t*>(weight),
                                static_cast<uint16_t*>(y), n_cols, eps));
}

extern "C" relaxkv_status relaxkv_rope(void* x, int64_t n_rows, int32_t n_heads, int32_t head_dim, const int32_t* positions,
                                       float theta, relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_rope");
  if (!x || !positions || !aligned16(x) || !(theta > 1.f)) return RELAXKV_ERR_INVALID_ARG;
  if (n_rows < 0 || n_heads < 1 || (head_dim != 64 && head_dim != 128)) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (n_rows == 0) return RELAXKV_OK;
  const long long n = n_rows * (head_dim / 16);
  rope_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<uint16_t*>(x), n_rows, n_heads, head_dim, positions, log2((double)theta));
  return launch_ok();
}

extern "C" relaxkv_status relaxkv_qk_norm_rope(void* q, void* k, int64_t n_rows, int32_t n_q_heads, int32_t n_kv_heads,
                                               int32_t head_dim, const void* w_q_norm, const void* w_k_norm, float eps,
                                               const int32_t* positions, float theta, relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_qk_norm_rope");
  if (!q || !k || !positions || !aligned16(q) || !aligned16(k) || !(theta > 1.f) || !(eps >= 0.f)) return RELAXKV_ERR_INVALID_ARG;
  if ((w_q_norm == nullptr) != (w_k_norm == nullptr)) return RELAXKV_ERR_INVALID_ARG;
  if (n_rows < 0 || n_q_heads < 1 || n_kv_heads < 1 || (head_dim != 64 && head_dim != 128)) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (n_rows == 0) return RELAXKV_OK;
  if (n_rows > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int heads_per_block = (n_rows >= 2048) ? n_q_heads + n_kv_heads : 4;
  const dim3 grid((unsigned)n_rows, (unsigned)((n_q_heads + n_kv_heads + heads_per_block - 1) / heads_per_block));
  uint16_t* qp = static_cast<uint16_t*>(q);
  uint16_t* kp = static_cast<uint16_t*>(k);
  const uint16_t* wq = static_cast<const uint16_t*>(w_q_norm);
  const uint16_t* wk = static_cast<const uint16_t*>(w_k_norm);
  // in double: a float log2(theta) is off by 1e-6, which at positions of tens of thousands turns the phase by 1e-3 rad
  const double log2_theta = log2((double)theta);
  const size_t row_bytes = (size_t)(n_q_heads + n_kv_heads) * head_dim * 2;
  if (n_rows >= kRowBulkMinRows && row_bytes <= (size_t)kRowBulkMaxBytes && (n_q_heads * head_dim * 2) % 16 == 0 &&
      (n_kv_heads * head_dim * 2) % 16 == 0) {
    DeviceStatus* dst = status_word();
    if (!dst) return RELAXKV_ERR_CUDA;
    const size_t smem = kRowWarps * row_bytes;
    auto kern = head_dim == 128 ? head_norm_rope_rows_bulk_kernel<128> : head_norm_rope_rows_bulk_kernel<64>;
    if (smem > 48 * 1024 - 256 && cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return RELAXKV_ERR_CUDA;
    kern<<<(unsigned)((n_rows + kRowWarps - 1) / kRowWarps), kRowWarps * 32, smem, st>>>(qp, kp, (long long)n_rows, n_q_heads, n_kv_heads,
                                                                                       wq, wk, eps, positions, log2_theta, dst);
    return launch_ok();
  }
  if (head_dim == 128)
    return cuda_ok(launch_chained(n_rows <= kChainedMaxRows, head_norm_rope_kernel<128>, grid, 128, 0, st, qp, kp, n_q_heads, n_kv_heads, heads_per_block,
                                  wq, wk, eps, positions, log2_theta));
  return cuda_ok(launch_chained(n_rows <= kChainedMaxRows, head_norm_rope_kernel<64>, grid, 128, 0, st, qp, kp, n_q_heads, n_kv_heads, heads_per_block,
                                wq, wk, eps, positions, log2_theta));
}

extern "C" relaxkv_status relaxkv_swiglu(const void* gate_up, void* out, int64_t n_rows, int32_t n_inter, relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_swiglu");
  if (!gate_up || !out || !aligned16(gate_up) || !aligned16(out)) return RELAXKV_ERR_INVALID_ARG;
  if (n_rows < 0 || n_inter < 8 || (n_inter % 8)) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (n_rows == 0) return RELAXKV_OK;
  const long long n = n_rows * (n_inter / 8);
  swiglu_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint16_t*>(gate_up), static_cast<uint16_t*>(out), n_rows, n_inter);
  return launch_ok();
}

extern "C" relaxkv_status relaxkv_target_positions(const relaxkv_shape* shape, const int32_t* u_pos, const int32_t* u_cu,
                                                   const int32_t* r_rank, const int32_t* r_cu_layer,
                                                   const int32_t* h_max_targets, int32_t* positions_out, relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_target_positions");
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if (!u_pos || !u_cu || !r_rank || !r_cu_layer || !h_max_targets || !positions_out) return RELAXKV_ERR_INVALID_ARG;
  ReqTable rt;
  fill_req_table(rt, shape, nullptr, nullptr);
  long long total = 0;
  for (int b = 0; b < shape->n_req; ++b) {
    if (h_max_targets[b] < 0) return RELAXKV_ERR_INVALID_ARG;
    total += h_max_targets[b];
    rt.tile_cu[b + 1] = (int)total;
  }
  if (total == 0) return RELAXKV_OK;
  if (total > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  target_positions_kernel<<<(unsigned)((total + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      rt, u_pos, u_cu, r_rank, r_cu_layer, positions_out, st);
  return launch_ok();
}

extern "C" relaxkv_status relaxkv_carry_rows(const relaxkv_shape* shape, const void* h_in, void* h_out, int32_t n_cols,
                                             const int32_t* r_rank, const int32_t* r_cu_layer, const int32_t* r_cu_next,
                                             const int32_t* h_max_next, relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_carry_rows");
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if (!h_in || !h_out || !r_rank || !r_cu_layer || !r_cu_next || !h_max_next || !aligned16(h_in) || !aligned16(h_out))
    return RELAXKV_ERR_INVALID_ARG;
  if (n_cols < 8 || (n_cols % 8)) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  ReqTable rt;
  fill_req_table(rt, shape, nullptr, nullptr);
  long long total = 0;
  for (int b = 0; b < shape->n_req; ++b) {
    if (h_max_next[b] < 0) return RELAXKV_ERR_INVALID_ARG;
    total += h_max_next[b];
    rt.tile_cu[b + 1] = (int)total;
  }
  if (total == 0) return RELAXKV_OK;
  if (total > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  if (total >= kRowBulkMinRows && n_cols * 2 <= kRowBulkMaxBytes) {
    const size_t smem = (size_t)kRowWarps * n_cols * 2;
    if (smem > 48 * 1024 - 256 &&
        cudaFuncSetAttribute(carry_rows_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return RELAXKV_ERR_CUDA;
    carry_rows_bulk_kernel<<<(unsigned)((total + kRowWarps - 1) / kRowWarps), kRowWarps * 32, smem, static_cast<cudaStream_t>(stream)>>>(
        rt, static_cast<const uint16_t*>(h_in), static_cast<uint16_t*>(h_out), n_cols, r_rank, r_cu_layer, r_cu_next, st);
    return launch_ok();
  }
  carry_rows_kernel<<<(unsigned)total, 128, 0, static_cast<cudaStream_t>(stream)>>>(
      rt, static_cast<const uint16_t*>(h_in), static_cast<uint16_t*>(h_out), n_cols, r_rank, r_cu_layer, r_cu_next, st);
  return launch_ok();
}
