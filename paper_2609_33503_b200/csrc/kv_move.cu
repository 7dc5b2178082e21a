// Bandwidth kernels of the repair path: the materialised mixed fresh/cached context (gather) and
// the cache update (scatter).  Pure bit copies, HBM-bound: whole token rows travel through shared memory with bulk
// asynchronous copies.
#include "common.cuh"
#include "kv_move.cuh"
#include "sm100_ptx.cuh"

namespace relaxkv {

#ifndef RELAXKV_GATHER_ROWS_PER_WARP
#define RELAXKV_GATHER_ROWS_PER_WARP 4
#endif
#ifndef RELAXKV_SCATTER_ROWS
#define RELAXKV_SCATTER_ROWS 32
#endif

// Warp-cooperative lower bound on an ascending list: 32 pivots per round instead of one.
// Returns the first index with a[idx] >= key (n if none).  All lanes get the result.
__device__ __forceinline__ int warp_lower_bound(const int* __restrict__ a, int n, int key, int lane) {
  int lo = 0, hi = n;                     // the answer lies in [lo, hi]
  while (hi > lo) {
    const int step = (hi - lo + 31) / 32;
    const int idx = lo + lane * step;
    const bool lt = (idx < hi) && (__ldg(a + idx) < key);
    const int n_lt = __popc(__ballot_sync(0xffffffffu, lt));   // pivots below the key: a prefix of the lanes
    if (n_lt == 0) {
      hi = lo;
    } else {
      hi = min(hi, lo + n_lt * step);
      lo = lo + (n_lt - 1) * step + 1;
    }
  }
  return lo;
}

// Rows travel global -> shared -> global through the copy engine (bulk asynchronous copies, this GPU's memory only,
// never multicast), so no thread ever holds the data and one lane keeps many kilobytes in flight.
using namespace ptx;

// After an expired wait the copies may still be in flight: give them time to land before the block's shared memory
// goes away (bounded; the same grace period the tensor-core kernels take).
__device__ __forceinline__ void grace_period() {
  const uint64_t t0 = global_timer_ns();
  while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
}

constexpr int kMoveWarps = 2;              // warps per block; every warp works on its own rows, no block-wide barrier
constexpr int kMoveMaxRowsPerWarp = 4;     // rows one warp stages at a time (its first lanes issue the copies)
constexpr int kMoveThreads = kMoveWarps * 32;
constexpr int kMoveWarpStageBytes = 4096;  // staging per warp: one token's K row + V row at 8 KV heads of 128 (measured best:
                                           // small blocks, many of them resident; 2 x 4096 B gave 0.85 of the copy bandwidth,
                                           // 4 x 16384 B 0.76)
constexpr int kMoveMaxSmem = 200 * 1024;

// Rows per warp and dynamic shared memory per block for rows of `row_bytes` bytes per tensor (K and V staged back to
// back).  0 rows: the shape is too large for the staging scheme.
inline void move_geometry(size_t row_bytes, int* rows_per_warp, size_t* smem) {
  int r = (int)(kMoveWarpStageBytes / (2 * row_bytes));
  if (r > kMoveMaxRowsPerWarp) r = kMoveMaxRowsPerWarp;
  if (r < 1) r = 1;
  *smem = (size_t)kMoveWarps * r * 2 * row_bytes;
  *rows_per_warp = (*smem <= (size_t)kMoveMaxSmem) ? r : 0;
}

// Copies one token row (all KV heads) of K and of V: global -> shared (issue) ...
__device__ __forceinline__ void issue_row_loads(uint32_t dst, const uint16_t* k_src, const uint16_t* v_src, int n_kv_heads,
                                                int head_dim, long long src_head_stride, uint32_t bar) {
  const uint32_t head_bytes = (uint32_t)head_dim * 2, row_bytes = head_bytes * n_kv_heads;
  if (src_head_stride == head_dim) {        // heads contiguous: one copy per tensor
    bulk_load(dst, k_src, row_bytes, bar);
    bulk_load(dst + row_bytes, v_src, row_bytes, bar);
  } else {
    for (int g = 0; g < n_kv_heads; ++g) {
      bulk_load(dst + g * head_bytes, k_src + g * src_head_stride, head_bytes, bar);
      bulk_load(dst + row_bytes + g * head_bytes, v_src + g * src_head_stride, head_bytes, bar);
    }
  }
}
// ... and shared -> global (issue; the caller commits and drains)
__device__ __forceinline__ void issue_row_stores(uint16_t* k_dst, uint16_t* v_dst, uint32_t src, int n_kv_heads, int head_dim,
                                                 long long dst_head_stride) {
  const uint32_t head_bytes = (uint32_t)head_dim * 2, row_bytes = head_bytes * n_kv_heads;
  if (dst_head_stride == head_dim) {
    bulk_store(k_dst, src, row_bytes);
    bulk_store(v_dst, src + row_bytes, row_bytes);
  } else {
    for (int g = 0; g < n_kv_heads; ++g) {
      bulk_store(k_dst + g * dst_head_stride, src + g * head_bytes, head_bytes);
      bulk_store(v_dst + g * dst_head_stride, src + row_bytes + g * head_bytes, head_bytes);
    }
  }
}

// Context row x of request b is the fresh state of target rho if its context entry is an active
// target of this layer, else the cached state at that position (Section 3.4 equation).
// A warp owns a few (rows_per_warp) consecutive context rows: it resolves their sources (one search of the layer's R list
// for the first row, a walk for the others), its first lanes then issue the bulk copies of one row each into the warp's
// staging area, and once they have landed the same lanes issue the copies to the materialised context.
__global__ void __launch_bounds__(kMoveThreads)
gather_ctx_kernel(ReqTable rt, int mode, int n_kv_heads, int head_dim,
                  const uint16_t* __restrict__ cache_k, const uint16_t* __restrict__ cache_v,
                  long long tok_stride, long long head_stride,
                  const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                  const int* __restrict__ u_pos, const int* __restrict__ u_cu,
                  const int* __restrict__ r_rank, const int* __restrict__ r_cu, const int* __restrict__ fresh_row,
                  uint16_t* __restrict__ k_out, uint16_t* __restrict__ v_out, long long ctx_rows,
                  long long fresh_map_rows, long long n_new_rows, int rows_per_warp, DeviceStatus* st) {
  // fresh_map_rows: entries of fresh_row that were written (the host bound on the context rows of an explicit-list
  // call); n_new_rows: rows k_new / v_new hold.  An index past either is reported and the row zero-filled.
  extern __shared__ __align__(128) uint8_t stage[];          // [warp][row of the warp][K row | V row]
  __shared__ __align__(8) unsigned long long bars[kMoveWarps];
  __shared__ volatile int gave_up[kMoveWarps];
  const int B = rt.n_req;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long x0 = ((long long)blockIdx.x * kMoveWarps + warp) * rows_per_warp;
  if (x0 >= ctx_rows) return;
  const uint32_t bar = smem_u32(&bars[warp]);
  if (lane == 0) { gave_up[warp] = 0; mbar_init(bar, 1); fence_barrier_init(); }
  const long long total = (mode == RELAXKV_CTX_UNION) ? (long long)__ldg(u_cu + B) : rt.ctx_cu[B];
  const uint32_t row_bytes = (uint32_t)n_kv_heads * head_dim * 2;
  const uint32_t my_stage = smem_u32(stage) + (uint32_t)(warp * rows_per_warp + lane) * 2u * row_bytes;   // lanes < rows_per_warp
  int my_kind = 3;                             // lane rr keeps the source of row rr: 0 = cache, 1 = fresh, 2 = zero fill, 3 = skip
  long long my_off = 0;
  int prev_b = -1, rho_next = 0;               // the R list of request prev_b has been walked up to rho_next
  for (int rr = 0; rr < rows_per_warp; ++rr) {
    const long long x = x0 + rr;
    int kind = 3;
    long long off = 0;
    if (x < ctx_rows) {
      if (x >= total) {
        kind = (x < total + kCtxPadRows) ? 2 : 3;
      } else {
        int b = 0, c = -1, p;
        if (mode == RELAXKV_CTX_UNION) {
          while (b + 1 < B && x >= __ldg(u_cu + b + 1)) ++b;
          c = (int)(x - __ldg(u_cu + b));
          p = __ldg(u_pos + x);
        } else {
          while (b + 1 < B && x >= rt.ctx_cu[b + 1]) ++b;
          p = (int)(x - rt.ctx_cu[b]);
          const int ub = __ldg(u_cu + b), nu = __ldg(u_cu + b + 1) - ub;
          const int lb = warp_lower_bound(u_pos + ub, nu, p, lane);
          if (lb < nu && __ldg(u_pos + ub + lb) == p) c = lb;
        }
        if (p < 0 || p >= rt.ctx_len[b]) {
          if (lane == 0) report(st, RELAXKV_ERR_BAD_INDEX, KID_GATHER, (int)x, p);
          kind = 2;
        } else {
          kind = 0;
          off = (rt.tok_off[b] + p) * tok_stride;
          if (k_new != nullptr && fresh_row != nullptr) {
            // explicit lists: the row of k_new that replaces this context entry was resolved beforehand
            if (x >= fresh_map_rows) {
              if (lane == 0) report(st, RELAXKV_ERR_BAD_INDEX, KID_GATHER, (int)x, (int)fresh_map_rows);
              kind = 2;
            } else {
              const int fr = __ldg(fresh_row + x);
              if (fr >= n_new_rows) {
                if (lane == 0) report(st, RELAXKV_ERR_BAD_INDEX, KID_GATHER, (int)x, fr);
                kind = 2;
              } else if (fr >= 0) {
                kind = 1; off = (long long)fr * n_kv_heads * head_dim;
              }
            }
          } else if (k_new != nullptr && c >= 0) {
            const int rb = __ldg(r_cu + b), nr = __ldg(r_cu + b + 1) - rb;
            // first index of the R list with rank >= c: searched for the warp's first row of a request, then the
            // list is walked (consecutive context ranks: the answer moves by at most one entry per row)
            int rho;
            if (b == prev_b) {
              rho = rho_next;
              while (rho < nr && __ldg(r_rank + rb + rho) < c) ++rho;     // only after a malformed (unsorted) list
            } else {
              rho = warp_lower_bound(r_rank + rb, nr, c, lane);
            }
            prev_b = b;
            rho_next = rho;
            if (rho < nr && __ldg(r_rank + rb + rho) == c) {
              rho_next = rho + 1;
              const long long frow = (long long)(rb - __ldg(r_cu)) + rho;
              if (frow >= n_new_rows) {
                if (lane == 0) report(st, RELAXKV_ERR_BAD_INDEX, KID_GATHER, (int)x, (int)frow);
                kind = 2;
              } else {
                kind = 1;
                off = frow * n_kv_heads * head_dim;
              }
            }
          }
        }
      }
    }
    if (lane == rr) { my_kind = kind; my_off = off; }
  }
  // rows that are copied: how many bytes the warp's barrier has to see
  const unsigned copy_mask = __ballot_sync(0xffffffffu, lane < rows_per_warp && my_kind <= 1);
  __syncwarp();
  if (lane == 0 && copy_mask) mbar_expect_tx(bar, (uint32_t)__popc(copy_mask) * 2u * row_bytes);
  __syncwarp();
  if (lane < rows_per_warp) {
    if (my_kind == 0)
      issue_row_loads(my_stage, cache_k + my_off, cache_v + my_off, n_kv_heads, head_dim, head_stride, bar);
    else if (my_kind == 1)
      issue_row_loads(my_stage, k_new + my_off, v_new + my_off, n_kv_heads, head_dim, head_dim, bar);
  }
  // zero-fill rows (the pad after the context, rows with a reported index): plain stores by the whole warp
  for (int rr = 0; rr < rows_per_warp; ++rr) {
    if (__shfl_sync(0xffffffffu, my_kind, rr) == 2) {
      const long long o = (x0 + rr) * n_kv_heads * head_dim;
      for (int i = lane; i < (int)(row_bytes / 16); i += 32) {
        *reinterpret_cast<uint4*>(k_out + o + i * 8) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(v_out + o + i * 8) = make_uint4(0, 0, 0, 0);
      }
    }
  }
  if (copy_mask) {
    bool ok = true;
    if (lane == 0) ok = mbar_wait(bar, 0, &gave_up[warp]);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (!ok) {
      if (lane == 0) { report(st, RELAXKV_ERR_TIMEOUT, KID_GATHER, (int)x0, -1); grace_period(); }
      __syncwarp();
    } else if (lane < rows_per_warp && my_kind <= 1) {
      const long long o = (x0 + lane) * n_kv_heads * head_dim;
      issue_row_stores(k_out + o, v_out + o, my_stage, n_kv_heads, head_dim, head_dim);
    }
    if (lane < rows_per_warp) bulk_store_commit_and_drain();      // shared memory must outlive the copies that read it
  }
}

// The fresh K/V of the active targets go into the cache (Section 3.4).  Same structure as the gather: a warp owns
// a few consecutive target rows, its first lanes resolve one destination each and move the row with bulk copies.
__global__ void __launch_bounds__(kMoveThreads)
scatter_kv_kernel(ReqTable rt, int n_kv_heads, int head_dim,
                  uint16_t* __restrict__ cache_k, uint16_t* __restrict__ cache_v,
                  long long tok_stride, long long head_stride,
                  const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                  const int* __restrict__ u_pos, const int* __restrict__ u_cu,
                  const int* __restrict__ r_rank, const int* __restrict__ r_cu, int direct, int rows_per_warp,
                  DeviceStatus* st) {
  // direct != 0: u_pos holds the targets' positions themselves (packed by r_cu); r_rank is not read
  extern __shared__ __align__(128) uint8_t stage[];          // [warp][row of the warp][K row | V row]
  __shared__ __align__(8) unsigned long long bars[kMoveWarps];
  __shared__ volatile int gave_up[kMoveWarps];
  const int B = rt.n_req;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long y0 = ((long long)blockIdx.x * kMoveWarps + warp) * rows_per_warp;
  griddep_launch();
  griddep_wait();                              // the rows and the index lists come from earlier kernels
  if (y0 >= rt.tile_cu[B]) return;             // rt.tile_cu = prefix of the host bounds on |R_{l,b}|
  const uint32_t bar = smem_u32(&bars[warp]);
  if (lane == 0) { gave_up[warp] = 0; mbar_init(bar, 1); fence_barrier_init(); }
  const uint32_t row_bytes = (uint32_t)n_kv_heads * head_dim * 2;
  const uint32_t my_stage = smem_u32(stage) + (uint32_t)(warp * rows_per_warp + lane) * 2u * row_bytes;   // lanes < rows_per_warp
  long long d = -1, s = 0;
  if (lane < rows_per_warp) {
    const long long y = y0 + lane;
    if (y < rt.tile_cu[B]) {
      int b = 0;
      while (b + 1 < B && y >= rt.tile_cu[b + 1]) ++b;
      const int rho = (int)(y - rt.tile_cu[b]);
      const int nr = r_cu[b + 1] - r_cu[b];
      if (rho == 0 && nr > rt.bound_a[b]) report(st, RELAXKV_ERR_BAD_INDEX, KID_SCATTER, b, nr);
      if (rho < nr) {
        int c = -1, p = -1;
        if (direct) {
          p = u_pos[r_cu[b] + rho];
        } else {
          c = r_rank[r_cu[b] + rho];
          const int nu = u_cu[b + 1] - u_cu[b];
          if (c >= 0 && c < nu) p = u_pos[u_cu[b] + c];
        }
        if (p < 0 || p >= rt.ctx_len[b]) {
          report(st, RELAXKV_ERR_BAD_INDEX, KID_SCATTER, c, p);
        } else {
          d = (rt.tok_off[b] + p) * tok_stride;
          s = (long long)(r_cu[b] - r_cu[0] + rho) * n_kv_heads * head_dim;
        }
      }
    }
  }
  const unsigned copy_mask = __ballot_sync(0xffffffffu, d >= 0);
  if (!copy_mask) return;
  if (lane == 0) mbar_expect_tx(bar, (uint32_t)__popc(copy_mask) * 2u * row_bytes);
  __syncwarp();
  if (d >= 0) issue_row_loads(my_stage, k_new + s, v_new + s, n_kv_heads, head_dim, head_dim, bar);
  bool ok = true;
  if (lane == 0) ok = mbar_wait(bar, 0, &gave_up[warp]);
  ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
  if (!ok) {
    if (lane == 0) { report(st, RELAXKV_ERR_TIMEOUT, KID_SCATTER, (int)y0, -1); grace_period(); }
    __syncwarp();
  } else if (d >= 0) {
    issue_row_stores(cache_k + d, cache_v + d, my_stage, n_kv_heads, head_dim, head_stride);
  }
  if (lane < rows_per_warp) bulk_store_commit_and_drain();
}

relaxkv_status launch_gather(const relaxkv_shape* shape, int mode, const relaxkv_cache_view* cache,
                             const void* k_new, const void* v_new, const int32_t* u_pos, const int32_t* u_cu,
                             const int32_t* r_rank, const int32_t* r_cu_layer, const int32_t* fresh_row,
                             long long fresh_map_rows, long long n_new_rows,
                             long long rows_to_cover, void* k_out, void* v_out, long long ctx_rows, cudaStream_t stream) {
  ReqTable rt;
  fill_req_table(rt, shape, cache, nullptr);
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  if (rows_to_cover > ctx_rows) rows_to_cover = ctx_rows;
  if (rows_to_cover <= 0) return RELAXKV_OK;
  int rows_per_warp = 0;
  size_t smem = 0;
  move_geometry((size_t)shape->n_kv_heads * shape->head_dim * 2, &rows_per_warp, &smem);
  if (rows_per_warp == 0) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(gather_ctx_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return RELAXKV_ERR_CUDA;
  const long long rows_per_block = (long long)kMoveWarps * rows_per_warp;
  const long long blocks = (rows_to_cover + rows_per_block - 1) / rows_per_block;
  RELAXKV_RANGE("gather_ctx_kernel");
  gather_ctx_kernel<<<(unsigned)blocks, kMoveThreads, smem, stream>>>(
      rt, mode, shape->n_kv_heads, shape->head_dim,
      static_cast<const uint16_t*>(cache->k), static_cast<const uint16_t*>(cache->v),
      cache->token_stride, cache->head_stride,
      static_cast<const uint16_t*>(k_new), static_cast<const uint16_t*>(v_new),
      u_pos, u_cu, r_rank, r_cu_layer, fresh_row, static_cast<uint16_t*>(k_out), static_cast<uint16_t*>(v_out), ctx_rows,
      fresh_map_rows, n_new_rows, rows_per_warp, st);
  return launch_ok();
}

// Launches the cache update for `total` target rows (host bound); direct: see scatter_kv_kernel.
static relaxkv_status launch_scatter(const relaxkv_shape* shape, const ReqTable& rt, const relaxkv_cache_view* cache,
                                     const void* k_new, const void* v_new, const int32_t* u_pos, const int32_t* u_cu,
                                     const int32_t* r_rank, const int32_t* r_cu, int direct, long long total,
                                     cudaStream_t stream) {
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  int rows_per_warp = 0;
  size_t smem = 0;
  move_geometry((size_t)shape->n_kv_heads * shape->head_dim * 2, &rows_per_warp, &smem);
  if (rows_per_warp == 0) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(scatter_kv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return RELAXKV_ERR_CUDA;
  const long long rows_per_block = (long long)kMoveWarps * rows_per_warp;
  const long long blocks = (total + rows_per_block - 1) / rows_per_block;
  RELAXKV_RANGE("scatter_kv_kernel");
  return cuda_ok(launch_chained(total <= kChainedMaxRows, scatter_kv_kernel, (unsigned)blocks, kMoveThreads, smem, stream,
      rt, shape->n_kv_heads, shape->head_dim, static_cast<uint16_t*>(cache->k), static_cast<uint16_t*>(cache->v),
      (long long)cache->token_stride, (long long)cache->head_stride, static_cast<const uint16_t*>(k_new),
      static_cast<const uint16_t*>(v_new), u_pos, u_cu, r_rank, r_cu, direct, rows_per_warp, st));
}

}  // namespace relaxkv

using namespace relaxkv;

static relaxkv_status check_lists(const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank, const int32_t* r_cu) {
  return (u_pos && u_cu && r_rank && r_cu) ? RELAXKV_OK : RELAXKV_ERR_INVALID_ARG;
}

extern "C" relaxkv_status relaxkv_gather_kv(
    const relaxkv_shape* shape, relaxkv_ctx_mode mode, const relaxkv_cache_view* cache,
    const void* k_new, const void* v_new,
    const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank, const int32_t* r_cu_layer,
    const int32_t* h_max_ctx, void* k_ctx_out, void* v_ctx_out, int64_t ctx_rows, relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_gather_kv");
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if ((rc = check_cache(shape, cache, true)) != RELAXKV_OK) return rc;
  if ((rc = check_lists(u_pos, u_cu, r_rank, r_cu_layer)) != RELAXKV_OK) return rc;
  if (mode != RELAXKV_CTX_UNION && mode != RELAXKV_CTX_FULL_PREFIX) return RELAXKV_ERR_INVALID_ARG;
  if ((k_new == nullptr) != (v_new == nullptr)) return RELAXKV_ERR_INVALID_ARG;
  if (!k_ctx_out || !v_ctx_out || !aligned16(k_ctx_out) || !aligned16(v_ctx_out)) return RELAXKV_ERR_INVALID_ARG;
  if (k_new && (!aligned16(k_new) || !aligned16(v_new))) return RELAXKV_ERR_INVALID_ARG;
  long long need = 0;
  for (int b = 0; b < shape->n_req; ++b) {
    if (mode == RELAXKV_CTX_UNION) {
      if (!h_max_ctx || h_max_ctx[b] < 0) return RELAXKV_ERR_INVALID_ARG;
      need += h_max_ctx[b];
    } else {
      need += shape->h_ctx_len[b];
    }
  }
  if (ctx_rows < need) return RELAXKV_ERR_INVALID_ARG;
  // this entry point is not told how many rows k_new / v_new hold: the fresh-row index is bounded by the R list only
  return launch_gather(shape, mode, cache, k_new, v_new, u_pos, u_cu, r_rank, r_cu_layer, nullptr, 0, 0x7fffffffffffffffLL,
                       need + kCtxPadRows, k_ctx_out, v_ctx_out, ctx_rows, static_cast<cudaStream_t>(stream));
}

extern "C" relaxkv_status relaxkv_scatter_kv(
    const relaxkv_shape* shape, const relaxkv_cache_view* cache, const void* k_new, const void* v_new,
    const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank, const int32_t* r_cu_layer,
    const int32_t* h_max_targets, relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_scatter_kv");
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if ((rc = check_cache(shape, cache, true)) != RELAXKV_OK) return rc;
  if ((rc = check_lists(u_pos, u_cu, r_rank, r_cu_layer)) != RELAXKV_OK) return rc;
  if (!k_new || !v_new || !aligned16(k_new) || !aligned16(v_new) || !h_max_targets) return RELAXKV_ERR_INVALID_ARG;
  ReqTable rt;
  fill_req_table(rt, shape, cache, nullptr);
  long long total = 0;
  for (int b = 0; b < shape->n_req; ++b) {
    if (h_max_targets[b] < 0) return RELAXKV_ERR_INVALID_ARG;
    rt.bound_a[b] = h_max_targets[b];
    total += h_max_targets[b];
    if (total > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
    rt.tile_cu[b + 1] = (int)total;
  }
  if (total == 0) return RELAXKV_OK;
  return launch_scatter(shape, rt, cache, k_new, v_new, u_pos, u_cu, r_rank, r_cu_layer, 0, total, static_cast<cudaStream_t>(stream));
}

extern "C" relaxkv_status relaxkv_scatter_kv_lists(
    const relaxkv_shape* shape, const relaxkv_cache_view* cache, const void* k_new, const void* v_new,
    const int32_t* tgt_pos, const int32_t* tgt_cu, const int32_t* h_max_targets, relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_scatter_kv_lists");
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if ((rc = check_cache(shape, cache, true)) != RELAXKV_OK) return rc;
  if (!tgt_pos || !tgt_cu || !k_new || !v_new || !aligned16(k_new) || !aligned16(v_new) || !h_max_targets)
    return RELAXKV_ERR_INVALID_ARG;
  ReqTable rt;
  fill_req_table(rt, shape, cache, nullptr);
  long long total = 0;
  for (int b = 0; b < shape->n_req; ++b) {
    if (h_max_targets[b] < 0) return RELAXKV_ERR_INVALID_ARG;
    rt.bound_a[b] = h_max_targets[b];
    total += h_max_targets[b];
    if (total > 0x7fffffffLL) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
    rt.tile_cu[b + 1] = (int)total;
  }
  if (total == 0) return RELAXKV_OK;
  return launch_scatter(shape, rt, cache, k_new, v_new, tgt_pos, tgt_cu, tgt_pos, tgt_cu, 1, total, static_cast<cudaStream_t>(stream));
}
