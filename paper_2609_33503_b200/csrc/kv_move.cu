// Bandwidth kernels of the repair path: the materialised mixed fresh/cached context (gather) and
// the cache update (scatter).  Pure bit copies in 16-byte pieces; HBM-bound.
#include "common.cuh"
#include "kv_move.cuh"

namespace relaxkv {

constexpr int kGatherRows = 8;            // one warp resolves the source of one context row
constexpr int kGatherThreads = 256;

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

// One block moves kGatherRows context rows (all KV heads, K and V).
// Context row x of request b is the fresh state of target rho if its context entry is an active
// target of this layer, else the cached state at that position (Section 3.4 equation).
__global__ void __launch_bounds__(kGatherThreads)
gather_ctx_kernel(ReqTable rt, int mode, int n_kv_heads, int head_dim,
                  const uint16_t* __restrict__ cache_k, const uint16_t* __restrict__ cache_v,
                  long long tok_stride, long long head_stride,
                  const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                  const int* __restrict__ u_pos, const int* __restrict__ u_cu,
                  const int* __restrict__ r_rank, const int* __restrict__ r_cu, const int* __restrict__ fresh_row,
                  uint16_t* __restrict__ k_out, uint16_t* __restrict__ v_out, long long ctx_rows,
                  long long fresh_map_rows, long long n_new_rows, DeviceStatus* st) {
  // fresh_map_rows: entries of fresh_row that were written (the host bound on the context rows of an explicit-list
  // call); n_new_rows: rows k_new / v_new hold.  An index past either is reported and the row zero-filled.
  __shared__ long long src_off[kGatherRows];   // element offset of the source row (head 0)
  __shared__ int src_kind[kGatherRows];        // 0 = cache, 1 = fresh, 2 = zero fill, 3 = skip
  const long long row0 = (long long)blockIdx.x * kGatherRows;
  const int B = rt.n_req;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  {
    const long long x = row0 + warp;
    int kind = 3;
    long long off = 0;
    const long long total = (mode == RELAXKV_CTX_UNION) ? (long long)__ldg(u_cu + B) : rt.ctx_cu[B];
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
            const int rho = warp_lower_bound(r_rank + rb, nr, c, lane);
            if (rho < nr && __ldg(r_rank + rb + rho) == c) {
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
    if (lane == 0) { src_kind[warp] = kind; src_off[warp] = off; }
  }
  __syncthreads();
  const int pieces_per_head = head_dim / 8;                 // 16-byte pieces
  const int pieces_per_row = n_kv_heads * pieces_per_head;
  const int total_pieces = kGatherRows * pieces_per_row;
  for (int i0 = threadIdx.x; i0 < total_pieces; i0 += 4 * kGatherThreads) {
    uint4 kk[4], vv[4];
    long long dst[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {                            // issue every load before the first store
      const int i = i0 + u * kGatherThreads;
      kk[u] = make_uint4(0, 0, 0, 0); vv[u] = make_uint4(0, 0, 0, 0); dst[u] = -1;
      if (i < total_pieces) {
        const int r = i / pieces_per_row;
        const int kind = src_kind[r];
        if (kind != 3) {
          const int pr = i - r * pieces_per_row;
          const int g = pr / pieces_per_head;
          const int part = pr - g * pieces_per_head;
          dst[u] = ((row0 + r) * n_kv_heads + g) * head_dim + part * 8;
          if (kind == 0) {
            const long long so = src_off[r] + g * head_stride + part * 8;
            kk[u] = __ldg(reinterpret_cast<const uint4*>(cache_k + so));
            vv[u] = __ldg(reinterpret_cast<const uint4*>(cache_v + so));
          } else if (kind == 1) {
            const long long so = src_off[r] + (long long)g * head_dim + part * 8;
            kk[u] = __ldg(reinterpret_cast<const uint4*>(k_new + so));
            vv[u] = __ldg(reinterpret_cast<const uint4*>(v_new + so));
          }
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (dst[u] >= 0) {
        *reinterpret_cast<uint4*>(k_out + dst[u]) = kk[u];
        *reinterpret_cast<uint4*>(v_out + dst[u]) = vv[u];
      }
    }
  }
}

constexpr int kScatterRows = 4;
constexpr int kScatterThreads = 256;

// One block writes the fresh K/V of kScatterRows active targets into the cache (Section 3.4).
__global__ void __launch_bounds__(kScatterThreads)
scatter_kv_kernel(ReqTable rt, int n_kv_heads, int head_dim,
                  uint16_t* __restrict__ cache_k, uint16_t* __restrict__ cache_v,
                  long long tok_stride, long long head_stride,
                  const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                  const int* __restrict__ u_pos, const int* __restrict__ u_cu,
                  const int* __restrict__ r_rank, const int* __restrict__ r_cu, int direct, DeviceStatus* st) {
  // direct != 0: u_pos holds the targets' positions themselves (packed by r_cu); r_rank is not read
  __shared__ long long dst_off[kScatterRows];
  __shared__ long long src_off[kScatterRows];
  const int B = rt.n_req;
  if (threadIdx.x < kScatterRows) {
    // rt.tile_cu = prefix of the host bounds on |R_{l,b}|
    const int y = blockIdx.x * kScatterRows + threadIdx.x;
    long long d = -1, s = 0;
    if (y < rt.tile_cu[B]) {
      int b = 0;
      while (b + 1 < B && y >= rt.tile_cu[b + 1]) ++b;
      const int rho = y - rt.tile_cu[b];
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
    dst_off[threadIdx.x] = d;
    src_off[threadIdx.x] = s;
  }
  __syncthreads();
  const int pieces_per_head = head_dim / 8;
  const int pieces_per_row = n_kv_heads * pieces_per_head;
  const int total_pieces = kScatterRows * pieces_per_row;
  for (int i = threadIdx.x; i < total_pieces; i += kScatterThreads) {
    const int r = i / pieces_per_row;
    if (dst_off[r] < 0) continue;
    const int pr = i - r * pieces_per_row;
    const int g = pr / pieces_per_head;
    const int part = pr - g * pieces_per_head;
    const long long s = src_off[r] + (long long)g * head_dim + part * 8;
    const long long d = dst_off[r] + g * head_stride + part * 8;
    const uint4 kk = __ldg(reinterpret_cast<const uint4*>(k_new + s));
    const uint4 vv = __ldg(reinterpret_cast<const uint4*>(v_new + s));
    *reinterpret_cast<uint4*>(cache_k + d) = kk;
    *reinterpret_cast<uint4*>(cache_v + d) = vv;
  }
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
  const long long blocks = (rows_to_cover + kGatherRows - 1) / kGatherRows;
  gather_ctx_kernel<<<(unsigned)blocks, kGatherThreads, 0, stream>>>(
      rt, mode, shape->n_kv_heads, shape->head_dim,
      static_cast<const uint16_t*>(cache->k), static_cast<const uint16_t*>(cache->v),
      cache->token_stride, cache->head_stride,
      static_cast<const uint16_t*>(k_new), static_cast<const uint16_t*>(v_new),
      u_pos, u_cu, r_rank, r_cu_layer, fresh_row, static_cast<uint16_t*>(k_out), static_cast<uint16_t*>(v_out), ctx_rows,
      fresh_map_rows, n_new_rows, st);
  return launch_ok();
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
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  const long long blocks = (total + kScatterRows - 1) / kScatterRows;
  scatter_kv_kernel<<<(unsigned)blocks, kScatterThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      rt, shape->n_kv_heads, shape->head_dim, static_cast<uint16_t*>(cache->k), static_cast<uint16_t*>(cache->v),
      cache->token_stride, cache->head_stride, static_cast<const uint16_t*>(k_new),
      static_cast<const uint16_t*>(v_new), u_pos, u_cu, r_rank, r_cu_layer, 0, st);
  return launch_ok();
}

extern "C" relaxkv_status relaxkv_scatter_kv_lists(
    const relaxkv_shape* shape, const relaxkv_cache_view* cache, const void* k_new, const void* v_new,
    const int32_t* tgt_pos, const int32_t* tgt_cu, const int32_t* h_max_targets, relaxkv_stream stream) {
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
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  const long long blocks = (total + kScatterRows - 1) / kScatterRows;
  scatter_kv_kernel<<<(unsigned)blocks, kScatterThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      rt, shape->n_kv_heads, shape->head_dim, static_cast<uint16_t*>(cache->k), static_cast<uint16_t*>(cache->v),
      cache->token_stride, cache->head_stride, static_cast<const uint16_t*>(k_new),
      static_cast<const uint16_t*>(v_new), tgt_pos, tgt_cu, tgt_pos, tgt_cu, 1, st);
  return launch_ok();
}
