// Shared host/device helpers of the RelaxKV CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#ifdef RELAXKV_NVTX
#include <nvtx3/nvToolsExt.h>
#endif

#include "relaxkv.h"

namespace relaxkv {

// ---- device status word -----------------------------------------------------------------
// One int4 per device: {status, kernel id, block, value}.  Kernels record the first problem they
// see with an atomic compare-and-swap and carry on without touching the offending data.
struct DeviceStatus {
  int status;
  int kernel;
  int block;
  int v0;
  int v1;
};

// Per-device values that are looked up once (defined in api.cu).  The lookups are idempotent, so the caches are
// plain atomics: two host threads that race on a first call both store the same value.
constexpr int kMaxDevices = 64;
DeviceStatus* status_word();             // device address of the status word of the current device; NULL on error
int sm_count_of_current_device();        // multiprocessors of the current device; 0 on error

// Optional NVTX ranges, one per C-ABI call and per kernel launch, so that a timeline taken of a caller's process
// can be attributed to the steps of Algorithm 1.  Compiled in with -DRELAXKV_NVTX (build.py: RELAXKV_NVTX=1).
#ifdef RELAXKV_NVTX
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};
#define RELAXKV_RANGE_CAT2(a, b) a##b
#define RELAXKV_RANGE_CAT(a, b) RELAXKV_RANGE_CAT2(a, b)
#define RELAXKV_RANGE(name) ::relaxkv::NvtxRange RELAXKV_RANGE_CAT(relaxkv_nvtx_range_, __LINE__)(name)
#else
#define RELAXKV_RANGE(name) do { } while (0)
#endif

enum KernelId : int {
  KID_SETS = 1, KID_SELECT = 2, KID_SCORE = 3, KID_GATHER = 4, KID_SCATTER = 5,
  KID_ATTN_SIMT = 6, KID_ATTN_SM100 = 7, KID_SCORE_SM100 = 8, KID_GEMM_SM100 = 9, KID_DENSE = 10
};

__device__ __forceinline__ void report(DeviceStatus* st, int status, int kernel, int v0, int v1) {
  if (atomicCAS(&st->status, 0, status) == 0) {
    st->kernel = kernel;
    st->block = (int)blockIdx.x;
    st->v0 = v0;
    st->v1 = v1;
  }
}

// ---- host-side checks -------------------------------------------------------------------
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline relaxkv_status check_shape(const relaxkv_shape* s) {
  if (!s || !s->h_ctx_len) return RELAXKV_ERR_INVALID_ARG;
  if (s->n_req < 1 || s->n_q_heads < 1 || s->n_kv_heads < 1) return RELAXKV_ERR_INVALID_ARG;
  if (s->n_q_heads % s->n_kv_heads != 0) return RELAXKV_ERR_INVALID_ARG;
  if (s->head_dim != 64 && s->head_dim != 128) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (s->n_q_heads / s->n_kv_heads > 16) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  if (s->n_req > 64) return RELAXKV_ERR_UNSUPPORTED_SHAPE;   // per-request scalars travel by value
  for (int b = 0; b < s->n_req; ++b)
    if (s->h_ctx_len[b] < 1) return RELAXKV_ERR_INVALID_ARG;
  if (!(s->softmax_scale > 0.f)) return RELAXKV_ERR_INVALID_ARG;
  return RELAXKV_OK;
}

inline relaxkv_status check_cache(const relaxkv_shape* s, const relaxkv_cache_view* c, bool need_v) {
  if (!c || !c->k || (need_v && !c->v) || !c->h_req_token_offset) return RELAXKV_ERR_INVALID_ARG;
  if (!aligned16(c->k) || (need_v && !aligned16(c->v))) return RELAXKV_ERR_INVALID_ARG;
  if (c->token_stride < s->head_dim || c->head_stride < s->head_dim) return RELAXKV_ERR_INVALID_ARG;
  if ((c->token_stride % 8) || (c->head_stride % 8)) return RELAXKV_ERR_INVALID_ARG;
  for (int b = 0; b < s->n_req; ++b)
    if (c->h_req_token_offset[b] < 0) return RELAXKV_ERR_INVALID_ARG;
  return RELAXKV_OK;
}

inline relaxkv_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? RELAXKV_OK : RELAXKV_ERR_CUDA; }
inline relaxkv_status launch_ok() { return cuda_ok(cudaGetLastError()); }

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- chained launches (programmatic dependent launch) ------------------------------------
// The short kernels of a decode step or of the query's pass (norms, one-row projections, appends, the one-token
// attention and its merge) follow one another on a stream, each a few microseconds long, and between two of them the
// device drains, launches and ramps up again.  Launched with the programmatic-serialization attribute, the next
// kernel's blocks become resident as soon as every block of the current one has called griddep_launch(); they may do
// whatever does not depend on earlier kernels (set-up, prefetching their weights) and then block in griddep_wait()
// until the earlier kernels have completed and their writes are visible.  Rules kept by every kernel that is launched
// this way: nothing written by another kernel is read, and nothing at all is written, before griddep_wait(); every
// block executes griddep_wait() (so a kernel never completes before its predecessors).  Both instructions do nothing
// in a kernel that was launched the plain way.  Only launches of a few rows are chained (`few_rows`: at most
// kChainedMaxRows): the same kernels at the query's 64-128 rows sit between large tensor-core launches that are
// launched the plain way, where the attribute measured 0.3 us per launch slower, not faster.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

bool chained_launch_enabled();           // process-wide switch (relaxkv_set_chained_launch), on by default
constexpr long long kChainedMaxRows = 8;

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(bool few_rows, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                  Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = (few_rows && chained_launch_enabled()) ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Up to this many requests have their per-request scalars passed by value in kernel parameters.
constexpr int kMaxReqInline = 64;

// Per-request scalars a kernel needs, by value (small batches) - avoids any host->device copy.
struct ReqTable {
  int n_req;
  int ctx_len[kMaxReqInline];
  int q_len[kMaxReqInline];
  int q_cu[kMaxReqInline + 1];      // prefix of q_len
  long long ctx_cu[kMaxReqInline + 1];  // prefix of ctx_len
  long long tok_off[kMaxReqInline];     // cache token offset
  int k[kMaxReqInline];
  int k_cu[kMaxReqInline + 1];
  int bound_a[kMaxReqInline];       // call-specific host bound (e.g. max targets)
  int bound_b[kMaxReqInline];       // call-specific host bound (e.g. max ctx)
  int tile_cu[kMaxReqInline + 1];   // call-specific prefix (e.g. q tiles)
};

// Fills the shape-derived fields of a ReqTable (host).
inline void fill_req_table(ReqTable& t, const relaxkv_shape* s, const relaxkv_cache_view* c, const int32_t* h_k) {
  t.n_req = s->n_req;
  t.q_cu[0] = 0; t.ctx_cu[0] = 0; t.k_cu[0] = 0; t.tile_cu[0] = 0;
  for (int b = 0; b < s->n_req; ++b) {
    t.ctx_len[b] = s->h_ctx_len[b];
    t.q_len[b] = s->h_q_len ? s->h_q_len[b] : 0;
    t.q_cu[b + 1] = t.q_cu[b] + t.q_len[b];
    t.ctx_cu[b + 1] = t.ctx_cu[b] + t.ctx_len[b];
    t.tok_off[b] = c ? c->h_req_token_offset[b] : 0;
    t.k[b] = h_k ? h_k[b] : 0;
    t.k_cu[b + 1] = t.k_cu[b] + t.k[b];
    t.bound_a[b] = 0; t.bound_b[b] = 0; t.tile_cu[b + 1] = 0;
  }
}

// ---- workspace layout -------------------------------------------------------------------
// Calls are stream-ordered, so the regions of different calls overlap.
constexpr int kScoreSplitsMax = 64;   // key-range splits of the scoring passes (grid.z), at most
constexpr int kScoreMaxRows = 640;    // query rows (token x head-in-group) resident per scoring CTA
constexpr int kScoreTokBox = 8;       // query tokens per TMA box of the scoring kernel
constexpr int kCtxPadRows = 128;      // zero rows after the materialised context
constexpr int kSplitRowsCap = 2048;   // (target rows) x (context splits) the split workspace holds
constexpr int kMaxCtxSplits = 32;

constexpr int kScoreLayersPerLaunch = 48;   // layers scored by one launch (their tensor maps travel as parameters)

// Key-range splits for a launch that scores `layers` layers at once: at least two waves of CTAs on the 148
// SMs (one CTA per SM), and a count that fills its last wave (every CTA of a launch does the same work).
inline int score_splits(long long units_times_heads, int layers) {
  const long long per = units_times_heads * layers;
  if (per <= 0) return 1;
  int best = 1;
  double best_eff = 0.0;
  for (int ns = 1; ns <= kScoreSplitsMax; ++ns) {
    const long long ctas = per * ns;
    if (ctas < 2 * 148 && ns < kScoreSplitsMax) continue;
    const long long waves = (ctas + 147) / 148;
    const double eff = (double)ctas / (double)(waves * 148);
    if (eff > best_eff + 0.02) { best_eff = eff; best = ns; }      // prefer fewer, longer CTAs unless clearly better
    if (ctas >= 16 * 148) break;
  }
  return best;
}

// Query-row blocks a request needs so that each block's rows fit resident (scoring kernel).
inline int score_blocks(int q_len, int group) {
  const int max_tok = kScoreMaxRows / group / kScoreTokBox * kScoreTokBox;
  return q_len > 0 ? (q_len + max_tok - 1) / max_tok : 0;
}

struct WsLayout {
  // attention: materialised mixed context K~ / V~  [ctx_rows_cap, H_kv, D] bf16
  size_t kctx, vctx; long long ctx_rows_cap;
  // explicit-list attention: limit [sumT] i32 | fresh_row [sumT] i32
  size_t list_limit, list_fresh;
  // context split across blocks (few targets): partial O [kSplitRowsCap, H, D] f32 | partial lse [kSplitRowsCap, H] f32
  size_t split_o, split_lse;
  // scoring (per launch of Lc <= kScoreLayersPerLaunch layers): lse [Lc, H, sumQ] f32 |
  // part [Lc, 2*n_splits, H, sumQ] float2 | colpart [Lc, 2*H_kv*max_blocks, sumT] f32
  size_t lse, part, colpart;
  // sets: counts [B + L*B] i32
  size_t counts;
  size_t total;
};

inline WsLayout ws_layout(const relaxkv_shape* s, int n_layers) {
  WsLayout w{};
  long long sum_t = 0, sum_q = 0;
  for (int b = 0; b < s->n_req; ++b) { sum_t += s->h_ctx_len[b]; sum_q += s->h_q_len ? s->h_q_len[b] : 0; }
  const size_t row_bytes = (size_t)s->n_kv_heads * s->head_dim * 2;
  w.ctx_rows_cap = sum_t + kCtxPadRows;
  size_t a = 0;
  w.kctx = a; a = align_up(a + (size_t)w.ctx_rows_cap * row_bytes, 1024);
  w.vctx = a; a = align_up(a + (size_t)w.ctx_rows_cap * row_bytes, 1024);
  w.list_limit = a; a = align_up(a + (size_t)sum_t * 4, 256);
  w.list_fresh = a; a = align_up(a + (size_t)sum_t * 4, 256);
  w.split_o = a; a = align_up(a + (size_t)kSplitRowsCap * s->n_q_heads * s->head_dim * 4, 256);
  w.split_lse = a; a = align_up(a + (size_t)kSplitRowsCap * s->n_q_heads * 4, 256);
  size_t attn_total = a;
  a = 0;
  const int lc_max = n_layers < kScoreLayersPerLaunch ? n_layers : kScoreLayersPerLaunch;
  w.lse = a; a = align_up(a + (size_t)lc_max * s->n_q_heads * sum_q * 4, 256);
  int max_blocks = 1;
  for (int b = 0; b < s->n_req; ++b) {
    const int nb = score_blocks(s->h_q_len ? s->h_q_len[b] : 0, s->n_q_heads / s->n_kv_heads);
    if (nb > max_blocks) max_blocks = nb;
  }
  long long units = 0;
  for (int b = 0; b < s->n_req; ++b) units += score_blocks(s->h_q_len ? s->h_q_len[b] : 0, s->n_q_heads / s->n_kv_heads);
  long long part_slots = 1;                 // max over launch sizes of layers x 2 x splits
  for (int lc = 1; lc <= lc_max; ++lc) {
    const long long v = (long long)lc * 2 * score_splits(units * s->n_kv_heads, lc);
    if (v > part_slots) part_slots = v;
  }
  w.part = a; a = align_up(a + (size_t)part_slots * s->n_q_heads * sum_q * 8, 256);
  w.colpart = a; a = align_up(a + (size_t)lc_max * 2 * s->n_kv_heads * max_blocks * sum_t * 4, 256);
  size_t score_total = a;
  w.counts = 0;
  size_t sets_total = align_up((size_t)(s->n_req + (size_t)n_layers * s->n_req + 2) * 4, 256);
  w.total = attn_total > score_total ? attn_total : score_total;
  if (sets_total > w.total) w.total = sets_total;
  return w;
}

// ---- small device helpers -----------------------------------------------------------------
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }

__device__ __forceinline__ int warp_reduce_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_reduce_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_reduce_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_reduce_min(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Find the request that owns global tile/row index x given an inclusive-exclusive prefix array.
__device__ __forceinline__ int find_segment(const int* cu, int n, int x) {
  int b = 0;
  while (b + 1 < n && x >= cu[b + 1]) ++b;
  return b;
}

}  // namespace relaxkv
