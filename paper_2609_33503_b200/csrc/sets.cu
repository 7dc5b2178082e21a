// Repair schedule: highest selected layer h_i, sorted union U, position->rank map and the per-layer
// active targets R_l as ranks into U (Section 3.2; Algorithm 1, steps 6-12).  Integer work only.
#include "common.cuh"

namespace relaxkv {

constexpr int kSetThreads = 1024;

__global__ void fill_i32_kernel(int* p, long long n, int v) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

// h[i] = max layer that selected position i.
__global__ void highest_layer_kernel(ReqTable rt, int n_layers, const int* __restrict__ anchors,
                                     int* __restrict__ h, DeviceStatus* st) {
  const int sum_k = rt.k_cu[rt.n_req];
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n_layers * sum_k) return;
  const int l = (int)(idx / sum_k);
  const int j = (int)(idx - (long long)l * sum_k);
  const int b = find_segment(rt.k_cu, rt.n_req, j);
  const int pos = anchors[idx];
  if (pos < 0 || pos >= rt.ctx_len[b]) { report(st, RELAXKV_ERR_BAD_INDEX, KID_SETS, (int)idx, pos); return; }
  atomicMax(&h[rt.ctx_cu[b] + pos], l);
}

// Exclusive block scan of two counters (blockDim.x == kSetThreads); returns the totals too.
__device__ __forceinline__ void block_scan2(int a, int b, int& a_excl, int& b_excl, int& a_tot, int& b_tot) {
  __shared__ int wa[32], wb[32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int ia = a, ib = b;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int ta = __shfl_up_sync(0xffffffffu, ia, o), tb = __shfl_up_sync(0xffffffffu, ib, o);
    if (lane >= o) { ia += ta; ib += tb; }
  }
  if (lane == 31) { wa[warp] = ia; wb[warp] = ib; }
  __syncthreads();
  if (warp == 0) {
    int va = wa[lane], vb = wb[lane];
    int sa = va, sb = vb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int ta = __shfl_up_sync(0xffffffffu, sa, o), tb = __shfl_up_sync(0xffffffffu, sb, o);
      if (lane >= o) { sa += ta; sb += tb; }
    }
    wa[lane] = sa - va; wb[lane] = sb - vb;          // exclusive warp offsets
    if (lane == 31) { wa[31] = sa - va; wb[31] = sb - vb; }
  }
  __syncthreads();
  a_excl = wa[warp] + ia - a;
  b_excl = wb[warp] + ib - b;
  __syncthreads();
  // totals: last thread's inclusive value
  __shared__ int ta_s, tb_s;
  if (threadIdx.x == kSetThreads - 1) { ta_s = a_excl + a; tb_s = b_excl + b; }
  __syncthreads();
  a_tot = ta_s; b_tot = tb_s;
  __syncthreads();
}

// Block (b, s): s == 0 counts |U_b|; s = l+1 counts |R_{l,b}|.  counts[b] and counts[B + l*B + b].
__global__ void __launch_bounds__(kSetThreads)
count_sets_kernel(ReqTable rt, int n_layers, const int* __restrict__ h, int* __restrict__ counts) {
  const int B = rt.n_req;
  const int b = blockIdx.x % B, s = blockIdx.x / B;
  const int T = rt.ctx_len[b];
  const int* hb = h + rt.ctx_cu[b];
  const int thr = (s == 0) ? 0 : (s - 1);
  int n = 0;
  for (int i = threadIdx.x; i < T; i += kSetThreads) n += (hb[i] >= thr) ? 1 : 0;
  __shared__ int red[32];
  n = warp_reduce_sum(n);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = n;
  __syncthreads();
  if (threadIdx.x < 32) {
    int v = red[threadIdx.x];
    v = warp_reduce_sum(v);
    if (threadIdx.x == 0) counts[s == 0 ? b : B + (s - 1) * B + b] = v;
  }
}

// u_cu[B+1] and r_cu[L*B+1] from the counts (one block; the arrays are short).
__global__ void prefix_counts_kernel(int B, int n_layers, const int* __restrict__ counts,
                                     int* __restrict__ u_cu, int* __restrict__ r_cu) {
  if (threadIdx.x == 0) {
    int a = 0;
    for (int b = 0; b < B; ++b) { u_cu[b] = a; a += counts[b]; }
    u_cu[B] = a;
  }
  if (threadIdx.x == 32) {
    int a = 0;
    const int n = n_layers * B;
    for (int i = 0; i < n; ++i) { r_cu[i] = a; a += counts[B + i]; }
    r_cu[n] = a;
  }
}

// Block (b, 0) writes u_pos / u_rank; block (b, l+1) writes the ranks of R_{l,b}.
__global__ void __launch_bounds__(kSetThreads)
write_sets_kernel(ReqTable rt, int n_layers, const int* __restrict__ h, const int* __restrict__ u_cu,
                  const int* __restrict__ r_cu, int* __restrict__ u_pos, int* __restrict__ u_rank,
                  int* __restrict__ r_rank) {
  const int B = rt.n_req;
  const int b = blockIdx.x % B, s = blockIdx.x / B;
  const int T = rt.ctx_len[b];
  const int* hb = h + rt.ctx_cu[b];
  const int thr = (s == 0) ? 0 : (s - 1);
  const int per = (T + kSetThreads - 1) / kSetThreads;
  const int i0 = min(T, (int)threadIdx.x * per), i1 = min(T, i0 + per);
  int nu = 0, nr = 0;
  for (int i = i0; i < i1; ++i) { const int v = hb[i]; nu += (v >= 0); nr += (v >= thr); }
  int eu, er, tu, tr;
  block_scan2(nu, nr, eu, er, tu, tr);
  if (s == 0) {
    int* up = u_pos + u_cu[b];
    int* ur = u_rank + rt.ctx_cu[b];
    for (int i = i0; i < i1; ++i) {
      if (hb[i] >= 0) { up[eu] = i; ur[i] = eu; ++eu; } else ur[i] = -1;
    }
  } else {
    int* rr = r_rank + r_cu[(s - 1) * B + b];
    for (int i = i0; i < i1; ++i) {
      const int v = hb[i];
      if (v >= thr) rr[er++] = eu;     // rank in U of this position = members of U before it
      if (v >= 0) ++eu;
    }
  }
}

}  // namespace relaxkv

using namespace relaxkv;

// The launch sequence both entry points share: `counts` (device int32 [B + n_layers*B]) is the only scratch.
static relaxkv_status build_sets(const relaxkv_shape* shape, int32_t n_layers, const int32_t* h_k, const int32_t* anchors,
                                 int32_t* highest_layer_out, int32_t* u_pos_out, int32_t* u_cu_out, int32_t* u_rank_out,
                                 int32_t* r_rank_out, int32_t* r_cu_out, int32_t* h_counts_pinned, int* counts,
                                 cudaStream_t stream) {
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  ReqTable rt;
  fill_req_table(rt, shape, nullptr, h_k);
  const int B = shape->n_req;
  const long long sum_t = rt.ctx_cu[B];
  // Nothing in `counts` has to start at zero: count_sets_kernel overwrites every entry that prefix_counts_kernel
  // and the copy below read.
  fill_i32_kernel<<<(unsigned)((sum_t + 255) / 256), 256, 0, stream>>>(highest_layer_out, sum_t, -1);
  const long long n_anchor = (long long)n_layers * rt.k_cu[B];
  highest_layer_kernel<<<(unsigned)((n_anchor + 255) / 256), 256, 0, stream>>>(rt, n_layers, anchors,
                                                                              highest_layer_out, st);
  const unsigned blocks = (unsigned)(B * (n_layers + 1));
  count_sets_kernel<<<blocks, kSetThreads, 0, stream>>>(rt, n_layers, highest_layer_out, counts);
  prefix_counts_kernel<<<1, 64, 0, stream>>>(B, n_layers, counts, u_cu_out, r_cu_out);
  write_sets_kernel<<<blocks, kSetThreads, 0, stream>>>(rt, n_layers, highest_layer_out, u_cu_out, r_cu_out,
                                                        u_pos_out, u_rank_out, r_rank_out);
  relaxkv_status rc = launch_ok();
  if (rc != RELAXKV_OK) return rc;
  if (h_counts_pinned)
    rc = cuda_ok(cudaMemcpyAsync(h_counts_pinned, counts, sizeof(int) * (size_t)(B + n_layers * B),
                                 cudaMemcpyDeviceToHost, stream));
  return rc;
}

static relaxkv_status check_sets_args(const relaxkv_shape* shape, int32_t n_layers, const int32_t* h_k,
                                      const int32_t* anchors, const int32_t* highest_layer_out, const int32_t* u_pos_out,
                                      const int32_t* u_cu_out, const int32_t* u_rank_out, const int32_t* r_rank_out,
                                      const int32_t* r_cu_out) {
  relaxkv_status rc = check_shape(shape);
  if (rc != RELAXKV_OK) return rc;
  if (n_layers < 1 || n_layers > 65535 || !h_k || !anchors || !highest_layer_out || !u_pos_out || !u_cu_out ||
      !u_rank_out || !r_rank_out || !r_cu_out)
    return RELAXKV_ERR_INVALID_ARG;
  for (int b = 0; b < shape->n_req; ++b)
    if (h_k[b] < 1 || h_k[b] > shape->h_ctx_len[b]) return RELAXKV_ERR_INVALID_ARG;
  return RELAXKV_OK;
}

extern "C" relaxkv_status relaxkv_build_active_sets(
    const relaxkv_shape* shape, int32_t n_layers, const int32_t* h_k, const int32_t* anchors,
    int32_t* highest_layer_out, int32_t* u_pos_out, int32_t* u_cu_out, int32_t* u_rank_out,
    int32_t* r_rank_out, int32_t* r_cu_out, int32_t* h_counts_pinned,
    void* workspace, size_t workspace_bytes, relaxkv_stream stream_) {
  RELAXKV_RANGE("relaxkv_build_active_sets");
  relaxkv_status rc = check_sets_args(shape, n_layers, h_k, anchors, highest_layer_out, u_pos_out, u_cu_out, u_rank_out,
                                      r_rank_out, r_cu_out);
  if (rc != RELAXKV_OK) return rc;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return RELAXKV_ERR_INVALID_ARG;
  const WsLayout ws = ws_layout(shape, n_layers);
  if (workspace_bytes < ws.total) return RELAXKV_ERR_WORKSPACE_TOO_SMALL;
  int* counts = reinterpret_cast<int*>(static_cast<char*>(workspace) + ws.counts);
  return build_sets(shape, n_layers, h_k, anchors, highest_layer_out, u_pos_out, u_cu_out, u_rank_out, r_rank_out, r_cu_out,
                    h_counts_pinned, counts, static_cast<cudaStream_t>(stream_));
}

// ---- variant whose scratch lives in the library image ------------------------------------------
// Some hosts of this library own every byte of device memory themselves and give an extension no
// way to ask for more: an inference-server plug-in that is handed its input and output tensors and
// nothing else, or an embedded runtime whose memory pool is sealed once start-up ends.  Such a
// caller cannot provide the `workspace` that relaxkv_build_active_sets needs.  For them the set
// counts are kept in this fixed array, which every GPU that loads the library holds until exit.
constexpr int kStaticCountsMax = 8192;           // ints: B + n_layers*B must fit
static __device__ __align__(256) int g_static_counts[kStaticCountsMax];

// Device address of g_static_counts on the current device.  In host code the array's name is only a
// handle; the address a kernel can use comes from cudaGetSymbolAddress, once per device, with that
// device current.
static relaxkv_status static_counts_ptr(int** out) {
  static std::atomic<int*> cached[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RELAXKV_ERR_CUDA;
  int* p = cached[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress((void**)&p, g_static_counts) != cudaSuccess || p == nullptr) return RELAXKV_ERR_CUDA;
    cached[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return RELAXKV_OK;
}

extern "C" relaxkv_status relaxkv_build_active_sets_static(
    const relaxkv_shape* shape, int32_t n_layers, const int32_t* h_k, const int32_t* anchors,
    int32_t* highest_layer_out, int32_t* u_pos_out, int32_t* u_cu_out, int32_t* u_rank_out,
    int32_t* r_rank_out, int32_t* r_cu_out, int32_t* h_counts_pinned, relaxkv_stream stream_) {
  RELAXKV_RANGE("relaxkv_build_active_sets_static");
  relaxkv_status rc = check_sets_args(shape, n_layers, h_k, anchors, highest_layer_out, u_pos_out, u_cu_out, u_rank_out,
                                      r_rank_out, r_cu_out);
  if (rc != RELAXKV_OK) return rc;
  const int B = shape->n_req;
  if ((long long)B + (long long)n_layers * B > kStaticCountsMax) return RELAXKV_ERR_UNSUPPORTED_SHAPE;
  int* counts = nullptr;
  if ((rc = static_counts_ptr(&counts)) != RELAXKV_OK) return rc;
  return build_sets(shape, n_layers, h_k, anchors, highest_layer_out, u_pos_out, u_cu_out, u_rank_out, r_rank_out, r_cu_out,
                    h_counts_pinned, counts, static_cast<cudaStream_t>(stream_));
}
