/*
 * relaxkv.h - C ABI of the RelaxKV selective cache-repair hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, as hand-written CUDA kernels, the two halves of the repair path of
 * "RelaxKV: Recomputation Guided by the Query with Sparse Context Attention":
 *   (a) query-guided anchor selection   - relaxkv_score_select, relaxkv_build_active_sets
 *   (b) sparse-context repair attention - relaxkv_sparse_ctx_attention, relaxkv_scatter_kv
 *
 * General conventions (they hold for every entry point unless it says otherwise)
 * -----------------------------------------------------------------------------
 * Pointers.   A name starting with h_ is a HOST pointer, read during the call only.  Every other
 *             pointer is a DEVICE pointer of the current CUDA device.  All buffers are owned by the
 *             caller; the library allocates nothing, frees nothing and keeps no pointer after the
 *             call returns.  Scratch comes from the caller's `workspace` (device memory, 256-byte
 *             aligned, at least relaxkv_workspace_bytes() bytes).
 * Types.      K, V, Q and attention outputs are bf16 (2 bytes); scores are fp32; every index is
 *             int32.  head_dim is contiguous in memory everywhere.  bf16 base pointers must be
 *             16-byte aligned and the cache strides multiples of 8 elements.
 * Batching.   A call covers n_req independent requests (a ragged batch).  Per-request arrays are
 *             packed back to back; "cu" arrays hold the n_req+1 exclusive prefix offsets.
 * Positions.  Context positions are request-local token indices 0..T_c-1.  Every index list is
 *             ascending and free of duplicates.  Active targets are stored as ranks into the
 *             sorted union U, so a target's causal limit is its own rank.
 * Heads.      Query head h reads KV head h / (n_q_heads / n_kv_heads).
 * Asynchrony. All work is enqueued on `stream`; no call synchronises except
 *             relaxkv_read_device_status.  Data-dependent set sizes stay on the device; the host
 *             passes upper bounds.
 * Errors.     Host-checkable violations (NULL, bad shape, misalignment, workspace too small) return
 *             a status before any launch.  Launch failures return RELAXKV_ERR_CUDA.  Problems only
 *             the device can see (an index out of range, a count above its host bound, a bounded
 *             wait that expired) are recorded in a device status word - the kernel skips the
 *             offending work and returns normally - and are read with relaxkv_read_device_status.
 *             The first problem recorded stays until it is read.  After an expired wait (RELAXKV_ERR_TIMEOUT)
 *             the tensor-core kernels of later calls on that device return at once without writing their
 *             outputs, until the status word has been read (and thereby cleared): a caller that sees garbage
 *             should read the status word first.
 * Graphs.     Every call only enqueues kernels, memsets and copies on `stream`, so calls can be recorded into a CUDA
 *             graph; make the first call of each kind on a device outside the capture (it looks up device
 *             addresses and opts kernels into large shared memory).  The host bounds and the choice of kernel form
 *             are frozen into the graph.
 * Threads.    Calls may be made from several host threads; the per-device values the library looks up once
 *             (device addresses, attribute opt-ins) are published with atomics.  The status word is per device,
 *             not per thread or stream.
 * Precision.  bf16 inputs, fp32 accumulation and softmax, probabilities rounded to bf16 before the
 *             P*V product, bf16 outputs.
 */
#ifndef RELAXKV_H_
#define RELAXKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RELAXKV_OK = 0,
  RELAXKV_ERR_INVALID_ARG = 1,
  RELAXKV_ERR_UNSUPPORTED_SHAPE = 2,
  RELAXKV_ERR_WORKSPACE_TOO_SMALL = 3,
  RELAXKV_ERR_CUDA = 4,
  RELAXKV_ERR_BAD_INDEX = 5,
  RELAXKV_ERR_TIMEOUT = 6
} relaxkv_status;

/* A CUDA stream handle (cudaStream_t) passed as an opaque pointer; NULL is the default stream. */
typedef void* relaxkv_stream;

/* Optional per-call overrides of choices the library otherwise makes from the size of the launch.  Every field:
 * 0 = automatic.  Meant for tests and measurements; results agree within the tolerances either way. */
typedef struct {
  int32_t attention_ctx_splits;  /* > 0: the attention calls split every query tile's context over this many thread   */
                                 /* blocks (up to 32, and as far as the workspace's 2048 row-splits allow) and merge   */
                                 /* the partial results by their log-sum-exp; automatic = only when the call has too   */
                                 /* few query tiles to fill the GPU (a query prefill, a decode step, few targets)      */
  int32_t attention_persistent;  /* the repair / list attention calls have a persistent form (one thread block per SM  */
                                 /* walks the call's query tiles, longest context first).  0: the library takes it     */
                                 /* for one-split calls over gathered contexts of at most 128 key tiles; 1: for every  */
                                 /* one-split call over a gathered context; 2: never.  Same results bit for bit.       */
  int32_t attention_grid_blocks; /* > 0: number of thread blocks of the persistent form (default: one per SM)          */
} relaxkv_tuning;

/* Shapes shared by all calls. */
typedef struct {
  int32_t n_req;              /* 1 <= B <= 64 requests in the batch                             */
  int32_t n_q_heads;          /* H                                                              */
  int32_t n_kv_heads;         /* H_kv, divides H; the group size G = H / H_kv must be <= 16     */
  int32_t head_dim;           /* D, 64 or 128                                                   */
  const int32_t* h_ctx_len;   /* host [B]: context tokens T_c of each request                   */
  const int32_t* h_q_len;     /* host [B]: query-suffix tokens Q of each request; read by       */
                              /* relaxkv_score_select and relaxkv_workspace_bytes only          */
  float softmax_scale;        /* multiplies q.k before the softmax (usually 1/sqrt(D))          */
  const relaxkv_tuning* h_tuning;  /* host, optional: NULL = every choice automatic             */
} relaxkv_shape;

/* One layer's KV cache.  Element (request b, token i, kv head g, dim d) of K lives at
 * k + (h_req_token_offset[b] + i) * token_stride + g * head_stride + d  (in elements), same for V.
 * This covers [tokens, H_kv, D] and [H_kv, tokens, D] storage. */
typedef struct {
  void* k;
  void* v;
  int64_t token_stride;
  int64_t head_stride;
  const int64_t* h_req_token_offset;   /* host [B]: first token row of each request */
} relaxkv_cache_view;

/* How the recomputation context of a target at position p is built. */
typedef enum {
  RELAXKV_CTX_UNION = 0,        /* C_l(p) = U intersect {j <= p}  (the method)                    */
  RELAXKV_CTX_FULL_PREFIX = 1   /* every position j <= p (the paper's Full-Prefix Control)        */
} relaxkv_ctx_mode;

const char* relaxkv_status_string(int32_t status);

/* Anchors per layer, k = max(1, round(r * T_c)) clamped to T_c; round is to nearest with halves to
 * even on the fp64 product.  (Appendix A.1, anchor-count equation; Section 3.2.)  Host only. */
int32_t relaxkv_anchor_count(int32_t ctx_len, double ratio);

/* Bytes of device scratch that suffice for any call below with these shapes.  h_k may be NULL.
 * Returns 0 for an invalid shape.  Host only. */
size_t relaxkv_workspace_bytes(const relaxkv_shape* shape, int32_t n_layers, const int32_t* h_k);

/*
 * Query-attention scoring and per-layer top-k anchors (Section 3.2, score equation and TopK;
 * Algorithm 1, steps 1-5; Appendix A.1).
 *
 * For each layer l < n_layers and request b, with Q = the request's query-suffix rows:
 *   s[h,t,i]  = softmax_scale * <q[t,h,:], K[i, h/G, :]>                i over all T_c cached tokens
 *   A[h,t,i]  = exp(s[h,t,i] - lse[h,t])     lse = log sum_i exp(s[h,t,i])  unless supplied
 *   raw[i]    = (1/(H*Q)) * sum_h sum_t A[h,t,i]
 *   norm[i]   = (raw[i] - min raw) / (max raw - min raw)                (all zeros if max == min)
 *   anchors   = positions of the k largest raw[i]; equal scores go to the lower position;
 *               written in ascending order.  (MinMax is monotone, so selecting on raw selects the
 *               same set as selecting on norm.)
 *
 * q_layers         host array [n_layers] of device bf16 [sum_b Q_b, H, D] (requests packed).
 * cache_layers     host array [n_layers]; only .k is read.
 * row_lse_layers   NULL, or host array [n_layers] of device fp32 [H, sum_b Q_b] (entry (h, row));
 *                  when given for a layer, its rows' log-normalisers are taken from it (e.g. from the
 *                  query's own forward pass, whose softmax also spans the query tokens) and the
 *                  statistics pass is skipped.  An entry may itself be NULL.
 * h_k              host [B]: anchors per layer for each request, 1 <= k_b <= T_c.
 * raw_scores_out   device fp32 [n_layers, sum_b T_c].
 * norm_scores_out  NULL or device fp32 [n_layers, sum_b T_c].
 * anchors_out      device int32 [n_layers, sum_b k_b]; request-local positions.  NULL: scoring only (no
 *                  selection, norm_scores_out is not written) - for callers that first combine the scores
 *                  of several head shards (mean over shards of equal size) and then call relaxkv_select_topk.
 * Results are deterministic: reductions run in a fixed order (no floating-point atomics).
 */
relaxkv_status relaxkv_score_select(
    const relaxkv_shape* shape, int32_t n_layers,
    const void* const* q_layers, const relaxkv_cache_view* cache_layers,
    const float* const* row_lse_layers, const int32_t* h_k,
    float* raw_scores_out, float* norm_scores_out, int32_t* anchors_out,
    void* workspace, size_t workspace_bytes, relaxkv_stream stream);

/*
 * The selection step of relaxkv_score_select on its own (Appendix A.1, TopK; Section 3.2, MinMax):
 * top-k anchors (and optionally the MinMax-normalised scores) of given raw scores.  Same layouts,
 * tie rule and output order as above.  Exists so the step can be checked and timed by itself.
 */
relaxkv_status relaxkv_select_topk(
    const relaxkv_shape* shape, int32_t n_layers, const int32_t* h_k, const float* raw_scores,
    float* norm_scores_out, int32_t* anchors_out, relaxkv_stream stream);

/*
 * Repair schedule from the per-layer anchors (Section 3.2, definitions of h_i, U, R_l;
 * Algorithm 1, steps 6-12; Appendix A.2: U is kept sorted and its members are numbered once per request).
 *
 *   h_i  = max{ l : i in S_l }  (-1 if i is in no S_l);   U = { i : h_i >= 0 } ascending;
 *   u_rank[i] = index of i in U (or -1);   R_l = { c : h_{U[c]} >= l } as ascending ranks c.
 *
 * anchors            device int32 [n_layers, sum_b k_b] as written by relaxkv_score_select.
 * highest_layer_out  device int32 [sum_b T_c].
 * u_pos_out          device int32, capacity sum_b min(T_c, n_layers*k_b): U of each request, packed.
 * u_cu_out           device int32 [B+1].
 * u_rank_out         device int32 [sum_b T_c].
 * r_rank_out         device int32, capacity n_layers * (capacity of u_pos_out): for layer l and
 *                    request b the ranks of R_{l,b}, packed in (l, b) order.
 * r_cu_out           device int32 [n_layers*B + 1]: offset of segment (l, b) at index l*B + b.
 * h_counts_pinned    NULL or pinned host int32 [B + n_layers*B]: |U_b| then |R_{l,b}|; valid once
 *                    the stream has been synchronised.
 */
relaxkv_status relaxkv_build_active_sets(
    const relaxkv_shape* shape, int32_t n_layers, const int32_t* h_k, const int32_t* anchors,
    int32_t* highest_layer_out, int32_t* u_pos_out, int32_t* u_cu_out, int32_t* u_rank_out,
    int32_t* r_rank_out, int32_t* r_cu_out, int32_t* h_counts_pinned,
    void* workspace, size_t workspace_bytes, relaxkv_stream stream);

/*
 * relaxkv_build_active_sets for callers that have no scratch memory to give.  (The paper has no
 * counterpart; this is a packaging variant of the call above and computes the same outputs.)
 *
 * Who needs it: code that runs inside a host which owns all device memory and lends an extension
 * only its input and output tensors - an inference-server plug-in, an embedded runtime whose
 * memory pool is sealed after start-up.  Such a caller can neither allocate a workspace nor ask
 * its host for one.  Here the scratch (the B + n_layers*B set counts) lives in a fixed array inside
 * the library image; the call allocates nothing and takes no workspace.  Inputs and outputs are
 * still the caller's buffers, exactly as above.
 *
 * Limits and rules:
 *  - B + n_layers*B must not exceed 8192 entries (32 KB, held by every GPU that loads the
 *    library until the process exits); larger problems get RELAXKV_ERR_UNSUPPORTED_SHAPE.
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *    that device current).  Make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps the previous call's contents.  Nothing
 *    in it needs to start at zero (each call overwrites every entry it later reads), but two calls
 *    that overlap on the GPU - different streams, no ordering between them - race on it: order them.
 *  - h_counts_pinned (optional) is filled from the array by a copy on `stream`, as above.
 */
relaxkv_status relaxkv_build_active_sets_static(
    const relaxkv_shape* shape, int32_t n_layers, const int32_t* h_k, const int32_t* anchors,
    int32_t* highest_layer_out, int32_t* u_pos_out, int32_t* u_cu_out, int32_t* u_rank_out,
    int32_t* r_rank_out, int32_t* r_cu_out, int32_t* h_counts_pinned, relaxkv_stream stream);

/*
 * Sparse-context repair attention of one layer (Section 3.3, C_l(p); Section 3.4, mixed
 * fresh/cached K/V; Algorithm 1, steps 16-19; Appendix A.2).
 *
 * Target row rho of request b has rank c* = r_rank[r_cu_layer[b] + rho] in U_b and position
 * p = u_pos[u_cu[b] + c*].  With the context list X = U_b (RELAXKV_CTX_UNION; limit = c*) or
 * X = (0..T_c-1) (RELAXKV_CTX_FULL_PREFIX; limit = p), and
 *   Kt[x] = k_new[row of x] if X[x] is an active target of this layer, else cache K at X[x]
 * (same for V), the call computes for every query head h
 *   out[rho,h,:] = sum_{x <= limit} softmax_x(softmax_scale * <q_new[rho,h,:], Kt[x, h/G, :]>) * Vt[x, h/G, :]
 * The target itself is part of its context.  The cache is not modified.
 *
 * q_new           device bf16 [n_target_rows, H, D]; the rows of request b start at
 *                 r_cu_layer[b] - r_cu_layer[0] and follow the order of its R list.
 * k_new, v_new    device bf16 [n_target_rows, H_kv, D], or both NULL to read the cache only.
 * u_pos, u_cu     as written by relaxkv_build_active_sets.
 * r_rank          base of the packed rank array written by relaxkv_build_active_sets.
 * r_cu_layer      r_cu_out + l*B for this layer (B+1 offsets into r_rank are read).
 * n_target_rows   rows allocated in q_new/k_new/v_new/out (>= the layer's true total).
 * h_max_targets   host [B]: upper bound of |R_{l,b}|.   h_max_ctx: host [B]: upper bound of |U_b|.
 *                 A true count above its bound is reported through the device status word.
 * out             device bf16 [n_target_rows, H, D].
 * lse_out         NULL or device fp32 [H, n_target_rows]: log-normaliser of each output row.
 */
relaxkv_status relaxkv_sparse_ctx_attention(
    const relaxkv_shape* shape, relaxkv_ctx_mode mode, const relaxkv_cache_view* cache,
    const void* q_new, const void* k_new, const void* v_new,
    const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank, const int32_t* r_cu_layer,
    int64_t n_target_rows, const int32_t* h_max_targets, const int32_t* h_max_ctx,
    void* out, float* lse_out,
    void* workspace, size_t workspace_bytes, relaxkv_stream stream);

/*
 * Cache update of one layer (Section 3.4; Algorithm 1, step 21): the fresh K/V of every active
 * target overwrite its cache entry; no other byte of the cache changes.  Idempotent.
 * Arguments as for relaxkv_sparse_ctx_attention; `cache` is written in place.
 */
relaxkv_status relaxkv_scatter_kv(
    const relaxkv_shape* shape, const relaxkv_cache_view* cache,
    const void* k_new, const void* v_new,
    const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank, const int32_t* r_cu_layer,
    const int32_t* h_max_targets, relaxkv_stream stream);

/*
 * Materialised mixed context of one layer (Section 3.4 equation; Algorithm 1, steps 17-18):
 * k_ctx_out / v_ctx_out, device bf16 [ctx_rows, H_kv, D], receive for request b, at rows
 * x_cu[b] .. , Kt/Vt of the context list X defined above, where x_cu = u_cu (UNION) or the prefix
 * sums of T_c (FULL_PREFIX).  The 128 rows after the last one are zero-filled (as far as ctx_rows
 * allows).  ctx_rows >= sum_b h_max_ctx[b] (UNION) or sum_b T_c (FULL_PREFIX).
 * relaxkv_sparse_ctx_attention runs this step itself into its workspace; the entry point exists
 * so the step can be checked and timed on its own.
 */
relaxkv_status relaxkv_gather_kv(
    const relaxkv_shape* shape, relaxkv_ctx_mode mode, const relaxkv_cache_view* cache,
    const void* k_new, const void* v_new,
    const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank, const int32_t* r_cu_layer,
    const int32_t* h_max_ctx, void* k_ctx_out, void* v_ctx_out, int64_t ctx_rows,
    relaxkv_stream stream);

/*
 * Repair attention for explicit target and context lists - the paper's controlled configurations
 * (Appendix A.3, table of configurations; Section 4.4 ablation; Appendix B): global repair targets P
 * with context C(p) = U intersect {j <= p} (RelaxKV^G, global target sweep), Global Sparse and Layerwise
 * Sparse context sets U_l with the method's targets R_l.  For request b the targets are the positions
 * tgt_pos[tgt_cu[b] .. tgt_cu[b+1]) and the context list is ctx_pos[ctx_cu[b] .. ctx_cu[b+1]), both
 * ascending; tgt_cu[0] must be 0.  Target rho at position p attends to the context entries with
 * position <= p; an entry whose position is itself a target contributes that target's fresh K/V, every
 * other entry the cached K/V (Section 3.4 equation with R_l := the target list).  A target need not be a
 * context entry (then it does not see itself); a target with no visible entry gets a zero output row and
 * lse = -inf (the paper does not define that case).  With ctx = U, tgt = R_l this equals
 * relaxkv_sparse_ctx_attention; with ctx = all positions, its full-prefix mode.
 * q_new/k_new/v_new/out rows follow the packed target order; other arguments as above.
 */
relaxkv_status relaxkv_list_attention(
    const relaxkv_shape* shape, const relaxkv_cache_view* cache,
    const void* q_new, const void* k_new, const void* v_new,
    const int32_t* ctx_pos, const int32_t* ctx_cu, const int32_t* tgt_pos, const int32_t* tgt_cu,
    int64_t n_target_rows, const int32_t* h_max_targets, const int32_t* h_max_ctx,
    void* out, float* lse_out, void* workspace, size_t workspace_bytes, relaxkv_stream stream);

/* Cache update for an explicit target list (Section 3.4): cache entries at tgt_pos receive k_new / v_new. */
relaxkv_status relaxkv_scatter_kv_lists(
    const relaxkv_shape* shape, const relaxkv_cache_view* cache, const void* k_new, const void* v_new,
    const int32_t* tgt_pos, const int32_t* tgt_cu, const int32_t* h_max_targets, relaxkv_stream stream);

/* Across-layer mean score g_i = (1/L) sum_l a_{l,i} (Appendix B; also the Global Sparse context source):
 * scores device fp32 [n_layers, sum_b T_c] -> mean_out device fp32 [sum_b T_c], summed in layer order.
 * Feed mean_out to relaxkv_select_topk (n_layers = 1) for the global target set or the shared context set. */
relaxkv_status relaxkv_mean_scores(const relaxkv_shape* shape, int32_t n_layers, const float* scores,
                                   float* mean_out, relaxkv_stream stream);

/*
 * The user query's own attention at one layer with the context scores taken from the same pass (Section 2,
 * the query's pass over the naive cache is what yields its attention to the context, layer by layer; Section 3.2, score
 * equation with the row normalisers of the query's real forward pass, whose softmax also spans the query's own
 * tokens).  For a serving caller this replaces relaxkv_score_select's scoring for the layer: the statistics pass
 * never runs, the scores come out of the forward pass the query makes anyway.
 *
 * For request b the cache holds the T_c = h_ctx_len[b] context rows followed by the Q_b = h_q_len[b] rows of the
 * query's own K/V (positions T_c .. T_c + Q_b - 1); it must hold h_req_token_offset[b] + T_c + Q_b token rows.
 *   out[t,h,:] = causal attention of query token t (position T_c + t) over positions 0 .. T_c + t of its request
 *   lse[h,t]   = log-normaliser of that row (context keys and the query's own keys up to t)
 *   raw[i]     = (1/(H*Q_b)) * sum_h sum_t exp(softmax_scale * <q[t,h,:], K[i,h/G,:]> - lse[h,t])      for i < T_c
 * q / out         device bf16 [sum_b Q_b, H, D]; lse_out device fp32 [H, sum_b Q_b] (required)
 * raw_scores_out  device fp32 [sum_b T_c], or NULL for the attention alone.  Stack the layers' rows and feed them to
 *                 relaxkv_select_topk for the anchors.
 * workspace       at least relaxkv_workspace_bytes() of the same shape with h_ctx_len[b] = T_c + Q_b.
 * Runs the cache-only attention kernel (which leaves the rows' normalisers), then the column-sum pass of the scoring
 * kernel over the context keys with those normalisers.
 */
relaxkv_status relaxkv_query_prefill_attention(
    const relaxkv_shape* shape, const relaxkv_cache_view* cache, const void* q, void* out, float* lse_out,
    float* raw_scores_out, void* workspace, size_t workspace_bytes, relaxkv_stream stream);

/* scores[l, i] *= factor, in place, for device fp32 [n_layers, sum_b T_c] (factor > 0).  Section 3.2's score is a mean
 * over all H query heads; when the heads are sharded over N devices of equal share, every device scores its own heads
 * (relaxkv_score_select with anchors_out = NULL), the devices' scores are summed by one all-reduce and this call with
 * factor = 1/N turns the sum of the shard means into the mean over all heads; relaxkv_select_topk follows. */
relaxkv_status relaxkv_scale_scores(const relaxkv_shape* shape, int32_t n_layers, float* scores, float factor,
                                    relaxkv_stream stream);

/*
 * ---- Dense block work of the active targets (Algorithm 1, steps 14, 16 and 20; Section 3.3 for the
 * position IDs).  The method leaves the Transformer block as it is and runs it on the |R_l| active rows only; these
 * calls are that block for a Llama-style pre-norm decoder.  All tensors bf16, row-major, 16-byte aligned,
 * feature counts multiples of 8; fp32 arithmetic inside.  The caller owns every buffer. ----
 */

/* y[r, :] = x[r, :] * rsqrt(mean(x[r, :]^2) + eps) * weight[:]      x, y [n_rows, n_cols], weight [n_cols] */
relaxkv_status relaxkv_rmsnorm(const void* x, const void* weight, void* y, int64_t n_rows, int32_t n_cols,
                               float eps, relaxkv_stream stream);

/* y = x weight^T (+ residual)      x [n_rows, n_in], weight [n_out, n_in] (the [out, in] layout),
 * residual NULL or [n_rows, n_out], y [n_rows, n_out] (may alias residual).  tcgen05 GEMM: 256-row tiles on SM pairs
 * for many rows; for 5 to 128 rows (the query's own tokens) 128 x 128 tiles whose K range is split over a
 * thread-block cluster and summed through distributed shared memory in a fixed order, so that all SMs stream
 * weights; calls of one to four rows (a decode token, the row that goes through the output head) stream the
 * weights once through a plain HBM-bound kernel instead. */
relaxkv_status relaxkv_linear(const void* x, const void* weight, const void* residual, void* y,
                              int64_t n_rows, int32_t n_out, int32_t n_in, relaxkv_stream stream);

/* The attention block's three input projections in one call: q = x Wq^T, k = x Wk^T, v = x Wv^T with
 * w_qkv [n_q + 2 n_kv, n_in] = the rows of Wq, then Wk, then Wv (stacked once when the weights are loaded).
 * x [n_rows, n_in]; q [n_rows, n_q], k and v [n_rows, n_kv]: three separate row-major buffers.  Same arithmetic per
 * output element as relaxkv_linear.  Up to 128 rows (a decode token, the query's own tokens) this is ONE kernel that
 * streams the stacked matrix once; for more rows it is one large GEMM whose epilogue writes the three buffers when
 * n_q and n_kv are multiples of 32, else the three projections one after the other.
 * n_q, n_kv, n_in multiples of 8. */
relaxkv_status relaxkv_linear_qkv(const void* x, const void* w_qkv, void* q, void* k, void* v, int64_t n_rows,
                                  int32_t n_q, int32_t n_kv, int32_t n_in, relaxkv_stream stream);

/* out = silu(x Wg^T) * (x Wu^T) in one kernel (the MLP's first half): the gate and up projections and the
 * activation, with one rounding to bf16.  weight_tiled [2 * n_inter, n_in] holds, for every block t of 128
 * intermediate features, the 128 gate rows Wg[128 t .. 128 t + 127] followed by the 128 up rows Wu[same range]
 * (a fixed re-ordering of the rows of [Wg; Wu], done once when the weights are loaded), so that a 128 x 256
 * output tile of the GEMM carries both halves of the same features.  n_inter a multiple of 128.
 * x [n_rows, n_in], out [n_rows, n_inter]. */
relaxkv_status relaxkv_linear_swiglu(const void* x, const void* weight_tiled, void* out, int64_t n_rows,
                                     int32_t n_inter, int32_t n_in, relaxkv_stream stream);

/* Rotary embedding in place, rotate-half convention: pair i < D/2 of each head vector is rotated by
 * positions[row] * theta^(-2i/D).  x [n_rows, n_heads, head_dim]; positions: device int32 [n_rows], the rows'
 * ORIGINAL global positions (Section 3.3: restricting the context does not renumber tokens).  Rotations
 * compose, so the same call re-aligns the cached keys of a chunk that is placed at another offset than the
 * one it was encoded at (Section 2, positional consistency): pass the offset difference (it may be negative)
 * as every token's position. */
relaxkv_status relaxkv_rope(void* x, int64_t n_rows, int32_t n_heads, int32_t head_dim, const int32_t* positions,
                            float theta, relaxkv_stream stream);

/* The per-head RMSNorm of the projected queries and keys (models that have one; pass NULL weights otherwise) followed by
 * the rotary embedding, on q [n_rows, n_q_heads, head_dim] and k [n_rows, n_kv_heads, head_dim] in place, in ONE
 * launch: the same results as relaxkv_rmsnorm on the head vectors of q and of k followed by relaxkv_rope on q and on
 * k (the normalised values are rounded to bf16 in between, as a store would), meant for the few rows of a query pass
 * or a decode step, where four launches cost more than their work.  w_q_norm, w_k_norm: [head_dim] or both NULL. */
relaxkv_status relaxkv_qk_norm_rope(void* q, void* k, int64_t n_rows, int32_t n_q_heads, int32_t n_kv_heads,
                                    int32_t head_dim, const void* w_q_norm, const void* w_k_norm, float eps,
                                    const int32_t* positions, float theta, relaxkv_stream stream);

/* out[r, i] = silu(gate_up[r, i]) * gate_up[r, n_inter + i]      gate_up [n_rows, 2*n_inter], out [n_rows, n_inter] */
relaxkv_status relaxkv_swiglu(const void* gate_up, void* out, int64_t n_rows, int32_t n_inter, relaxkv_stream stream);

/* positions_out[row] = position of target row of this layer (row order = the layer's R lists, requests
 * packed): u_pos[u_cu[b] + r_rank[r_cu_layer[b] + rho]].  Feeds relaxkv_rope. */
relaxkv_status relaxkv_target_positions(const relaxkv_shape* shape, const int32_t* u_pos, const int32_t* u_cu,
                                        const int32_t* r_rank, const int32_t* r_cu_layer,
                                        const int32_t* h_max_targets, int32_t* positions_out, relaxkv_stream stream);

/* Hidden-state carry between layers (Section 3.2: a token stays active through its highest selected layer):
 * h_out gets, in the row order of layer l+1's targets, the rows of h_in (row order of layer l's targets)
 * that stay active.  r_cu_layer = r_cu + l*B, r_cu_next = r_cu + (l+1)*B; h_max_next: host bounds on
 * |R_{l+1,b}|.  h_in, h_out [rows, n_cols], distinct buffers. */
relaxkv_status relaxkv_carry_rows(const relaxkv_shape* shape, const void* h_in, void* h_out, int32_t n_cols,
                                  const int32_t* r_rank, const int32_t* r_cu_layer, const int32_t* r_cu_next,
                                  const int32_t* h_max_next, relaxkv_stream stream);

/*
 * Test utility: the same result as relaxkv_sparse_ctx_attention from a plain SIMT kernel (one warp
 * per output row, fp32 throughout, no tensor cores).  A second opinion for debugging; far slower.
 */
relaxkv_status relaxkv_sparse_ctx_attention_simt(
    const relaxkv_shape* shape, relaxkv_ctx_mode mode, const relaxkv_cache_view* cache,
    const void* q_new, const void* k_new, const void* v_new,
    const int32_t* u_pos, const int32_t* u_cu, const int32_t* r_rank, const int32_t* r_cu_layer,
    int64_t n_target_rows, const int32_t* h_max_targets, const int32_t* h_max_ctx,
    void* out, float* lse_out,
    void* workspace, size_t workspace_bytes, relaxkv_stream stream);

/*
 * Attention of given token positions over the cache's own causal prefix, cache only: target t of request b,
 * at position p = tgt_pos[tgt_cu[b] + t], attends to every cache entry j <= p of its request.  This is the pass
 * the paper runs after the repair loop (the user query's prefill rows and the first decode step read the
 * repaired cache; Section 3.4 and the TTFT protocol of the reproducibility appendix): the caller has appended
 * the K/V of those tokens to the cache, `shape->h_ctx_len[b]` counts them.  No context is gathered: the
 * kernel's tiled loads read the cache through its strides, so the call moves K and V once.
 *   q_new  device bf16 [n_target_rows, H, D], rows in tgt order, requests packed
 *   tgt_pos / tgt_cu  device int32: ascending positions per request, packed; offsets [B + 1], tgt_cu[0] = 0
 *   h_max_targets  host [B] upper bounds on the target counts
 *   out  device bf16 [n_target_rows, H, D]; lse_out optional device fp32 [H, n_target_rows]
 * The cache must hold max_b(h_req_token_offset[b] + h_ctx_len[b]) token rows.  Errors as for
 * relaxkv_sparse_ctx_attention (positions out of range are reported in the device status word).
 * When every h_max_targets[b] <= 1 (a decode step) the call takes a streaming kernel instead of the 128-row tensor-core
 * tiles: K and V tiles through a TMA ring, the request's few query heads in one warp-level MMA fragment, the context
 * split over one wave of thread blocks and merged in a fixed order.
 */
relaxkv_status relaxkv_cache_attention(
    const relaxkv_shape* shape, const relaxkv_cache_view* cache, const void* q_new,
    const int32_t* tgt_pos, const int32_t* tgt_cu, int64_t n_target_rows, const int32_t* h_max_targets,
    void* out, float* lse_out, void* workspace, size_t workspace_bytes, relaxkv_stream stream);

/*
 * Test utility for the bounded waits (the paper has no counterpart): launches one thread that waits on
 * a barrier nothing will ever complete.  The wait gives up after its limit (0.4 s), the kernel ends
 * normally and RELAXKV_ERR_TIMEOUT is recorded in the device status word - the same path a stuck
 * pipeline takes in the attention and scoring kernels.  Nothing hangs or faults.
 */
relaxkv_status relaxkv_debug_wait_timeout(relaxkv_stream stream);

/*
 * Chained launches.  The short kernels of a decode step (RMSNorm, norm + rotary and the cache append
 * of at most 8 rows, the one- to four-row projections, the one-token attention and its merge) are
 * launched with CUDA's programmatic stream serialization: the next kernel's blocks become resident
 * while the current kernel finishes, request the head of their weights into L2 (weights depend on
 * no earlier kernel) and then wait, inside the kernel, until every earlier kernel of the stream has
 * completed and its writes are visible.  Results are identical to plain
 * launches; stream order as the caller sees it is unchanged; the launches can be captured into a
 * CUDA graph.  relaxkv_set_chained_launch(0) switches to plain launches for the whole process
 * (1 = chained, the default) and returns the previous setting; it affects calls made after it.
 */
int32_t relaxkv_set_chained_launch(int32_t on);

/*
 * Synchronises `stream`, copies the device status word (a relaxkv_status: RELAXKV_OK,
 * RELAXKV_ERR_BAD_INDEX or RELAXKV_ERR_TIMEOUT, the first problem recorded wins) to
 * *h_status_out and clears it.  h_detail_out (NULL or host int32[4]) receives where it happened:
 * kernel id, block, and two kernel-specific values.
 */
relaxkv_status relaxkv_read_device_status(int32_t* h_status_out, int32_t* h_detail_out, relaxkv_stream stream);

#ifdef __cplusplus
}
#endif
#endif  /* RELAXKV_H_ */
