/*
 * RelaxKV selective cache-repair hot path: plain fp64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement
 * of what the path computes.  It shares no code with the CUDA library and is
 * imported only by the tests, the smoke check and the benchmark's CPU-baseline
 * leg.  Nothing here is blocked, fused or reordered beyond what the paper's
 * definitions state; OpenMP only spreads independent rows over cores.
 *
 * Inputs are bf16 bit patterns (uint16_t), widened exactly to double; all
 * arithmetic is fp64.  Layout conventions:
 *   Q      [n_rows, H, D]          (row = query token or active target)
 *   K, V   element (i, g, d) at  i*tok_stride + g*head_stride + d   (elements)
 *   query head h reads KV head h / (H / H_kv)
 *
 * Parity pins: every function below is pinned by tests/test_oracle_pins.py
 * against closed forms, library routines and a dense-mask brute force
 * (tests/bruteforce.py).  What cannot be pinned here is the behaviour of the
 * method on real models (quality, realised set ratios): "parity unpinned" for
 * that, since it needs weights and datasets.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <fenv.h>

static inline double bf16_to_f64(uint16_t b) {
    union { uint32_t u; float f; } x;
    x.u = ((uint32_t)b) << 16;
    return (double)x.f;
}

static double dot_qk(const uint16_t* q, const uint16_t* k, int D) {
    double s = 0.0;
    for (int d = 0; d < D; ++d) s += bf16_to_f64(q[d]) * bf16_to_f64(k[d]);
    return s;
}

/* ---- Section 3.2, score equation: the log-normaliser of each query row ----
 * lse[h*Q + t] = log sum_i exp(scale * <q_{t,h}, k_{i, h/G}>)  over all context
 * positions i (softmax domain = the cached context). */
void relaxkv_oracle_row_lse(const uint16_t* q, int Q, int H, int Hkv, int D,
                            const uint16_t* k, int64_t T, int64_t tok_stride, int64_t head_stride,
                            double scale, double* lse) {
    const int G = H / Hkv;
    #pragma omp parallel for collapse(2) schedule(static)
    for (int h = 0; h < H; ++h) {
        for (int t = 0; t < Q; ++t) {
            const uint16_t* qr = q + ((int64_t)t * H + h) * D;
            const int g = h / G;
            double m = -INFINITY;
            for (int64_t i = 0; i < T; ++i) {
                double s = scale * dot_qk(qr, k + i * tok_stride + g * head_stride, D);
                if (s > m) m = s;
            }
            double z = 0.0;
            for (int64_t i = 0; i < T; ++i) {
                double s = scale * dot_qk(qr, k + i * tok_stride + g * head_stride, D);
                z += exp(s - m);
            }
            lse[(int64_t)h * Q + t] = m + log(z);
        }
    }
}

/* ---- Section 3.2, score equation (before MinMax) ----
 * raw[i] = 1/(H*Q) * sum_h sum_t A[h,t,i],  A[h,t,i] = exp(s[h,t,i] - lse[h,t]).
 * With lse from relaxkv_oracle_row_lse, A is the softmax over the context; a
 * caller-supplied lse (e.g. one that also covers the query's own keys) gives the
 * attention weights of that wider softmax restricted to the context. */
void relaxkv_oracle_raw_scores(const uint16_t* q, int Q, int H, int Hkv, int D,
                               const uint16_t* k, int64_t T, int64_t tok_stride, int64_t head_stride,
                               double scale, const double* lse, double* raw) {
    const int G = H / Hkv;
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < T; ++i) {
        double acc = 0.0;
        for (int h = 0; h < H; ++h) {
            const uint16_t* kr = k + i * tok_stride + (h / G) * head_stride;
            for (int t = 0; t < Q; ++t) {
                double s = scale * dot_qk(q + ((int64_t)t * H + h) * D, kr, D);
                acc += exp(s - lse[(int64_t)h * Q + t]);
            }
        }
        raw[i] = acc / ((double)H * (double)Q);
    }
}

/* ---- Section 3.2: MinMax within the layer.  No epsilon; a constant vector maps to zeros. */
void relaxkv_oracle_minmax(const double* raw, int64_t T, double* a) {
    double lo = INFINITY, hi = -INFINITY;
    for (int64_t i = 0; i < T; ++i) { if (raw[i] < lo) lo = raw[i]; if (raw[i] > hi) hi = raw[i]; }
    for (int64_t i = 0; i < T; ++i) a[i] = (hi > lo) ? (raw[i] - lo) / (hi - lo) : 0.0;
}

/* ---- Appendix A.1, anchor-count equation: k = max(1, round(r*T_c)), clamped to T_c.
 * round = nearest, halves to even, on the fp64 product (what Python's round does). */
int64_t relaxkv_oracle_anchor_count(int64_t T, double r) {
    fesetround(FE_TONEAREST);
    double x = nearbyint(r * (double)T);
    int64_t k = (int64_t)x;
    if (k < 1) k = 1;
    if (k > T) k = T;
    return k;
}

/* ---- Appendix A.1, TopK: the k highest scores; equal scores -> lower index first;
 * emitted in ascending position order. */
typedef struct { double s; int32_t i; } scored;
static int cmp_scored(const void* a, const void* b) {
    const scored* x = (const scored*)a; const scored* y = (const scored*)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->i > y->i) - (x->i < y->i);
}
static int cmp_i32(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return (x > y) - (x < y);
}
void relaxkv_oracle_topk(const double* score, int64_t T, int64_t k, int32_t* out) {
    scored* v = (scored*)malloc(sizeof(scored) * (size_t)T);
    for (int64_t i = 0; i < T; ++i) { v[i].s = score[i]; v[i].i = (int32_t)i; }
    qsort(v, (size_t)T, sizeof(scored), cmp_scored);
    for (int64_t j = 0; j < k; ++j) out[j] = v[j].i;
    qsort(out, (size_t)k, sizeof(int32_t), cmp_i32);
    free(v);
}

/* ---- Section 3.2 / Algorithm 1 (union, highest selected layer, active targets) ----
 * anchors [L][k] positions.  Outputs: h[T] (-1 outside U); u_pos[n_u] ascending;
 * u_rank[T] (position -> index in u_pos, -1 outside U); for each layer the active
 * targets as ascending indices into u_pos, packed at r_cu[l] .. r_cu[l+1].
 * r_rank must hold L*T entries at most. */
void relaxkv_oracle_active_sets(const int32_t* anchors, int L, int64_t k, int64_t T,
                                int32_t* h, int32_t* u_pos, int32_t* n_u, int32_t* u_rank,
                                int32_t* r_rank, int32_t* r_cu) {
    for (int64_t i = 0; i < T; ++i) h[i] = -1;
    for (int l = 0; l < L; ++l)
        for (int64_t j = 0; j < k; ++j) {
            int32_t i = anchors[(int64_t)l * k + j];
            if (l > h[i]) h[i] = l;
        }
    int32_t n = 0;
    for (int64_t i = 0; i < T; ++i) {
        if (h[i] >= 0) { u_pos[n] = (int32_t)i; u_rank[i] = n; ++n; } else u_rank[i] = -1;
    }
    *n_u = n;
    int32_t w = 0;
    for (int l = 0; l < L; ++l) {
        r_cu[l] = w;
        for (int32_t c = 0; c < n; ++c)
            if (h[u_pos[c]] >= l) r_rank[w++] = c;
    }
    r_cu[L] = w;
}

/* ---- Section 3.4 / Appendix A.2, mixed fresh-cached context ----
 * ctx[c] = new[rho] if c == r_rank[rho] for some rho, else cache[u_pos[c]].
 * Bit copy.  ctx_k/ctx_v are dense [n_u, Hkv, D]. */
void relaxkv_oracle_mix_context(const uint16_t* cache_k, const uint16_t* cache_v,
                                int64_t tok_stride, int64_t head_stride,
                                const uint16_t* k_new, const uint16_t* v_new,
                                const int32_t* u_pos, int32_t n_u,
                                const int32_t* r_rank, int32_t n_r,
                                int Hkv, int D, uint16_t* ctx_k, uint16_t* ctx_v) {
    for (int32_t c = 0; c < n_u; ++c)
        for (int g = 0; g < Hkv; ++g) {
            const int64_t src = (int64_t)u_pos[c] * tok_stride + (int64_t)g * head_stride;
            memcpy(ctx_k + ((int64_t)c * Hkv + g) * D, cache_k + src, sizeof(uint16_t) * D);
            memcpy(ctx_v + ((int64_t)c * Hkv + g) * D, cache_v + src, sizeof(uint16_t) * D);
        }
    if (k_new && v_new)
        for (int32_t rho = 0; rho < n_r; ++rho) {
            const int32_t c = r_rank[rho];
            memcpy(ctx_k + (int64_t)c * Hkv * D, k_new + (int64_t)rho * Hkv * D, sizeof(uint16_t) * Hkv * D);
            memcpy(ctx_v + (int64_t)c * Hkv * D, v_new + (int64_t)rho * Hkv * D, sizeof(uint16_t) * Hkv * D);
        }
}

/* ---- Appendix A.3 (controlled configurations): any target list against any context list ----
 * The variants (global targets P, Global / Layerwise Sparse context sets U_l) keep the definition
 * C_l(p) = X intersect {j <= p} with their own context list X and target list; a target need not be
 * a member of X.  limit[rho] = (number of context positions <= tgt_pos[rho]) - 1, i.e. -1 when the
 * target sees nothing.  Both lists ascending. */
void relaxkv_oracle_limits(const int32_t* ctx_pos, int32_t n_ctx, const int32_t* tgt_pos, int32_t n_tgt, int32_t* limit) {
    for (int32_t r = 0; r < n_tgt; ++r) {
        int32_t n = 0;
        for (int32_t c = 0; c < n_ctx; ++c) if (ctx_pos[c] <= tgt_pos[r]) ++n;
        limit[r] = n - 1;
    }
}

/* Mixed context for explicit lists (Section 3.4 equation with R_l := the target list):
 * ctx[c] = new[rho] if ctx_pos[c] == tgt_pos[rho] for some rho, else cache[ctx_pos[c]]. */
void relaxkv_oracle_mix_context_lists(const uint16_t* cache_k, const uint16_t* cache_v,
                                      int64_t tok_stride, int64_t head_stride,
                                      const uint16_t* k_new, const uint16_t* v_new,
                                      const int32_t* ctx_pos, int32_t n_ctx, const int32_t* tgt_pos, int32_t n_tgt,
                                      int Hkv, int D, uint16_t* ctx_k, uint16_t* ctx_v) {
    for (int32_t c = 0; c < n_ctx; ++c) {
        int32_t rho = -1;
        if (k_new && v_new)
            for (int32_t r = 0; r < n_tgt; ++r) if (tgt_pos[r] == ctx_pos[c]) rho = r;
        for (int g = 0; g < Hkv; ++g) {
            uint16_t* dk = ctx_k + ((int64_t)c * Hkv + g) * D;
            uint16_t* dv = ctx_v + ((int64_t)c * Hkv + g) * D;
            if (rho >= 0) {
                memcpy(dk, k_new + ((int64_t)rho * Hkv + g) * D, sizeof(uint16_t) * D);
                memcpy(dv, v_new + ((int64_t)rho * Hkv + g) * D, sizeof(uint16_t) * D);
            } else {
                const int64_t src = (int64_t)ctx_pos[c] * tok_stride + (int64_t)g * head_stride;
                memcpy(dk, cache_k + src, sizeof(uint16_t) * D);
                memcpy(dv, cache_v + src, sizeof(uint16_t) * D);
            }
        }
    }
}

/* ---- Appendix B (global repair target sweep): g_i = (1/L) sum_l a_{l,i} ---- */
void relaxkv_oracle_mean_scores(const double* scores, int L, int64_t T, double* g) {
    for (int64_t i = 0; i < T; ++i) {
        double a = 0.0;
        for (int l = 0; l < L; ++l) a += scores[(int64_t)l * T + i];
        g[i] = a / (double)L;
    }
}

/* ---- Section 3.3 / Algorithm 1, sparse-context repair attention ----
 * For each listed target row rho (rows[] indexes q_new and limit[]), head h:
 *   O[rho,h,:] = sum_{c<=limit[rho]} softmax_c(scale*<q, ctx_k[c, h/G]>) * ctx_v[c, h/G, :]
 * limit[rho] = index in the context list of the target's own position, so the sum
 * runs over C_l(p) = U intersect {j <= p}, the target itself included.
 * out [n_rows, H, D] and lse [n_rows, H] follow the order of rows[]. */
void relaxkv_oracle_attention(const uint16_t* q_new, const uint16_t* ctx_k, const uint16_t* ctx_v,
                              const int32_t* limit, const int32_t* rows, int64_t n_rows,
                              int H, int Hkv, int D, double scale, double* out, double* lse) {
    const int G = H / Hkv;
    #pragma omp parallel for collapse(2) schedule(dynamic, 4)
    for (int64_t r = 0; r < n_rows; ++r) {
        for (int h = 0; h < H; ++h) {
            const int32_t rho = rows[r];
            const int32_t cmax = limit[rho];
            const int g = h / G;
            if (cmax < 0) {            /* empty context (only possible with explicit lists): defined as zero output */
                for (int d = 0; d < D; ++d) out[((int64_t)r * H + h) * D + d] = 0.0;
                if (lse) lse[(int64_t)r * H + h] = -INFINITY;
                continue;
            }
            const uint16_t* qr = q_new + ((int64_t)rho * H + h) * D;
            double m = -INFINITY;
            for (int32_t c = 0; c <= cmax; ++c) {
                double s = scale * dot_qk(qr, ctx_k + ((int64_t)c * Hkv + g) * D, D);
                if (s > m) m = s;
            }
            double z = 0.0;
            double* o = out + ((int64_t)r * H + h) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            for (int32_t c = 0; c <= cmax; ++c) {
                double s = scale * dot_qk(qr, ctx_k + ((int64_t)c * Hkv + g) * D, D);
                double w = exp(s - m);
                z += w;
                const uint16_t* vr = ctx_v + ((int64_t)c * Hkv + g) * D;
                for (int d = 0; d < D; ++d) o[d] += w * bf16_to_f64(vr[d]);
            }
            for (int d = 0; d < D; ++d) o[d] /= z;
            if (lse) lse[(int64_t)r * H + h] = m + log(z);
        }
    }
}

/* ---- Section 3.4 / Algorithm 1, cache update: entries of the active targets are
 * overwritten with the fresh states; everything else is untouched. */
void relaxkv_oracle_scatter(uint16_t* cache_k, uint16_t* cache_v, int64_t tok_stride, int64_t head_stride,
                            const uint16_t* k_new, const uint16_t* v_new,
                            const int32_t* positions, int32_t n_r, int Hkv, int D) {
    for (int32_t rho = 0; rho < n_r; ++rho)
        for (int g = 0; g < Hkv; ++g) {
            const int64_t dst = (int64_t)positions[rho] * tok_stride + (int64_t)g * head_stride;
            memcpy(cache_k + dst, k_new + ((int64_t)rho * Hkv + g) * D, sizeof(uint16_t) * D);
            memcpy(cache_v + dst, v_new + ((int64_t)rho * Hkv + g) * D, sizeof(uint16_t) * D);
        }
}

/* ---- Appendix A.2, edge count of one layer: sum over active targets of |C_l(p)|. */
int64_t relaxkv_oracle_edges(const int32_t* limit, int64_t n_r) {
    int64_t e = 0;
    for (int64_t r = 0; r < n_r; ++r) e += (int64_t)limit[r] + 1;
    return e;
}
