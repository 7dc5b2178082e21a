"""Dense-matrix numpy fp64 brute force of the repair path, for tiny inputs only.

It takes a different route from the C oracle on purpose: full [H, Q, T] softmax
matrices, a dense boolean [targets, T] visibility mask built from *positions*
(not ranks), `np.where` for the fresh/cached mix, `np.lexsort` for top-k and
Python set algebra for the sets.  Used only to check the oracle.
"""
from __future__ import annotations

import numpy as np


def f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def raw_scores(q_bits, k_bits, scale):
    q, k = f64(q_bits), f64(k_bits)                  # [Q,H,D], [T,Hkv,D]
    Qn, H, D = q.shape
    T, Hkv, _ = k.shape
    kx = np.repeat(k, H // Hkv, axis=1)               # [T,H,D]  (HF repeat_kv order)
    s = np.einsum("thd,ihd->hti", q, kx) * scale      # [H,Q,T]
    s = s - s.max(axis=-1, keepdims=True)
    a = np.exp(s)
    a /= a.sum(axis=-1, keepdims=True)
    return a.mean(axis=(0, 1))


def minmax(raw):
    lo, hi = raw.min(), raw.max()
    return np.zeros_like(raw) if hi == lo else (raw - lo) / (hi - lo)


def topk(score, k):
    T = score.shape[0]
    order = np.lexsort((np.arange(T), -score))        # primary: score descending; then index
    return np.sort(order[:k]).astype(np.int32)


def sets(anchor_lists, T):
    """anchor_lists: list over layers of iterables of positions."""
    S = [set(int(i) for i in a) for a in anchor_lists]
    U = set().union(*S)
    h = {i: max(l for l, s in enumerate(S) if i in s) for i in U}
    R = [sorted(i for i in U if h[i] >= l) for l in range(len(S))]
    return sorted(U), h, R


def attention(cache_k, cache_v, q_new, k_new, v_new, U, R_pos, scale, full_prefix=False):
    """Dense route: scatter the fresh states into full-length copies, build the
    [n_r, T] visibility mask from positions, masked softmax, P @ V."""
    ck, cv, q = f64(cache_k), f64(cache_v), f64(q_new)
    T, Hkv, D = ck.shape
    n_r, H, _ = q.shape
    G = H // Hkv
    R_pos = np.asarray(R_pos, dtype=np.int64)
    is_r = np.zeros(T, dtype=bool)
    is_r[R_pos] = True
    kn_full = np.zeros_like(ck)
    vn_full = np.zeros_like(cv)
    if k_new is not None:
        kn_full[R_pos] = f64(k_new)
        vn_full[R_pos] = f64(v_new)
        k_eff = np.where(is_r[:, None, None], kn_full, ck)
        v_eff = np.where(is_r[:, None, None], vn_full, cv)
    else:
        k_eff, v_eff = ck, cv
    in_ctx = np.ones(T, dtype=bool) if full_prefix else np.isin(np.arange(T), np.asarray(U))
    vis = in_ctx[None, :] & (np.arange(T)[None, :] <= R_pos[:, None])        # [n_r, T]
    out = np.zeros((n_r, H, D))
    lse = np.zeros((n_r, H))
    for h in range(H):
        s = (q[:, h, :] @ k_eff[:, h // G, :].T) * scale                      # [n_r, T]
        s = np.where(vis, s, -np.inf)
        m = s.max(axis=1, keepdims=True)
        empty = ~np.isfinite(m[:, 0])                                         # no visible position at all
        m = np.where(np.isfinite(m), m, 0.0)
        p = np.exp(s - m)
        z = p.sum(axis=1, keepdims=True)
        z_safe = np.where(z > 0, z, 1.0)
        out[:, h, :] = (p / z_safe) @ v_eff[:, h // G, :]
        with np.errstate(divide="ignore"):
            lse[:, h] = np.where(empty, -np.inf, (m + np.log(z_safe))[:, 0])
    return out, lse, int(vis.sum())
