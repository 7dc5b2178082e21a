"""fp64 numpy oracle of the dense per-row block work around the repair attention (Algorithm 1, steps 14, 16,
20: the projections of the active repair targets, then the block's own output projection, residuals,
normalisation and MLP, all unchanged; Section 3.3: RoPE keeps the original global position IDs).

TEST INFRASTRUCTURE ONLY, like relaxkv_oracle: plain definitions of a Llama-style pre-norm decoder block
(RMSNorm -> fused QKV projection -> rotary embedding on q and k -> [attention] -> output projection +
residual -> RMSNorm -> SwiGLU MLP + residual), one function per operation, no blocking or fusion.  bf16
tensors come in as uint16 bit patterns and are widened exactly; all arithmetic is float64.
"""
from __future__ import annotations

import numpy as np


def f64(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rmsnorm(x: np.ndarray, w: np.ndarray, eps: float) -> np.ndarray:
    """y = x / sqrt(mean(x^2) + eps) * w, row-wise.  x [rows, C], w [C] (float64)."""
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * w


def linear(x: np.ndarray, weight: np.ndarray, residual=None) -> np.ndarray:
    """y = x @ weight^T (+ residual).  x [rows, K], weight [N, K] (the HF [out, in] layout)."""
    y = x @ weight.T
    return y if residual is None else y + residual


def rope(x: np.ndarray, positions: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, rotate-half convention (Llama / Qwen): for pair i < D/2 of head vector v,
    angle = position * theta^(-2i/D); (v[i], v[i + D/2]) is rotated by that angle.
    x [rows, heads, D], positions [rows] (the tokens' ORIGINAL global positions)."""
    rows, heads, D = x.shape
    half = D // 2
    inv_freq = theta ** (-np.arange(half, dtype=np.float64) * 2.0 / D)
    ang = positions.astype(np.float64)[:, None] * inv_freq[None, :]          # [rows, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def swiglu(gate_up: np.ndarray) -> np.ndarray:
    """silu(gate) * up for a fused projection output [rows, 2*I] = [gate | up]."""
    inter = gate_up.shape[-1] // 2
    g, u = gate_up[..., :inter], gate_up[..., inter:]
    return g / (1.0 + np.exp(-g)) * u


def compact_rows(h: np.ndarray, ranks_l: np.ndarray, ranks_next: np.ndarray) -> np.ndarray:
    """Hidden states of the targets that stay active: rows of h (ordered like R_l) whose rank is in R_{l+1}
    (R_{l+1} is a subset of R_l; both ascending)."""
    keep = np.isin(ranks_l, ranks_next)
    assert keep.sum() == len(ranks_next)
    return h[keep]


def decoder_block(h: np.ndarray, W: dict, n_q_heads: int, n_kv_heads: int, head_dim: int, positions: np.ndarray,
                  eps: float, theta: float, attend, store=lambda t: t) -> np.ndarray:
    """One pre-norm decoder block on the given rows, written out operation by operation in the order the paper's
    loop runs them (Algorithm 1, steps 14-22 for the active targets; the same block serves the query's prefill rows
    and a decode token): input RMSNorm, Q/K/V projections, per-head Q/K RMSNorm when the weights have one, rotary
    embedding at `positions`, attention, output projection + residual, post-attention RMSNorm, SwiGLU MLP + residual.

    h [rows, hidden] float64; W: float64 weights (w_in_norm, wq, wk, wv, optional w_q_norm / w_k_norm, wo, w_post_norm,
    w_gate_up = [gate; up] stacked, w_down).  attend(q [rows, H, D], k [rows, Hkv, D], v [rows, Hkv, D]) -> o [rows, H, D]
    is the attention of these rows (the caller decides what they see).  `store` is applied wherever a tensor is
    written to memory between two operations (identity: pure float64; a bf16 rounding models bf16 storage)."""
    n = h.shape[0]
    H, Hkv, D = n_q_heads, n_kv_heads, head_dim
    x = store(rmsnorm(h, W["w_in_norm"], eps))
    q = store(linear(x, W["wq"])).reshape(n, H, D)
    k = store(linear(x, W["wk"])).reshape(n, Hkv, D)
    v = store(linear(x, W["wv"])).reshape(n, Hkv, D)
    if "w_q_norm" in W:
        q = store(rmsnorm(q.reshape(n * H, D), W["w_q_norm"], eps)).reshape(n, H, D)
        k = store(rmsnorm(k.reshape(n * Hkv, D), W["w_k_norm"], eps)).reshape(n, Hkv, D)
    q, k = store(rope(q, positions, theta)), store(rope(k, positions, theta))
    o = store(attend(q, k, v)).reshape(n, H * D)
    a = store(linear(o, W["wo"], h))
    x2 = store(rmsnorm(a, W["w_post_norm"], eps))
    m = store(swiglu(linear(x2, W["w_gate_up"])))
    return store(linear(m, W["w_down"], a))


def output_head(h_row: np.ndarray, w_final_norm: np.ndarray, w_head: np.ndarray, eps: float, store=lambda t: t) -> np.ndarray:
    """Logits of one row per request: final RMSNorm, then the output projection [vocab, hidden]."""
    return store(linear(store(rmsnorm(h_row, w_final_norm, eps)), w_head))
