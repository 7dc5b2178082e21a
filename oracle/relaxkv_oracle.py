"""ctypes front end of the fp64 CPU oracle (oracle/relaxkv_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this module, and this module never imports them.

All functions take and return numpy arrays; bf16 tensors travel as uint16 bit
patterns.  Each wrapper names the passage of the paper its C function follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "relaxkv_oracle.c")
_LIB = os.path.join(_HERE, "librelaxkv_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (fp64, OpenMP over independent rows)."""
    with _lock:
        stale = force or (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                                   "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.relaxkv_oracle_anchor_count.restype = ctypes.c_int64
        _lib.relaxkv_oracle_anchor_count.argtypes = [ctypes.c_int64, ctypes.c_double]
        _lib.relaxkv_oracle_edges.restype = ctypes.c_int64
    return _lib


def n_threads() -> int:
    """Threads the OpenMP loops use (the host cores visible to this process)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _kv_strides(k: np.ndarray) -> Tuple[int, int]:
    """Element strides (token, head) of a [T, Hkv, D] uint16 array with D contiguous."""
    assert k.ndim == 3 and k.strides[2] == 2
    return k.strides[0] // 2, k.strides[1] // 2


# -- scores ------------------------------------------------------------------

def row_lse(q: np.ndarray, k: np.ndarray, scale: float) -> np.ndarray:
    """Log-normaliser of each query row's softmax over the context (Section 3.2).
    q [Q,H,D], k [T,Hkv,D] uint16 bf16 bits -> [H,Q] float64."""
    lib = _load()
    q = _u16(q)
    Qn, H, D = q.shape
    T, Hkv, _ = k.shape
    ts, hs = _kv_strides(k)
    out = np.empty((H, Qn), dtype=np.float64)
    lib.relaxkv_oracle_row_lse(_p(q), Qn, H, Hkv, D, _p(k), ctypes.c_int64(T), ctypes.c_int64(ts),
                               ctypes.c_int64(hs), ctypes.c_double(scale), _p(out))
    return out


def raw_scores(q: np.ndarray, k: np.ndarray, scale: float, lse: Optional[np.ndarray] = None) -> np.ndarray:
    """Mean over heads and query positions of the query's attention to each context
    position (Section 3.2, the argument of MinMax).  Returns [T] float64."""
    lib = _load()
    q = _u16(q)
    Qn, H, D = q.shape
    T, Hkv, _ = k.shape
    ts, hs = _kv_strides(k)
    if lse is None:
        lse = row_lse(q, k, scale)
    lse = np.ascontiguousarray(lse, dtype=np.float64)
    assert lse.shape == (H, Qn)
    raw = np.empty(T, dtype=np.float64)
    lib.relaxkv_oracle_raw_scores(_p(q), Qn, H, Hkv, D, _p(k), ctypes.c_int64(T), ctypes.c_int64(ts),
                                  ctypes.c_int64(hs), ctypes.c_double(scale), _p(lse), _p(raw))
    return raw


def minmax(raw: np.ndarray) -> np.ndarray:
    """MinMax normalisation within a layer (Section 3.2)."""
    lib = _load()
    raw = np.ascontiguousarray(raw, dtype=np.float64)
    a = np.empty_like(raw)
    lib.relaxkv_oracle_minmax(_p(raw), ctypes.c_int64(raw.shape[0]), _p(a))
    return a


def anchor_count(T: int, r: float) -> int:
    """k = max(1, round(r T_c)), clamped to T_c (Appendix A.1)."""
    return int(_load().relaxkv_oracle_anchor_count(int(T), float(r)))


def topk(score: np.ndarray, k: int) -> np.ndarray:
    """Positions of the k highest scores, ties to the lower index, ascending (Appendix A.1)."""
    lib = _load()
    score = np.ascontiguousarray(score, dtype=np.float64)
    out = np.empty(int(k), dtype=np.int32)
    lib.relaxkv_oracle_topk(_p(score), ctypes.c_int64(score.shape[0]), ctypes.c_int64(int(k)), _p(out))
    return out


# -- sets --------------------------------------------------------------------

class ActiveSets:
    """h_i, U (sorted positions), position->rank map and the per-layer active targets
    R_l as ascending ranks into U (Section 3.2; Algorithm 1)."""

    def __init__(self, h, u_pos, u_rank, r_rank, r_cu):
        self.h, self.u_pos, self.u_rank, self.r_rank, self.r_cu = h, u_pos, u_rank, r_rank, r_cu

    @property
    def n_layers(self) -> int:
        return len(self.r_cu) - 1

    def ranks(self, l: int) -> np.ndarray:
        return self.r_rank[self.r_cu[l]:self.r_cu[l + 1]]

    def positions(self, l: int) -> np.ndarray:
        return self.u_pos[self.ranks(l)]


def active_sets(anchors: np.ndarray, T: int) -> ActiveSets:
    lib = _load()
    anchors = _i32(anchors)
    L, k = anchors.shape
    h = np.empty(T, dtype=np.int32)
    u_pos = np.empty(T, dtype=np.int32)
    u_rank = np.empty(T, dtype=np.int32)
    r_rank = np.empty(L * T, dtype=np.int32)
    r_cu = np.empty(L + 1, dtype=np.int32)
    n_u = ctypes.c_int32(0)
    lib.relaxkv_oracle_active_sets(_p(anchors), L, ctypes.c_int64(k), ctypes.c_int64(T), _p(h), _p(u_pos),
                                   ctypes.byref(n_u), _p(u_rank), _p(r_rank), _p(r_cu))
    return ActiveSets(h, u_pos[:n_u.value].copy(), u_rank, r_rank[:r_cu[L]].copy(), r_cu)


# -- context, attention, update ----------------------------------------------

def mix_context(cache_k, cache_v, k_new, v_new, u_pos, r_rank):
    """Mixed fresh/cached K/V over the context list (Section 3.4 equation).
    Returns ctx_k, ctx_v [n_u, Hkv, D] uint16."""
    lib = _load()
    T, Hkv, D = cache_k.shape
    ts, hs = _kv_strides(cache_k)
    assert _kv_strides(cache_v) == (ts, hs)
    u_pos, r_rank = _i32(u_pos), _i32(r_rank)
    n_u, n_r = u_pos.shape[0], r_rank.shape[0]
    ck = np.empty((n_u, Hkv, D), dtype=np.uint16)
    cv = np.empty((n_u, Hkv, D), dtype=np.uint16)
    kn = None if k_new is None else _u16(k_new)
    vn = None if v_new is None else _u16(v_new)
    lib.relaxkv_oracle_mix_context(_p(cache_k), _p(cache_v), ctypes.c_int64(ts), ctypes.c_int64(hs),
                                   _p(kn), _p(vn), _p(u_pos), n_u, _p(r_rank), n_r, Hkv, D, _p(ck), _p(cv))
    return ck, cv


def attention(q_new, ctx_k, ctx_v, limit, scale, rows: Optional[Sequence[int]] = None):
    """Sparse-context repair attention for the listed target rows (all if None)
    (Section 3.3; Algorithm 1).  Returns out [n, H, D], lse [n, H] float64."""
    lib = _load()
    q_new, ctx_k, ctx_v = _u16(q_new), _u16(ctx_k), _u16(ctx_v)
    n_r, H, D = q_new.shape
    _, Hkv, _ = ctx_k.shape
    limit = _i32(limit)
    assert limit.shape[0] == n_r
    rows = np.arange(n_r, dtype=np.int32) if rows is None else _i32(rows)
    out = np.empty((rows.shape[0], H, D), dtype=np.float64)
    lse = np.empty((rows.shape[0], H), dtype=np.float64)
    lib.relaxkv_oracle_attention(_p(q_new), _p(ctx_k), _p(ctx_v), _p(limit), _p(rows),
                                 ctypes.c_int64(rows.shape[0]), H, Hkv, D, ctypes.c_double(scale),
                                 _p(out), _p(lse))
    return out, lse


def repair_attention(cache_k, cache_v, q_new, k_new, v_new, u_pos, r_rank, scale,
                     full_prefix: bool = False, rows: Optional[Sequence[int]] = None):
    """One layer of repair attention in the paper's order: gather the context,
    replace the active entries with the fresh states, attend under the causal
    restriction.  full_prefix=True is the Full-Prefix Control of Appendix A.3/A.4:
    same targets, context = every position j <= p."""
    u_pos, r_rank = _i32(u_pos), _i32(r_rank)
    if full_prefix:
        T = cache_k.shape[0]
        pos = u_pos[r_rank]
        ck, cv = mix_context(cache_k, cache_v, k_new, v_new, np.arange(T, dtype=np.int32), pos)
        limit = pos
    else:
        ck, cv = mix_context(cache_k, cache_v, k_new, v_new, u_pos, r_rank)
        limit = r_rank
    return attention(q_new, ck, cv, limit, scale, rows)


def limits(ctx_pos, tgt_pos) -> np.ndarray:
    """Causal limit of each target in an arbitrary context list: index of the last context position
    <= the target's position, -1 if there is none (Appendix A.3: C_l(p) = X intersect {j <= p})."""
    lib = _load()
    ctx_pos, tgt_pos = _i32(ctx_pos), _i32(tgt_pos)
    out = np.empty(tgt_pos.shape[0], dtype=np.int32)
    lib.relaxkv_oracle_limits(_p(ctx_pos), ctx_pos.shape[0], _p(tgt_pos), tgt_pos.shape[0], _p(out))
    return out


def mix_context_lists(cache_k, cache_v, k_new, v_new, ctx_pos, tgt_pos):
    """Mixed fresh/cached K/V over an explicit context list for an explicit target list."""
    lib = _load()
    T, Hkv, D = cache_k.shape
    ts, hs = _kv_strides(cache_k)
    assert _kv_strides(cache_v) == (ts, hs)
    ctx_pos, tgt_pos = _i32(ctx_pos), _i32(tgt_pos)
    ck = np.empty((ctx_pos.shape[0], Hkv, D), dtype=np.uint16)
    cv = np.empty_like(ck)
    kn = None if k_new is None else _u16(k_new)
    vn = None if v_new is None else _u16(v_new)
    lib.relaxkv_oracle_mix_context_lists(_p(cache_k), _p(cache_v), ctypes.c_int64(ts), ctypes.c_int64(hs), _p(kn), _p(vn),
                                         _p(ctx_pos), ctx_pos.shape[0], _p(tgt_pos), tgt_pos.shape[0], Hkv, D,
                                         _p(ck), _p(cv))
    return ck, cv


def list_attention(cache_k, cache_v, q_new, k_new, v_new, ctx_pos, tgt_pos, scale, rows=None):
    """Repair attention of the controlled configurations (Appendix A.3): targets tgt_pos (any ascending
    list) attend to the context list ctx_pos under C(p) = ctx intersect {j <= p}; context entries that
    are targets contribute their fresh K/V.  A target with an empty context yields zeros (lse = -inf)."""
    ck, cv = mix_context_lists(cache_k, cache_v, k_new, v_new, ctx_pos, tgt_pos)
    return attention(q_new, ck, cv, limits(ctx_pos, tgt_pos), scale, rows)


def mean_scores(scores: np.ndarray) -> np.ndarray:
    """g_i = mean over layers of a_{l,i} (Appendix B, global repair target sweep)."""
    lib = _load()
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    L, T = scores.shape
    g = np.empty(T, dtype=np.float64)
    lib.relaxkv_oracle_mean_scores(_p(scores), L, ctypes.c_int64(T), _p(g))
    return g


def scatter(cache_k, cache_v, k_new, v_new, positions) -> None:
    """Cache update in place on the numpy arrays (Section 3.4)."""
    lib = _load()
    T, Hkv, D = cache_k.shape
    ts, hs = _kv_strides(cache_k)
    assert _kv_strides(cache_v) == (ts, hs)
    assert cache_k.flags.writeable and cache_v.flags.writeable
    positions = _i32(positions)
    lib.relaxkv_oracle_scatter(_p(cache_k), _p(cache_v), ctypes.c_int64(ts), ctypes.c_int64(hs),
                               _p(_u16(k_new)), _p(_u16(v_new)), _p(positions), positions.shape[0], Hkv, D)


def edges(limit) -> int:
    """Causal attention edges of one layer: sum over targets of |C_l(p)| (Appendix A.2)."""
    limit = _i32(limit)
    return int(_load().relaxkv_oracle_edges(_p(limit), ctypes.c_int64(limit.shape[0])))
