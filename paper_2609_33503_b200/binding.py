"""Python binding of the RelaxKV C ABI (include/relaxkv.h): argument marshalling only.

Every function here has the name of the C entry point it calls and does nothing but turn torch
tensors and Python lists into pointers and sizes.  All computation runs in the CUDA kernels of
librelaxkv.so; there is no CPU path and no fallback: if the library has not been built, loading
fails with an error.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librelaxkv.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_BAD_INDEX, ERR_TIMEOUT = range(7)
CTX_UNION, CTX_FULL_PREFIX = 0, 1

ENTRY_POINTS = (
    "relaxkv_status_string", "relaxkv_anchor_count", "relaxkv_workspace_bytes", "relaxkv_score_select",
    "relaxkv_build_active_sets", "relaxkv_sparse_ctx_attention", "relaxkv_scatter_kv", "relaxkv_gather_kv",
    "relaxkv_sparse_ctx_attention_simt", "relaxkv_read_device_status", "relaxkv_select_topk",
    "relaxkv_build_active_sets_static", "relaxkv_debug_wait_timeout",
    "relaxkv_list_attention", "relaxkv_cache_attention",
    "relaxkv_scatter_kv_lists", "relaxkv_mean_scores", "relaxkv_scale_scores", "relaxkv_query_prefill_attention", "relaxkv_rmsnorm", "relaxkv_linear", "relaxkv_linear_qkv", "relaxkv_linear_swiglu", "relaxkv_rope", "relaxkv_qk_norm_rope",
    "relaxkv_swiglu", "relaxkv_target_positions", "relaxkv_carry_rows", "relaxkv_set_chained_launch",
)


class RelaxKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class _Tuning(ctypes.Structure):
    _fields_ = [("attention_ctx_splits", ctypes.c_int32), ("attention_persistent", ctypes.c_int32),
                ("attention_grid_blocks", ctypes.c_int32)]


class _Shape(ctypes.Structure):
    _fields_ = [("n_req", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("h_ctx_len", ctypes.POINTER(ctypes.c_int32)),
                ("h_q_len", ctypes.POINTER(ctypes.c_int32)), ("softmax_scale", ctypes.c_float),
                ("h_tuning", ctypes.POINTER(_Tuning))]


class _CacheView(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("token_stride", ctypes.c_int64),
                ("head_stride", ctypes.c_int64), ("h_req_token_offset", ctypes.POINTER(ctypes.c_int64))]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_33503_b200.build` "
                               "(nvcc, sm_100a). There is no CPU fallback.")
        l = ctypes.CDLL(LIB_PATH)
        l.relaxkv_status_string.restype = ctypes.c_char_p
        l.relaxkv_status_string.argtypes = [ctypes.c_int32]
        l.relaxkv_anchor_count.restype = ctypes.c_int32
        l.relaxkv_anchor_count.argtypes = [ctypes.c_int32, ctypes.c_double]
        l.relaxkv_workspace_bytes.restype = ctypes.c_size_t
        l.relaxkv_workspace_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p]
        for name in ENTRY_POINTS[3:]:
            getattr(l, name).restype = ctypes.c_int32
        _lib = l
    return _lib


def status_string(status: int) -> str:
    return lib().relaxkv_status_string(int(status)).decode()


def relaxkv_set_chained_launch(on: bool) -> bool:
    """Chained (programmatic dependent) launches of the short kernels on or off, process-wide; returns the previous
    setting."""
    return bool(lib().relaxkv_set_chained_launch(1 if on else 0))


def _check(status: int, where: str) -> None:
    if status != OK:
        raise RelaxKVError(status, where)


def _i32(xs: Optional[Sequence[int]]):
    if xs is None:
        return None
    return (ctypes.c_int32 * len(xs))(*[int(x) for x in xs])


def _ptr(t: Optional[torch.Tensor]):
    return ctypes.c_void_p(None) if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


class Shape:
    """Host-side relaxkv_shape; keeps its arrays alive."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, ctx_lens: Sequence[int],
                 q_lens: Optional[Sequence[int]] = None, softmax_scale: Optional[float] = None,
                 attention_ctx_splits: int = 0, attention_persistent: int = 0, attention_grid_blocks: int = 0):
        self.ctx_lens = [int(x) for x in ctx_lens]
        self.q_lens = None if q_lens is None else [int(x) for x in q_lens]
        self._ctx = _i32(self.ctx_lens)
        self._q = _i32(self.q_lens)
        self.c = _Shape()
        self.c.n_req = len(self.ctx_lens)
        self.c.n_q_heads, self.c.n_kv_heads, self.c.head_dim = int(n_q_heads), int(n_kv_heads), int(head_dim)
        self.c.h_ctx_len = ctypes.cast(self._ctx, ctypes.POINTER(ctypes.c_int32))
        self.c.h_q_len = ctypes.cast(self._q, ctypes.POINTER(ctypes.c_int32)) if self._q is not None else None
        self.c.softmax_scale = float(softmax_scale if softmax_scale is not None else head_dim ** -0.5)
        self._tuning = None
        self.set_tuning(attention_ctx_splits, attention_persistent, attention_grid_blocks)

    def set_tuning(self, attention_ctx_splits: int = 0, attention_persistent: int = 0, attention_grid_blocks: int = 0) -> None:
        """relaxkv_tuning of the calls made with this shape (0 = the library's automatic choice)."""
        if attention_ctx_splits or attention_persistent or attention_grid_blocks:
            self._tuning = _Tuning(int(attention_ctx_splits), int(attention_persistent), int(attention_grid_blocks))
            self.c.h_tuning = ctypes.pointer(self._tuning)
        else:
            self._tuning = None
            self.c.h_tuning = None

    @property
    def n_req(self) -> int:
        return len(self.ctx_lens)

    def ref(self):
        return ctypes.byref(self.c)


class CacheView:
    """Host-side relaxkv_cache_view over torch tensors k, v of logical shape [tokens, H_kv, D]
    (any token/head strides, D contiguous); requests start at the given token rows."""

    def __init__(self, k: torch.Tensor, v: Optional[torch.Tensor], req_token_offsets: Sequence[int]):
        assert k.dim() == 3 and k.stride(2) == 1 and k.dtype == torch.bfloat16
        if v is not None:
            assert v.shape == k.shape and v.stride() == k.stride() and v.dtype == torch.bfloat16
        self.k, self.v = k, v
        self._off = (ctypes.c_int64 * len(req_token_offsets))(*[int(x) for x in req_token_offsets])
        self.c = _CacheView()
        self.c.k = k.data_ptr()
        self.c.v = v.data_ptr() if v is not None else None
        self.c.token_stride, self.c.head_stride = int(k.stride(0)), int(k.stride(1))
        self.c.h_req_token_offset = ctypes.cast(self._off, ctypes.POINTER(ctypes.c_int64))

    def ref(self):
        return ctypes.byref(self.c)


def relaxkv_anchor_count(ctx_len: int, ratio: float) -> int:
    return int(lib().relaxkv_anchor_count(int(ctx_len), float(ratio)))


def relaxkv_workspace_bytes(shape: Shape, n_layers: int, k: Optional[Sequence[int]] = None) -> int:
    return int(lib().relaxkv_workspace_bytes(shape.ref(), int(n_layers), _i32(k)))


def relaxkv_score_select(shape: Shape, q_layers: List[torch.Tensor], cache_layers: List[CacheView],
                         k: Sequence[int], raw_scores_out: torch.Tensor, anchors_out: Optional[torch.Tensor],
                         workspace: torch.Tensor, norm_scores_out: Optional[torch.Tensor] = None,
                         row_lse_layers: Optional[List[Optional[torch.Tensor]]] = None, stream=None) -> None:
    n_layers = len(q_layers)
    qs = (ctypes.c_void_p * n_layers)(*[q.data_ptr() for q in q_layers])
    caches = (_CacheView * n_layers)(*[c.c for c in cache_layers])
    lses = None
    if row_lse_layers is not None:
        lses = (ctypes.c_void_p * n_layers)(*[(t.data_ptr() if t is not None else None) for t in row_lse_layers])
    _check(lib().relaxkv_score_select(shape.ref(), n_layers, qs, caches, lses, _i32(k), _ptr(raw_scores_out),
                                      _ptr(norm_scores_out), _ptr(anchors_out), _ptr(workspace),
                                      ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)),
           "relaxkv_score_select")


def relaxkv_select_topk(shape: Shape, n_layers: int, k: Sequence[int], raw_scores: torch.Tensor,
                        anchors_out: torch.Tensor, norm_scores_out: Optional[torch.Tensor] = None,
                        stream=None) -> None:
    _check(lib().relaxkv_select_topk(shape.ref(), int(n_layers), _i32(k), _ptr(raw_scores), _ptr(norm_scores_out),
                                     _ptr(anchors_out), _stream(stream)), "relaxkv_select_topk")


def relaxkv_build_active_sets(shape: Shape, n_layers: int, k: Sequence[int], anchors: torch.Tensor,
                              highest_layer_out: torch.Tensor, u_pos_out: torch.Tensor, u_cu_out: torch.Tensor,
                              u_rank_out: torch.Tensor, r_rank_out: torch.Tensor, r_cu_out: torch.Tensor,
                              workspace: torch.Tensor, counts_pinned: Optional[torch.Tensor] = None,
                              stream=None) -> None:
    _check(lib().relaxkv_build_active_sets(shape.ref(), int(n_layers), _i32(k), _ptr(anchors),
                                           _ptr(highest_layer_out), _ptr(u_pos_out), _ptr(u_cu_out),
                                           _ptr(u_rank_out), _ptr(r_rank_out), _ptr(r_cu_out), _ptr(counts_pinned),
                                           _ptr(workspace),
                                           ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                           _stream(stream)),
           "relaxkv_build_active_sets")


def relaxkv_build_active_sets_static(shape: Shape, n_layers: int, k: Sequence[int], anchors: torch.Tensor,
                                     highest_layer_out: torch.Tensor, u_pos_out: torch.Tensor,
                                     u_cu_out: torch.Tensor, u_rank_out: torch.Tensor, r_rank_out: torch.Tensor,
                                     r_cu_out: torch.Tensor, counts_pinned: Optional[torch.Tensor] = None,
                                     stream=None) -> None:
    """Same outputs as relaxkv_build_active_sets, for callers that cannot supply a workspace: the
    scratch is a fixed array inside the library (at most 8192 counts: n_req * (1 + n_layers))."""
    _check(lib().relaxkv_build_active_sets_static(shape.ref(), int(n_layers), _i32(k), _ptr(anchors),
                                                  _ptr(highest_layer_out), _ptr(u_pos_out), _ptr(u_cu_out),
                                                  _ptr(u_rank_out), _ptr(r_rank_out), _ptr(r_cu_out),
                                                  _ptr(counts_pinned), _stream(stream)),
           "relaxkv_build_active_sets_static")


def _attention(fn_name, shape, mode, cache, q_new, k_new, v_new, u_pos, u_cu, r_rank, r_cu_layer, max_targets,
               max_ctx, out, lse_out, workspace, stream):
    fn = getattr(lib(), fn_name)
    _check(fn(shape.ref(), int(mode), cache.ref(), _ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(u_pos), _ptr(u_cu),
              _ptr(r_rank), _ptr(r_cu_layer), ctypes.c_int64(q_new.shape[0]), _i32(max_targets), _i32(max_ctx),
              _ptr(out), _ptr(lse_out), _ptr(workspace),
              ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)), fn_name)


def relaxkv_sparse_ctx_attention(shape: Shape, mode: int, cache: CacheView, q_new: torch.Tensor,
                                 k_new: Optional[torch.Tensor], v_new: Optional[torch.Tensor],
                                 u_pos: torch.Tensor, u_cu: torch.Tensor, r_rank: torch.Tensor,
                                 r_cu_layer: torch.Tensor, max_targets: Sequence[int], max_ctx: Sequence[int],
                                 out: torch.Tensor, workspace: torch.Tensor,
                                 lse_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """n_target_rows is q_new.shape[0]; k_new/v_new/out must have as many rows."""
    _attention("relaxkv_sparse_ctx_attention", shape, mode, cache, q_new, k_new, v_new, u_pos, u_cu, r_rank,
               r_cu_layer, max_targets, max_ctx, out, lse_out, workspace, stream)


def relaxkv_sparse_ctx_attention_simt(shape, mode, cache, q_new, k_new, v_new, u_pos, u_cu, r_rank, r_cu_layer,
                                      max_targets, max_ctx, out, workspace, lse_out=None, stream=None) -> None:
    _attention("relaxkv_sparse_ctx_attention_simt", shape, mode, cache, q_new, k_new, v_new, u_pos, u_cu, r_rank,
               r_cu_layer, max_targets, max_ctx, out, lse_out, workspace, stream)


def relaxkv_scatter_kv(shape: Shape, cache: CacheView, k_new: torch.Tensor, v_new: torch.Tensor,
                       u_pos: torch.Tensor, u_cu: torch.Tensor, r_rank: torch.Tensor, r_cu_layer: torch.Tensor,
                       max_targets: Sequence[int], stream=None) -> None:
    _check(lib().relaxkv_scatter_kv(shape.ref(), cache.ref(), _ptr(k_new), _ptr(v_new), _ptr(u_pos), _ptr(u_cu),
                                    _ptr(r_rank), _ptr(r_cu_layer), _i32(max_targets), _stream(stream)),
           "relaxkv_scatter_kv")


def relaxkv_gather_kv(shape: Shape, mode: int, cache: CacheView, k_new: Optional[torch.Tensor],
                      v_new: Optional[torch.Tensor], u_pos: torch.Tensor, u_cu: torch.Tensor, r_rank: torch.Tensor,
                      r_cu_layer: torch.Tensor, max_ctx: Sequence[int], k_ctx_out: torch.Tensor,
                      v_ctx_out: torch.Tensor, stream=None) -> None:
    _check(lib().relaxkv_gather_kv(shape.ref(), int(mode), cache.ref(), _ptr(k_new), _ptr(v_new), _ptr(u_pos),
                                   _ptr(u_cu), _ptr(r_rank), _ptr(r_cu_layer), _i32(max_ctx), _ptr(k_ctx_out),
                                   _ptr(v_ctx_out), ctypes.c_int64(k_ctx_out.shape[0]), _stream(stream)),
           "relaxkv_gather_kv")


def relaxkv_list_attention(shape: Shape, cache: CacheView, q_new: torch.Tensor, k_new: Optional[torch.Tensor],
                           v_new: Optional[torch.Tensor], ctx_pos: torch.Tensor, ctx_cu: torch.Tensor,
                           tgt_pos: torch.Tensor, tgt_cu: torch.Tensor, max_targets: Sequence[int],
                           max_ctx: Sequence[int], out: torch.Tensor, workspace: torch.Tensor,
                           lse_out: Optional[torch.Tensor] = None, stream=None) -> None:
    _check(lib().relaxkv_list_attention(shape.ref(), cache.ref(), _ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(ctx_pos),
                                        _ptr(ctx_cu), _ptr(tgt_pos), _ptr(tgt_cu), ctypes.c_int64(q_new.shape[0]),
                                        _i32(max_targets), _i32(max_ctx), _ptr(out), _ptr(lse_out), _ptr(workspace),
                                        ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)),
           "relaxkv_list_attention")


def relaxkv_cache_attention(shape: Shape, cache: CacheView, q_new: torch.Tensor, tgt_pos: torch.Tensor, tgt_cu: torch.Tensor,
                            max_targets: Sequence[int], out: torch.Tensor, workspace: torch.Tensor,
                            lse_out: Optional[torch.Tensor] = None, stream=None) -> None:
    _check(lib().relaxkv_cache_attention(shape.ref(), cache.ref(), _ptr(q_new), _ptr(tgt_pos), _ptr(tgt_cu),
                                         ctypes.c_int64(q_new.shape[0]), _i32(max_targets), _ptr(out), _ptr(lse_out),
                                         _ptr(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                         _stream(stream)),
           "relaxkv_cache_attention")


def relaxkv_query_prefill_attention(shape: Shape, cache: CacheView, q: torch.Tensor, out: torch.Tensor, lse_out: torch.Tensor,
                                    raw_scores_out: Optional[torch.Tensor], workspace: torch.Tensor, stream=None) -> None:
    """shape.ctx_lens = context tokens, shape.q_lens = query tokens; the cache holds both (context rows first)."""
    _check(lib().relaxkv_query_prefill_attention(shape.ref(), cache.ref(), _ptr(q), _ptr(out), _ptr(lse_out),
                                                 _ptr(raw_scores_out), _ptr(workspace),
                                                 ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                                 _stream(stream)),
           "relaxkv_query_prefill_attention")


def relaxkv_scatter_kv_lists(shape: Shape, cache: CacheView, k_new: torch.Tensor, v_new: torch.Tensor,
                             tgt_pos: torch.Tensor, tgt_cu: torch.Tensor, max_targets: Sequence[int], stream=None) -> None:
    _check(lib().relaxkv_scatter_kv_lists(shape.ref(), cache.ref(), _ptr(k_new), _ptr(v_new), _ptr(tgt_pos), _ptr(tgt_cu),
                                          _i32(max_targets), _stream(stream)), "relaxkv_scatter_kv_lists")


def relaxkv_mean_scores(shape: Shape, n_layers: int, scores: torch.Tensor, mean_out: torch.Tensor, stream=None) -> None:
    _check(lib().relaxkv_mean_scores(shape.ref(), int(n_layers), _ptr(scores), _ptr(mean_out), _stream(stream)),
           "relaxkv_mean_scores")


def relaxkv_scale_scores(shape: Shape, n_layers: int, scores: torch.Tensor, factor: float, stream=None) -> None:
    """scores *= factor in place (fp32 [n_layers, sum T_c] on the device)."""
    _check(lib().relaxkv_scale_scores(shape.ref(), int(n_layers), _ptr(scores), ctypes.c_float(factor), _stream(stream)),
           "relaxkv_scale_scores")


def relaxkv_rmsnorm(x: torch.Tensor, weight: torch.Tensor, y: torch.Tensor, eps: float, stream=None) -> None:
    _check(lib().relaxkv_rmsnorm(_ptr(x), _ptr(weight), _ptr(y), ctypes.c_int64(x.shape[0]), int(x.shape[1]),
                                 ctypes.c_float(eps), _stream(stream)), "relaxkv_rmsnorm")


def relaxkv_linear(x: torch.Tensor, weight: torch.Tensor, y: torch.Tensor, residual: Optional[torch.Tensor] = None,
                   stream=None) -> None:
    """y = x weight^T (+ residual); weight is [n_out, n_in]."""
    _check(lib().relaxkv_linear(_ptr(x), _ptr(weight), _ptr(residual), _ptr(y), ctypes.c_int64(x.shape[0]),
                                int(weight.shape[0]), int(weight.shape[1]), _stream(stream)), "relaxkv_linear")


def stack_qkv(wq: torch.Tensor, wk: torch.Tensor, wv: torch.Tensor) -> torch.Tensor:
    """[Wq; Wk; Wv] along the output features: the weight layout relaxkv_linear_qkv reads (a copy, made once when the
    weights are loaded)."""
    return torch.cat([wq, wk, wv], dim=0).contiguous()


def relaxkv_linear_qkv(x: torch.Tensor, w_qkv: torch.Tensor, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, stream=None) -> None:
    """q, k, v = x Wq^T, x Wk^T, x Wv^T with w_qkv = [Wq; Wk; Wv] stacked along the output features.
    q [n, n_q] (or any contiguous view of it), k and v [n, n_kv]."""
    n = x.shape[0]
    n_q, n_kv = q.numel() // max(n, 1), k.numel() // max(n, 1)
    assert w_qkv.shape[0] == n_q + 2 * n_kv and v.numel() == k.numel()
    _check(lib().relaxkv_linear_qkv(_ptr(x), _ptr(w_qkv), _ptr(q), _ptr(k), _ptr(v), ctypes.c_int64(n), int(n_q), int(n_kv),
                                    int(w_qkv.shape[1]), _stream(stream)), "relaxkv_linear_qkv")


def tile_gate_up(w_gate_up: torch.Tensor) -> torch.Tensor:
    """[Wg; Wu] of shape [2 * I, K] -> the row order relaxkv_linear_swiglu reads: per block of 128 features, its gate
    rows then its up rows.  A weight-loading step (done once), not part of the path."""
    two_i, k = w_gate_up.shape
    inter = two_i // 2
    assert inter % 128 == 0
    g = w_gate_up[:inter].view(inter // 128, 128, k)
    u = w_gate_up[inter:].view(inter // 128, 128, k)
    return torch.cat([g, u], dim=1).reshape(two_i, k).contiguous()


def relaxkv_linear_swiglu(x: torch.Tensor, weight_tiled: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    _check(lib().relaxkv_linear_swiglu(_ptr(x), _ptr(weight_tiled), _ptr(out), ctypes.c_int64(x.shape[0]),
                                       int(weight_tiled.shape[0] // 2), int(weight_tiled.shape[1]), _stream(stream)),
           "relaxkv_linear_swiglu")


def relaxkv_rope(x: torch.Tensor, positions: torch.Tensor, theta: float, stream=None) -> None:
    """In place on x [rows, heads, D]; positions int32 [rows]."""
    _check(lib().relaxkv_rope(_ptr(x), ctypes.c_int64(x.shape[0]), int(x.shape[1]), int(x.shape[2]), _ptr(positions),
                              ctypes.c_float(theta), _stream(stream)), "relaxkv_rope")


def relaxkv_qk_norm_rope(q: torch.Tensor, k: torch.Tensor, positions: torch.Tensor, theta: float,
                         w_q_norm: Optional[torch.Tensor] = None, w_k_norm: Optional[torch.Tensor] = None, eps: float = 1e-6,
                         stream=None) -> None:
    """Per-head RMSNorm (when weights are given) and rotary embedding of q [n, H, D] and k [n, H_kv, D], in place."""
    _check(lib().relaxkv_qk_norm_rope(_ptr(q), _ptr(k), ctypes.c_int64(q.shape[0]), int(q.shape[1]), int(k.shape[1]),
                                      int(q.shape[2]), _ptr(w_q_norm), _ptr(w_k_norm), ctypes.c_float(eps), _ptr(positions),
                                      ctypes.c_float(theta), _stream(stream)), "relaxkv_qk_norm_rope")


def relaxkv_swiglu(gate_up: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    _check(lib().relaxkv_swiglu(_ptr(gate_up), _ptr(out), ctypes.c_int64(gate_up.shape[0]), int(out.shape[1]),
                                _stream(stream)), "relaxkv_swiglu")


def relaxkv_target_positions(shape: Shape, u_pos, u_cu, r_rank, r_cu_layer, max_targets: Sequence[int],
                             positions_out: torch.Tensor, stream=None) -> None:
    _check(lib().relaxkv_target_positions(shape.ref(), _ptr(u_pos), _ptr(u_cu), _ptr(r_rank), _ptr(r_cu_layer),
                                          _i32(max_targets), _ptr(positions_out), _stream(stream)),
           "relaxkv_target_positions")


def relaxkv_carry_rows(shape: Shape, h_in: torch.Tensor, h_out: torch.Tensor, r_rank, r_cu_layer, r_cu_next,
                       max_next: Sequence[int], stream=None) -> None:
    _check(lib().relaxkv_carry_rows(shape.ref(), _ptr(h_in), _ptr(h_out), int(h_in.shape[1]), _ptr(r_rank),
                                    _ptr(r_cu_layer), _ptr(r_cu_next), _i32(max_next), _stream(stream)),
           "relaxkv_carry_rows")


def relaxkv_debug_wait_timeout(stream=None) -> None:
    """Launches the bounded-wait probe: ends after ~0.4 s with RELAXKV_ERR_TIMEOUT in the status word."""
    _check(lib().relaxkv_debug_wait_timeout(_stream(stream)), "relaxkv_debug_wait_timeout")


def relaxkv_read_device_status(stream=None):
    """Synchronises the stream; returns (status, [kernel id, block, v0, v1]) and clears the word."""
    st = ctypes.c_int32(0)
    detail = (ctypes.c_int32 * 4)()
    _check(lib().relaxkv_read_device_status(ctypes.byref(st), detail, _stream(stream)), "relaxkv_read_device_status")
    return int(st.value), list(detail)
