"""Buffer bookkeeping around the C ABI: allocates the device arrays one repair request batch needs
and issues the calls in the order of Algorithm 1.  No arithmetic of the method happens here; every
step runs in the kernels behind `binding`.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as B


class RepairSession:
    """Device buffers for one batch of requests: scores, anchors, the repair schedule and the
    scratch workspace.  Sizes follow include/relaxkv.h."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, ctx_lens: Sequence[int],
                 q_lens: Sequence[int], n_layers: int, k: Sequence[int], device="cuda",
                 softmax_scale: Optional[float] = None, want_norm: bool = False):
        self.shape = B.Shape(n_q_heads, n_kv_heads, head_dim, ctx_lens, q_lens, softmax_scale)
        self.n_layers = int(n_layers)
        self.k = [int(x) for x in k]
        self.device = torch.device(device)
        nb = self.shape.n_req
        self.sum_t = sum(self.shape.ctx_lens)
        self.sum_k = sum(self.k)
        self.cap_u = sum(min(t, self.n_layers * kb) for t, kb in zip(self.shape.ctx_lens, self.k))
        i32 = dict(dtype=torch.int32, device=self.device)
        self.raw = torch.empty(self.n_layers, self.sum_t, dtype=torch.float32, device=self.device)
        self.norm = torch.empty_like(self.raw) if want_norm else None
        self.anchors = torch.empty(self.n_layers, self.sum_k, **i32)
        self.highest_layer = torch.empty(self.sum_t, **i32)
        self.u_pos = torch.empty(self.cap_u, **i32)
        self.u_cu = torch.empty(nb + 1, **i32)
        self.u_rank = torch.empty(self.sum_t, **i32)
        self.r_rank = torch.empty(self.n_layers * self.cap_u, **i32)
        self.r_cu = torch.empty(self.n_layers * nb + 1, **i32)
        self.counts_pinned = torch.empty(nb + self.n_layers * nb, dtype=torch.int32, pin_memory=True)
        ws = B.relaxkv_workspace_bytes(self.shape, self.n_layers, self.k)
        if ws == 0:
            raise B.RelaxKVError(B.ERR_INVALID_ARG, "relaxkv_workspace_bytes")
        self.workspace = torch.empty(ws + 256, dtype=torch.uint8, device=self.device)
        off = (-self.workspace.data_ptr()) % 256
        self.workspace = self.workspace[off:off + ws]
        self._counts = None

    # -- (a) selection --------------------------------------------------------------------------
    def score_select(self, q_layers: List[torch.Tensor], cache_layers: List[B.CacheView],
                     row_lse_layers=None, stream=None) -> None:
        B.relaxkv_score_select(self.shape, q_layers, cache_layers, self.k, self.raw, self.anchors, self.workspace,
                               norm_scores_out=self.norm, row_lse_layers=row_lse_layers, stream=stream)

    def build_active_sets(self, anchors: Optional[torch.Tensor] = None, stream=None) -> None:
        B.relaxkv_build_active_sets(self.shape, self.n_layers, self.k, self.anchors if anchors is None else anchors,
                                    self.highest_layer, self.u_pos, self.u_cu, self.u_rank, self.r_rank, self.r_cu,
                                    self.workspace, counts_pinned=self.counts_pinned, stream=stream)
        self._counts = None

    def counts(self):
        """(|U_b| per request, |R_{l,b}| as [n_layers][n_req]) - synchronises the device."""
        if self._counts is None:
            torch.cuda.synchronize(self.device)
            nb = self.shape.n_req
            c = self.counts_pinned.tolist()
            self._counts = (c[:nb], [c[nb + l * nb: nb + (l + 1) * nb] for l in range(self.n_layers)])
        return self._counts

    def r_cu_layer(self, layer: int) -> torch.Tensor:
        nb = self.shape.n_req
        return self.r_cu[layer * nb: layer * nb + nb + 1]

    # -- (b) repair -----------------------------------------------------------------------------
    def attention(self, layer: int, cache: B.CacheView, q_new, k_new, v_new, out, max_targets, max_ctx,
                  mode: int = B.CTX_UNION, lse_out=None, stream=None, simt: bool = False) -> None:
        fn = B.relaxkv_sparse_ctx_attention_simt if simt else B.relaxkv_sparse_ctx_attention
        fn(self.shape, mode, cache, q_new, k_new, v_new, self.u_pos, self.u_cu, self.r_rank,
           self.r_cu_layer(layer), max_targets, max_ctx, out, self.workspace, lse_out=lse_out, stream=stream)

    def scatter(self, layer: int, cache: B.CacheView, k_new, v_new, max_targets, stream=None) -> None:
        B.relaxkv_scatter_kv(self.shape, cache, k_new, v_new, self.u_pos, self.u_cu, self.r_rank,
                             self.r_cu_layer(layer), max_targets, stream=stream)

    def gather(self, layer: int, cache: B.CacheView, k_new, v_new, max_ctx, k_ctx_out, v_ctx_out,
               mode: int = B.CTX_UNION, stream=None) -> None:
        B.relaxkv_gather_kv(self.shape, mode, cache, k_new, v_new, self.u_pos, self.u_cu, self.r_rank,
                            self.r_cu_layer(layer), max_ctx, k_ctx_out, v_ctx_out, stream=stream)
