"""The user query's own forward pass and the first decode step over the context cache: what surrounds the repair
loop in the paper's time-to-first-token region (Section 2: the scores come from a pass of the query over the naive
cache, one attention per layer; reproducibility appendix: query prefill and the first token's decode close the timed
region).  Call sequencing over torch buffers only; every operation runs in the CUDA kernels behind
`binding`.

Per layer the query's rows run the decoder block: RMSNorm, the stacked Q/K/V projection, per-head Q/K norm where the
model has one and rotary embedding at positions T_c, T_c + 1, ... (one launch), their K/V are appended to the cache behind the context rows,
then causal attention over [context, query] (`relaxkv_query_prefill_attention`, which can emit the context scores of
that very pass), output projection + residual, MLP + residual.  The decode step is the same block for one new token
(the projections take the streaming one-row kernel), followed by the final norm and the output head.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import torch

from . import binding as B
from .inputs import BlockShape


class QueryPass:
    """Buffers for the block work of the query rows of a batch (`q_lens` tokens per request after `ctx_lens` context
    tokens).  The caches handed to `prefill` / `decode` must have room for ctx + query (+ decoded) tokens per request."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, ctx_lens: Sequence[int], q_lens: Sequence[int],
                 blk: BlockShape, device="cuda", softmax_scale: Optional[float] = None, extra_tokens: int = 1):
        self.blk = blk
        self.ctx_lens, self.q_lens = [int(x) for x in ctx_lens], [int(x) for x in q_lens]
        self.device = torch.device(device)
        H, Hkv, D, C, I = n_q_heads, n_kv_heads, head_dim, blk.hidden, blk.inter
        self.H, self.Hkv, self.D = H, Hkv, D
        nb = len(self.ctx_lens)
        n = sum(self.q_lens)
        bf = dict(dtype=torch.bfloat16, device=self.device)
        i32 = dict(dtype=torch.int32, device=self.device)
        # shapes: context + query (prefill), and + the decoded tokens so far (decode)
        self.shape_prefill = B.Shape(H, Hkv, D, self.ctx_lens, self.q_lens, softmax_scale)
        ext = [c + q for c, q in zip(self.ctx_lens, self.q_lens)]
        self.shape_ext = B.Shape(H, Hkv, D, ext, self.q_lens, softmax_scale)
        self.shape_dec = B.Shape(H, Hkv, D, [e + extra_tokens for e in ext], [1] * nb, softmax_scale)
        nbytes = max(B.relaxkv_workspace_bytes(self.shape_ext, 1), B.relaxkv_workspace_bytes(self.shape_dec, 1))
        ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        off = (-ws.data_ptr()) % 256
        self.workspace = ws[off:off + nbytes]
        e = lambda *s: torch.empty(*s, **bf)
        self.x, self.a, self.h = e(n, C), e(n, C), [e(n, C), e(n, C)]
        self.q, self.k, self.v, self.o = e(n, H, D), e(n, Hkv, D), e(n, Hkv, D), e(n, H, D)
        self.gu, self.m = e(n, 2 * I), e(n, I)
        self.lse = torch.empty(H, n, dtype=torch.float32, device=self.device)
        # positions of the query tokens (request-local) and their offsets: plain index data, built once
        pos, cu = [], [0]
        for c, q in zip(self.ctx_lens, self.q_lens):
            pos.append(torch.arange(c, c + q, dtype=torch.int32))
            cu.append(cu[-1] + q)
        self.q_pos = torch.cat(pos).to(self.device)
        self.q_cu = torch.tensor(cu, **i32)
        self.last_rows = torch.tensor([c - 1 for c in cu[1:]], dtype=torch.long, device=self.device)
        # decode buffers: one row per request
        self.dx, self.da, self.dh = e(nb, C), e(nb, C), [e(nb, C), e(nb, C)]
        self.dq, self.dk, self.dv, self.do = e(nb, H, D), e(nb, Hkv, D), e(nb, Hkv, D), e(nb, H, D)
        self.dgu, self.dm = e(nb, 2 * I), e(nb, I)
        self.d_cu = torch.arange(nb + 1, **i32)
        self._dec_pos = {}

    def decode_positions(self, step: int) -> torch.Tensor:
        """Device tensor of the decoded token's position per request (T_c + Q_b + step), built once per step index so
        that `decode` itself performs no host-to-device copy (it can then be captured into a CUDA graph)."""
        if step not in self._dec_pos:
            self._dec_pos[step] = torch.tensor([c + q + step for c, q in zip(self.ctx_lens, self.q_lens)],
                                               dtype=torch.int32, device=self.device)
        return self._dec_pos[step]

    def _block(self, l, w, cache, h, x, a, q, k, v, o, gu, m, h_out, pos, cu, counts, shape, attend, rec):
        blk, D, n = self.blk, self.D, h.shape[0]
        rec("norm", lambda: B.relaxkv_rmsnorm(h, w["w_in_norm"], x, blk.eps))
        if "w_qkv" not in w:                            # weight-loading step, once per layer: [Wq; Wk; Wv] stacked
            w["w_qkv"] = B.stack_qkv(w["wq"], w["wk"], w["wv"])
        rec("qkv_proj", lambda: B.relaxkv_linear_qkv(x, w["w_qkv"], q.view(n, -1), k.view(n, -1), v.view(n, -1)))
        rec("rope", lambda: B.relaxkv_qk_norm_rope(q, k, pos, blk.rope_theta, w.get("w_q_norm"), w.get("w_k_norm"), blk.eps))
        rec("append_kv", lambda: B.relaxkv_scatter_kv_lists(shape, cache, k, v, pos, cu, counts))
        rec("attention", attend)
        rec("o_proj", lambda: B.relaxkv_linear(o.view(n, -1), w["wo"], a, residual=h))
        rec("norm", lambda: B.relaxkv_rmsnorm(a, w["w_post_norm"], x, blk.eps))
        if blk.inter % 128 == 0:
            if "w_gate_up_tiled" not in w:              # weight-loading step, once per layer
                w["w_gate_up_tiled"] = B.tile_gate_up(w["w_gate_up"])
            rec("mlp", lambda: B.relaxkv_linear_swiglu(x, w["w_gate_up_tiled"], m))
        else:
            rec("mlp", lambda: (B.relaxkv_linear(x, w["w_gate_up"], gu), B.relaxkv_swiglu(gu, m)))
        rec("mlp", lambda: B.relaxkv_linear(m, w["w_down"], h_out, residual=a))

    @staticmethod
    def _rec(events):
        def rec(name, fn):
            if events is None:
                fn(); return
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record(); events.append((name, a, b))
        return rec

    def prefill(self, h0: torch.Tensor, weights: List[Dict[str, torch.Tensor]], caches: List[B.CacheView],
                scores_out: Optional[torch.Tensor] = None, events: Optional[list] = None,
                taps: Optional[list] = None) -> torch.Tensor:
        """h0: input representations of the query tokens [sum Q_b, hidden].  caches[l]: layer l's cache with the context
        rows in place and room behind them; the query's K/V are written there.  scores_out: fp32 [n_layers, sum T_c]
        or None; when given, row l receives the context scores of layer l from this very pass.  Returns the hidden rows
        after the last layer."""
        rec = self._rec(events)
        h = h0
        for l, w in enumerate(weights):
            h_out = self.h[l % 2]
            raw = scores_out[l] if scores_out is not None else None

            def attend():
                B.relaxkv_query_prefill_attention(self.shape_prefill, caches[l], self.q, self.o, self.lse, raw, self.workspace)
            self._block(l, w, caches[l], h, self.x, self.a, self.q, self.k, self.v, self.o, self.gu, self.m, h_out,
                        self.q_pos, self.q_cu, self.q_lens, self.shape_ext, attend, rec)
            if taps is not None:
                taps.append((h.clone(), h_out.clone()))
            h = h_out
        return h

    def decode(self, h_tok: torch.Tensor, weights: List[Dict[str, torch.Tensor]], caches: List[B.CacheView], step: int = 0,
               events: Optional[list] = None) -> torch.Tensor:
        """One decode step: h_tok [n_req, hidden] = the new token's input representation per request; its position is
        T_c + Q_b + step.  Appends its K/V to the caches and returns the hidden row after the last layer."""
        rec = self._rec(events)
        nb = len(self.ctx_lens)
        pos = self.decode_positions(step)
        h = h_tok
        for l, w in enumerate(weights):
            h_out = self.dh[l % 2]

            def attend():
                B.relaxkv_cache_attention(self.shape_dec, caches[l], self.dq, pos, self.d_cu, [1] * nb, self.do, self.workspace)
            self._block(l, w, caches[l], h, self.dx, self.da, self.dq, self.dk, self.dv, self.do, self.dgu, self.dm, h_out,
                        pos, self.d_cu, [1] * nb, self.shape_dec, attend, rec)
            h = h_out
        return h

    def output_head(self, h: torch.Tensor, final_norm: torch.Tensor, w_head: torch.Tensor, logits: torch.Tensor,
                    rows: Optional[torch.Tensor] = None, events: Optional[list] = None) -> torch.Tensor:
        """Final RMSNorm and the output projection of one row per request (by default the last query token's):
        logits [n_req, vocab]."""
        rec = self._rec(events)
        nb = len(self.ctx_lens)
        last = h if h.shape[0] == nb else h.index_select(0, self.last_rows if rows is None else rows)
        rec("head", lambda: (B.relaxkv_rmsnorm(last, final_norm, self.dx, self.blk.eps),
                             B.relaxkv_linear(self.dx, w_head, logits)))
        return logits
