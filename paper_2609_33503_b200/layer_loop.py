"""The repair loop of Algorithm 1 (steps 13-22) with the dense block work included: for every layer the
active targets run the whole decoder block - RMSNorm, Q/K/V projections, the per-head Q/K norm where the
model has one, rotary embedding at their original
positions, sparse-context repair attention, cache update, output projection, MLP - and the hidden rows of
the targets that stay active are carried to the next layer.  This module only sequences calls of the C ABI
(`binding`) over torch buffers; every operation runs in the CUDA kernels.
"""
from __future__ import annotations

from typing import Dict, List, Optional

import torch

from . import binding as B
from .inputs import BlockShape
from .pipeline import RepairSession


class LayerLoop:
    """Buffers for the block work of up to `max_rows` active rows (|U| summed over the batch)."""

    def __init__(self, session: RepairSession, blk: BlockShape, max_rows: int):
        self.s, self.blk = session, blk
        sh = session.shape.c
        H, Hkv, D, C, I = sh.n_q_heads, sh.n_kv_heads, sh.head_dim, blk.hidden, blk.inter
        dev, bf = session.device, torch.bfloat16
        n = max(1, int(max_rows))
        e = lambda *shape: torch.empty(*shape, dtype=bf, device=dev)
        self.x, self.a, self.h_next = e(n, C), e(n, C), e(n, C)
        self.h_carry = [e(n, C), e(n, C)]            # layer inputs after the carry, ping-pong
        self.q, self.k, self.v, self.o = e(n, H, D), e(n, Hkv, D), e(n, Hkv, D), e(n, H, D)
        self.gu, self.m = e(n, 2 * I), e(n, I)
        self.pos = torch.empty(n, dtype=torch.int32, device=dev)

    def run(self, h: torch.Tensor, weights: List[Dict[str, torch.Tensor]], caches: List[B.CacheView],
            events: Optional[list] = None, taps: Optional[list] = None) -> torch.Tensor:
        """h: hidden rows of R_0 = U (requests packed) [sum |U_b|, hidden].  Returns the hidden rows of the
        last layer's targets after that layer.  The caches are repaired in place.  `taps` (a list) receives a
        copy of every layer's (input rows, output rows), for checks that look at one layer at a time."""
        s, blk = self.s, self.blk
        n_u, n_r = s.counts()
        L = s.n_layers
        D = s.shape.c.head_dim

        def rec(name, fn):
            if events is None:
                fn(); return
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record(); events.append((name, a, b))

        for l in range(L):
            w = weights[l]
            n = sum(n_r[l])
            if n == 0:
                break
            x, a, q, k, v, o = self.x[:n], self.a[:n], self.q[:n], self.k[:n], self.v[:n], self.o[:n]
            gu, m, pos = self.gu[:n], self.m[:n], self.pos[:n]
            rec("norm", lambda: B.relaxkv_rmsnorm(h, w["w_in_norm"], x, blk.eps))
            if "w_qkv" not in w:                            # weight-loading step, once per layer: [Wq; Wk; Wv] stacked
                w["w_qkv"] = B.stack_qkv(w["wq"], w["wk"], w["wv"])
            rec("qkv_proj", lambda: B.relaxkv_linear_qkv(x, w["w_qkv"], q.view(n, -1), k.view(n, -1), v.view(n, -1)))
            # per-head RMSNorm of the projected queries and keys (models that have one) and the rotary embedding at the
            # targets' original positions: one pass over q and k
            rec("rope", lambda: (B.relaxkv_target_positions(s.shape, s.u_pos, s.u_cu, s.r_rank, s.r_cu_layer(l), n_r[l], pos),
                                 B.relaxkv_qk_norm_rope(q, k, pos, blk.rope_theta, w.get("w_q_norm"), w.get("w_k_norm"), blk.eps)))
            rec("attention", lambda: s.attention(l, caches[l], q, k, v, o, n_r[l], n_u))
            rec("scatter", lambda: s.scatter(l, caches[l], k, v, n_r[l]))
            rec("o_proj", lambda: B.relaxkv_linear(o.view(n, -1), w["wo"], a, residual=h))
            rec("norm", lambda: B.relaxkv_rmsnorm(a, w["w_post_norm"], x, blk.eps))
            if blk.inter % 128 == 0:
                if "w_gate_up_tiled" not in w:          # weight-loading step, once per layer
                    w["w_gate_up_tiled"] = B.tile_gate_up(w["w_gate_up"])
                rec("mlp", lambda: B.relaxkv_linear_swiglu(x, w["w_gate_up_tiled"], m))
            else:
                rec("mlp", lambda: (B.relaxkv_linear(x, w["w_gate_up"], gu), B.relaxkv_swiglu(gu, m)))
            h_out = self.h_next[:n]
            rec("mlp", lambda: B.relaxkv_linear(m, w["w_down"], h_out, residual=a))
            if taps is not None:
                taps.append((h[:n].clone(), h_out.clone()))
            if l + 1 < L:
                n_next = sum(n_r[l + 1])
                carried = self.h_carry[l % 2][:n_next]
                if n_next:
                    rec("carry", lambda: B.relaxkv_carry_rows(s.shape, h_out, carried, s.r_rank, s.r_cu_layer(l),
                                                              s.r_cu_layer(l + 1), n_r[l + 1]))
                h = carried
            else:
                h = h_out
        return h
