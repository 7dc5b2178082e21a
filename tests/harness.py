"""Shared test scaffolding: builds one synthetic case, runs the CPU oracle on it, and lays the same
bits out for the CUDA path.  The oracle never sees anything the CUDA path produced."""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np
import torch

from oracle import relaxkv_oracle as orc
from paper_2609_33503_b200 import inputs


@dataclasses.dataclass
class LayerFresh:
    q_new: torch.Tensor          # [sum_b |R_{l,b}|, H, D] bf16 (device), requests packed
    k_new: torch.Tensor
    v_new: torch.Tensor
    row_cu: List[int]            # request offsets into the packed rows


class Case:
    """Inputs + oracle results of one workload.  Everything per layer is packed over requests."""

    def __init__(self, w: inputs.Workload, device="cuda", gen_device=None, head_major_cache: bool = False,
                 score_layers: Optional[List[int]] = None, anchors_override=None):
        self.w = w
        self.device = torch.device(device)
        gen_device = gen_device or device
        self.scale = w.head_dim ** -0.5
        nb, L = w.n_req, w.n_layers
        self.ctx_cu = np.concatenate([[0], np.cumsum(w.ctx_lens)]).astype(np.int64)
        self.q_cu = np.concatenate([[0], np.cumsum(w.q_lens)]).astype(np.int64)
        self.q_layers, self.k_cache, self.v_cache = [], [], []
        for l in range(L):
            qs, ks, vs = zip(*[inputs.layer_qkv(w, l, b, gen_device) for b in range(nb)])
            q, k, v = torch.cat(qs).to(self.device), torch.cat(ks).to(self.device), torch.cat(vs).to(self.device)
            if head_major_cache:     # [H_kv, tokens, D] storage viewed as [tokens, H_kv, D]
                k = k.permute(1, 0, 2).contiguous().permute(1, 0, 2)
                v = v.permute(1, 0, 2).contiguous().permute(1, 0, 2)
            self.q_layers.append(q)
            self.k_cache.append(k)
            self.v_cache.append(v)
        self.k_bits = [inputs.bf16_bits(k) for k in self.k_cache]      # host copies, [sum_t, Hkv, D] contiguous
        self.v_bits = [inputs.bf16_bits(v) for v in self.v_cache]
        self.q_bits = [inputs.bf16_bits(q) for q in self.q_layers]
        self.k = [orc.anchor_count(t, w.ratio) for t in w.ctx_lens]
        self.k_cu = np.concatenate([[0], np.cumsum(self.k)]).astype(np.int64)
        # ---- oracle: scores, anchors, sets -------------------------------------------------------
        self.raw: Dict[tuple, np.ndarray] = {}
        self.anchors = [[None] * nb for _ in range(L)]
        layers = range(L) if score_layers is None else score_layers
        for l in range(L):
            for b in range(nb):
                if anchors_override is not None:
                    self.anchors[l][b] = np.asarray(anchors_override[l][b], dtype=np.int32)
                    continue
                assert l in layers
                raw = orc.raw_scores(self.req_q(l, b), self.req_k(l, b), self.scale)
                self.raw[(l, b)] = raw
                self.anchors[l][b] = orc.topk(raw, self.k[b])
        self.sets = [orc.active_sets(np.stack([self.anchors[l][b] for l in range(L)]), w.ctx_lens[b])
                     for b in range(nb)]
        # ---- fresh states of the active targets -------------------------------------------------
        self.fresh: List[LayerFresh] = []
        for l in range(L):
            qs, ks, vs, cu = [], [], [], [0]
            for b in range(nb):
                pos = torch.from_numpy(self.sets[b].positions(l).astype(np.int64))
                lo, hi = int(self.ctx_cu[b]), int(self.ctx_cu[b + 1])
                q, k, v = inputs.fresh_qkv(w, l, b, self.k_cache[l][lo:hi], self.v_cache[l][lo:hi], pos)
                qs.append(q); ks.append(k); vs.append(v)
                cu.append(cu[-1] + len(pos))
            self.fresh.append(LayerFresh(torch.cat(qs).contiguous(), torch.cat(ks).contiguous(),
                                         torch.cat(vs).contiguous(), cu))

    # per-request host views (bf16 bits)
    def req_q(self, l, b): return self.q_bits[l][self.q_cu[b]:self.q_cu[b + 1]]
    def req_k(self, l, b): return self.k_bits[l][self.ctx_cu[b]:self.ctx_cu[b + 1]]
    def req_v(self, l, b): return self.v_bits[l][self.ctx_cu[b]:self.ctx_cu[b + 1]]

    def fresh_bits(self, l, b):
        f = self.fresh[l]
        lo, hi = f.row_cu[b], f.row_cu[b + 1]
        return (inputs.bf16_bits(f.q_new[lo:hi]), inputs.bf16_bits(f.k_new[lo:hi]), inputs.bf16_bits(f.v_new[lo:hi]))

    def oracle_attention(self, l, b, full_prefix=False, rows=None, use_fresh_kv=True):
        qn, kn, vn = self.fresh_bits(l, b)
        s = self.sets[b]
        return orc.repair_attention(self.req_k(l, b), self.req_v(l, b), qn, kn if use_fresh_kv else None,
                                    vn if use_fresh_kv else None, s.u_pos, s.ranks(l), self.scale,
                                    full_prefix=full_prefix, rows=rows)

    def anchors_tensor(self) -> torch.Tensor:
        """[L, sum_k] int32 on the device, in the layout relaxkv_score_select writes."""
        a = np.stack([np.concatenate(self.anchors[l]) for l in range(self.w.n_layers)])
        return torch.from_numpy(a.astype(np.int32)).to(self.device)

    def make_session(self, want_norm=False):
        from paper_2609_33503_b200.pipeline import RepairSession
        w = self.w
        return RepairSession(w.n_q_heads, w.n_kv_heads, w.head_dim, w.ctx_lens, w.q_lens, w.n_layers, self.k,
                             device=self.device, softmax_scale=self.scale, want_norm=want_norm)

    def cache_views(self, k_list=None, v_list=None):
        from paper_2609_33503_b200 import binding as B
        k_list = k_list or self.k_cache
        v_list = v_list or self.v_cache
        return [B.CacheView(k, v, [int(x) for x in self.ctx_cu[:-1]]) for k, v in zip(k_list, v_list)]

    def max_targets(self, l): return [len(self.sets[b].ranks(l)) for b in range(self.w.n_req)]
    def max_ctx(self): return [len(self.sets[b].u_pos) for b in range(self.w.n_req)]


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def attention_errors(out_gpu: torch.Tensor, ref: np.ndarray):
    d = np.abs(bf16_to_f64(out_gpu) - ref)
    return float(d.max()) if d.size else 0.0, float(d.mean()) if d.size else 0.0


def check_anchor_band(raw_ref: np.ndarray, k: int, got: np.ndarray, rel: float = 1e-3):
    """Selected indices must contain every position clearly above the k-th score and none clearly
    below it; inside the tolerance band any choice is fine.  |got| = k, ascending, unique."""
    assert got.shape == (k,)
    assert np.all(np.diff(got) > 0)
    tau = np.sort(raw_ref)[::-1][k - 1]
    must = np.nonzero(raw_ref > tau * (1 + rel))[0]
    never = np.nonzero(raw_ref < tau * (1 - rel))[0]
    gs = set(got.tolist())
    assert set(must.tolist()) <= gs
    assert not (set(never.tolist()) & gs)
