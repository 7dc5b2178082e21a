"""Algorithm 1's selection + repair loop for callers whose inputs live in pinned HOST memory.

The per-layer fresh Q/K/V rows of the active targets travel host -> device through a small ring of
staging buffers on a copy-in stream, the kernels run on a compute stream, and every layer's repaired
attention output returns on a copy-out stream, so the PCIe transfers of layers l+1.. and l-1 run
under the kernels of layer l.  Call sequencing and buffer bookkeeping only: every step of the method
runs in the kernels behind `binding`; the KV cache itself stays resident on the device.
"""
from __future__ import annotations

from typing import List, Sequence

import torch

from . import binding as B
from .pipeline import RepairSession


class HostStreamedRepair:
    """Three-stream pipeline around a `RepairSession`.

    `max_rows` bounds the number of active-target rows of any one layer (sum over the requests of the
    batch); `depth` is the number of layers in flight between the copy engines and the kernels.
    """

    def __init__(self, session: RepairSession, max_rows: int, depth: int = 3):
        self.s = session
        self.depth = int(depth)
        sh = session.shape
        dev = session.device
        bf = dict(dtype=torch.bfloat16, device=dev)
        self.q_dev = None                      # query-row buffers, sized on first use
        self.ring_q = [torch.empty(max_rows, sh.c.n_q_heads, sh.c.head_dim, **bf) for _ in range(self.depth)]
        self.ring_k = [torch.empty(max_rows, sh.c.n_kv_heads, sh.c.head_dim, **bf) for _ in range(self.depth)]
        self.ring_v = [torch.empty(max_rows, sh.c.n_kv_heads, sh.c.head_dim, **bf) for _ in range(self.depth)]
        self.ring_o = [torch.empty(max_rows, sh.c.n_q_heads, sh.c.head_dim, **bf) for _ in range(self.depth)]
        self.max_rows = int(max_rows)
        self.s_in = torch.cuda.Stream(device=dev)
        self.s_run = torch.cuda.Stream(device=dev)
        self.s_out = torch.cuda.Stream(device=dev)
        self.h2d_bytes = 0
        self.d2h_bytes = 0

    def run(self, host_q_layers: Sequence[torch.Tensor], score_caches: List[B.CacheView],
            repair_caches: List[B.CacheView], host_fresh: Sequence[Sequence[torch.Tensor]],
            host_out: Sequence[torch.Tensor], mode: int = B.CTX_UNION):
        """host_q_layers[l]: the query suffix's Q rows of layer l; host_fresh[l] = (Q_new, K_new, V_new) rows of
        R_l in list order; host_out[l] receives the repaired attention output of layer l.  All pinned.
        Returns the (|U_b|, |R_{l,b}|) counts.  The caller's current stream waits for the whole pipeline."""
        s, L = self.s, self.s.n_layers
        cur = torch.cuda.current_stream(s.device)
        start = torch.cuda.Event()
        start.record(cur)
        self.h2d_bytes = self.d2h_bytes = 0
        if self.q_dev is None:
            self.q_dev = [torch.empty(q.shape, dtype=q.dtype, device=s.device) for q in host_q_layers]
        # 1. query rows in, selection and schedule on the compute stream
        self.s_in.wait_event(start)
        self.s_run.wait_event(start)
        self.s_out.wait_event(start)
        with torch.cuda.stream(self.s_in):
            for dst, src in zip(self.q_dev, host_q_layers):
                dst.copy_(src, non_blocking=True)
                self.h2d_bytes += src.numel() * src.element_size()
            q_ready = torch.cuda.Event()
            q_ready.record(self.s_in)
        with torch.cuda.stream(self.s_run):
            self.s_run.wait_event(q_ready)
            s.score_select(self.q_dev, score_caches)
            s.build_active_sets()
        n_u, n_r = s.counts()                   # host sync: the row counts of every layer
        # 2. layers: copy-in | attention + scatter | copy-out, `depth` layers in flight
        in_ready = [None] * L
        run_done = [None] * L
        out_done = [None] * L
        for l in range(L):
            slot = l % self.depth
            n = sum(n_r[l])
            if n > self.max_rows:
                raise B.RelaxKVError(B.ERR_INVALID_ARG, f"layer {l}: {n} target rows exceed the ring's {self.max_rows}")
            fq, fk, fv = host_fresh[l]
            if fq.shape[0] != n or fk.shape[0] != n or fv.shape[0] != n or host_out[l].shape[0] != n:
                raise B.RelaxKVError(B.ERR_INVALID_ARG, f"layer {l}: host buffers must hold exactly {n} rows")
            with torch.cuda.stream(self.s_in):
                if l >= self.depth:
                    self.s_in.wait_event(run_done[l - self.depth])      # the slot's last reader is done
                for ring, src in ((self.ring_q, fq), (self.ring_k, fk), (self.ring_v, fv)):
                    if n:
                        ring[slot][:n].copy_(src, non_blocking=True)
                    self.h2d_bytes += src.numel() * src.element_size()
                in_ready[l] = torch.cuda.Event()
                in_ready[l].record(self.s_in)
            with torch.cuda.stream(self.s_run):
                self.s_run.wait_event(in_ready[l])
                if l >= self.depth:
                    self.s_run.wait_event(out_done[l - self.depth])     # the slot's output has left
                if n:
                    s.attention(l, repair_caches[l], self.ring_q[slot][:n], self.ring_k[slot][:n], self.ring_v[slot][:n],
                                self.ring_o[slot][:n], n_r[l], n_u, mode=mode)
                    s.scatter(l, repair_caches[l], self.ring_k[slot][:n], self.ring_v[slot][:n], n_r[l])
                run_done[l] = torch.cuda.Event()
                run_done[l].record(self.s_run)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(run_done[l])
                if n:
                    host_out[l].copy_(self.ring_o[slot][:n], non_blocking=True)
                self.d2h_bytes += host_out[l].numel() * host_out[l].element_size()
                out_done[l] = torch.cuda.Event()
                out_done[l].record(self.s_out)
        for st in (self.s_in, self.s_run, self.s_out):
            e = torch.cuda.Event()
            e.record(st)
            cur.wait_event(e)
        return n_u, n_r
