"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds input recipes only: random Q/K/V tensors, the planted "relevant
chunk" structure and the perturbation that stands for freshly recomputed K/V. It
contains none of the method's arithmetic (no scores, no top-k, no sets, no
attention) and is the only module shared by the CPU oracle's tests and the CUDA
path's tests and benchmark.  Both sides always consume the *same* bf16 bit
patterns: tensors are generated once (on whichever device is asked for) and the
oracle receives a host copy of those bits.

Workload shapes follow the paper's evaluation set-up (Section 4.1 and the
reproducibility appendix): 512-token chunks, decoder models with grouped-query
attention (Llama-3.1-8B: 32 query / 8 KV heads; Qwen3-14B: 40 / 8; head_dim
128), contexts of 8K-32K tokens (up to 64K in the ragged batch), anchor ratios
5-30 % with 15 % as the default.  The paper's benchmark suites and model
weights are not used; these tensors stand in for them.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence, Tuple

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic repair workload (a batch of independent requests)."""

    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    chunk: int
    ctx_lens: Tuple[int, ...]            # T_c per request
    q_lens: Tuple[int, ...]              # query-suffix length per request
    ratio: float                         # anchor ratio r
    base_seed: int = 0
    planted_chunks: Tuple[Tuple[int, ...], ...] = ()   # per request, 0-based chunk ids
    # "literal": only the planted chunks are shared across layers.
    # "calibrated": in addition a per-request warm set of tokens is shifted (see
    # `shift_mask`) so that |U|/T_c and the active-target ratio land near the
    # ratios the paper reports for its 32K runs (Appendix, full-prefix control).
    variant: str = "literal"
    warm_frac: float = 0.78
    warm_seed: int = 12345
    shift: float = 0.5
    fresh_std: float = 0.1

    @property
    def n_req(self) -> int:
        return len(self.ctx_lens)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def layer_seed(w: Workload, layer: int, req: int) -> int:
    return w.base_seed + 1000 * req + layer


def shift_mask(w: Workload, layer: int, req: int) -> torch.Tensor:
    """Boolean [T_c] mask (CPU) of the context tokens whose keys are shifted
    towards the query direction at this layer.

    Planted chunks are shifted at every layer.  In the "calibrated" variant a
    Bernoulli(warm_frac) subset W of the other tokens (fixed per request) is
    shifted too; a random half of W is shifted only in the first half of the
    layers, which gives tokens whose highest selected layer is mid-stack.
    """
    T = w.ctx_lens[req]
    m = torch.zeros(T, dtype=torch.bool)
    for c in (w.planted_chunks[req] if w.planted_chunks else ()):
        m[c * w.chunk:(c + 1) * w.chunk] = True
    if w.variant == "calibrated":
        g = _gen("cpu", w.warm_seed + req)
        warm = torch.rand(T, generator=g) < w.warm_frac
        early_only = torch.rand(T, generator=g) < 0.5
        warm &= ~m
        if layer >= w.n_layers // 2:
            warm &= ~early_only
        m |= warm
    elif w.variant != "literal":
        raise ValueError(f"unknown variant {w.variant!r}")
    return m


def layer_qkv(w: Workload, layer: int, req: int, device="cpu"):
    """Query-suffix Q [Q, H, D] and cached K, V [T_c, H_kv, D] for one layer of one
    request, bf16 on `device`.

    Q, K, V ~ N(0,1) in fp32.  For KV head g, u_g is the unit vector of the mean
    of the G*Q query rows that read head g; shifted tokens (see `shift_mask`) get
    K[i, g, :] += shift * sqrt(D) * u_g.  Everything is then cast to bf16.
    """
    T, Qn = w.ctx_lens[req], w.q_lens[req]
    H, Hkv, D, G = w.n_q_heads, w.n_kv_heads, w.head_dim, w.group
    g = _gen(device, layer_seed(w, layer, req))
    q = torch.randn(Qn, H, D, generator=g, device=device, dtype=torch.float32)
    k = torch.randn(T, Hkv, D, generator=g, device=device, dtype=torch.float32)
    v = torch.randn(T, Hkv, D, generator=g, device=device, dtype=torch.float32)
    mask = shift_mask(w, layer, req).to(device)
    if bool(mask.any()):
        qm = q.view(Qn, Hkv, G, D).mean(dim=(0, 2))                 # [Hkv, D]
        u = qm / qm.norm(dim=-1, keepdim=True).clamp_min(1e-20)
        k[mask] += (w.shift * math.sqrt(D)) * u.unsqueeze(0)
    return q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)


def fresh_qkv(w: Workload, layer: int, req: int, k_cache: torch.Tensor, v_cache: torch.Tensor,
              positions: torch.Tensor):
    """Stand-in for the recomputed states of the active targets at `positions`
    (ascending int positions, request-local): Q_new [n, H, D] ~ N(0,1) and
    K_new/V_new [n, H_kv, D] = cached + N(0, fresh_std^2), added in fp32 and cast
    to bf16.  The noise of a position does not depend on which other positions
    are asked for.
    """
    device = k_cache.device
    T = w.ctx_lens[req]
    H, Hkv, D = w.n_q_heads, w.n_kv_heads, w.head_dim
    g = _gen(device, layer_seed(w, layer, req) + 500_000)
    pos = positions.to(device=device, dtype=torch.long)
    nk = torch.randn(T, Hkv, D, generator=g, device=device, dtype=torch.float32)
    k_new = (k_cache[pos].float() + w.fresh_std * nk[pos]).to(torch.bfloat16)
    del nk
    nv = torch.randn(T, Hkv, D, generator=g, device=device, dtype=torch.float32)
    v_new = (v_cache[pos].float() + w.fresh_std * nv[pos]).to(torch.bfloat16)
    del nv
    qa = torch.randn(T, H, D, generator=g, device=device, dtype=torch.float32)
    q_new = qa[pos].to(torch.bfloat16)
    del qa
    return q_new, k_new, v_new


def bf16_bits(t: torch.Tensor):
    """Host numpy uint16 view of a bf16 tensor's bit patterns (what the oracle reads)."""
    import numpy as np
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


# ----------------------------------------------------------------------------
# Named workloads
# ----------------------------------------------------------------------------

def tiny() -> Workload:
    """1 layer, 4 query / 1 KV head, D=64, 1024 context tokens as 4 chunks of 256,
    32 query tokens, r = 15 %; chunk index 2 planted."""
    return Workload("tiny", 1, 4, 1, 64, 256, (1024,), (32,), 0.15, base_seed=0,
                    planted_chunks=((2,),))


def llama8b_16k() -> Workload:
    """Llama-3.1-8B-shaped single layer: 32/8 heads, D=128, 16K context as 32 chunks
    of 512, 64 query tokens, r = 15 %, three planted chunks."""
    return Workload("llama8b_16k", 1, 32, 8, 128, 512, (16384,), (64,), 0.15, base_seed=0,
                    planted_chunks=((5, 14, 27),))


def llama8b_stack(ctx_len: int = 8192, n_layers: int = 32, q_len: int = 64) -> Workload:
    """Llama-3.1-8B-shaped full stack (32 layers, 32/8 heads, D=128) on one context built from 512-token chunks -
    the model and context class of the paper's global repair target sweep; three planted chunks, calibrated variant."""
    n_chunks = max(3, ctx_len // 512)
    planted = tuple(sorted({n_chunks // 6, n_chunks // 2, (5 * n_chunks) // 6}))
    return Workload(f"llama8b_{ctx_len // 1024}k_stack", n_layers, 32, 8, 128, 512, (ctx_len,), (q_len,), 0.15, base_seed=0,
                    planted_chunks=(planted,), variant="calibrated")


def qwen14b_32k(variant: str = "calibrated", ratio: float = 0.15, n_layers: int = 40) -> Workload:
    """Qwen3-14B-shaped stack: 40 layers, 40/8 heads, D=128, 32K context as 64 chunks
    of 512, 128 query tokens; per-layer tensors seeded by the layer id."""
    return Workload(f"qwen14b_32k_{variant}", n_layers, 40, 8, 128, 512, (32768,), (128,), ratio,
                    base_seed=0, planted_chunks=((9, 30, 52),), variant=variant)


RAGGED_CTX = (8192, 12288, 16384, 24576, 32768, 40960, 49152, 65536)


def ragged8(n_layers: int = 40) -> Workload:
    """Eight Qwen3-14B-shaped requests with 8K..64K contexts built from 512-token
    chunks, query lengths uniform in 32..256 (numpy PCG64, seed 5), r = 15 %."""
    import numpy as np
    rng = np.random.Generator(np.random.PCG64(5))
    q_lens = tuple(int(x) for x in rng.integers(32, 257, size=len(RAGGED_CTX)))
    planted = []
    for b, T in enumerate(RAGGED_CTX):
        n_chunks = T // 512
        cr = np.random.Generator(np.random.PCG64(100 + b))
        planted.append(tuple(sorted(int(c) for c in cr.choice(n_chunks, size=3, replace=False))))
    return Workload("ragged8", n_layers, 40, 8, 128, 512, RAGGED_CTX, q_lens, 0.15, base_seed=0,
                    planted_chunks=tuple(planted), variant="calibrated")


def scaled_down(w: Workload, ctx_lens: Sequence[int], q_lens: Optional[Sequence[int]] = None,
                n_layers: Optional[int] = None, chunk: Optional[int] = None) -> Workload:
    """Same head geometry and recipe at smaller sizes (parity-test cases the oracle
    finishes in seconds).  Planted chunks are re-drawn inside the shorter context."""
    chunk = chunk or w.chunk
    planted = []
    for b, T in enumerate(ctx_lens):
        n_chunks = max(1, T // chunk)
        ids = sorted({(3 * b + 1) % n_chunks, (n_chunks * 2) // 3})
        planted.append(tuple(ids))
    return w.replace(name=w.name + "_small", ctx_lens=tuple(int(t) for t in ctx_lens),
                     q_lens=tuple(int(x) for x in (q_lens or w.q_lens[:len(ctx_lens)])),
                     n_layers=n_layers or w.n_layers, chunk=chunk, planted_chunks=tuple(planted))


NAMED: Dict[str, object] = {
    "tiny": tiny,
    "llama8b_16k": llama8b_16k,
    "qwen14b_32k": qwen14b_32k,
    "llama8b_stack": llama8b_stack,
    "ragged8": ragged8,
}


# ----------------------------------------------------------------------------
# Synthetic decoder-block weights (the paper's models are not here)
# ----------------------------------------------------------------------------

@dataclasses.dataclass(frozen=True)
class BlockShape:
    """Llama-style pre-norm decoder block: hidden size, SwiGLU width, rotary base, RMSNorm epsilon; `qk_norm`
    adds the per-head RMSNorm of the projected queries and keys (Qwen3)."""
    hidden: int
    inter: int
    rope_theta: float = 1.0e6
    eps: float = 1.0e-6
    qk_norm: bool = False


QWEN3_14B_BLOCK = BlockShape(hidden=5120, inter=17408, qk_norm=True)
LLAMA31_8B_BLOCK = BlockShape(hidden=4096, inter=14336, rope_theta=5.0e5, eps=1.0e-5)


def block_weights(w: Workload, blk: BlockShape, layer: int, device="cpu") -> Dict[str, torch.Tensor]:
    """Random-init weights of one block, bf16: projections ~ N(0, 1/fan_in) in the [out, in] layout, norm gains
    ~ 1 + 0.1 N(0,1).  `w_gate_up` stacks the gate rows on top of the up rows."""
    g = _gen(device, 7_000_000 + w.base_seed + layer)
    C, H, Hkv, D, I = blk.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, blk.inter

    def lin(n_out, n_in):
        return (torch.randn(n_out, n_in, generator=g, device=device, dtype=torch.float32) * n_in ** -0.5).to(torch.bfloat16)

    def gain(n):
        return (1.0 + 0.1 * torch.randn(n, generator=g, device=device, dtype=torch.float32)).to(torch.bfloat16)

    out = {"w_in_norm": gain(C), "wq": lin(H * D, C), "wk": lin(Hkv * D, C), "wv": lin(Hkv * D, C), "wo": lin(C, H * D),
           "w_post_norm": gain(C), "w_gate_up": lin(2 * I, C), "w_down": lin(C, I)}
    if blk.qk_norm:
        out["w_q_norm"], out["w_k_norm"] = gain(D), gain(D)
    return out


def input_representations(w: Workload, blk: BlockShape, req: int, positions: torch.Tensor, device="cpu") -> torch.Tensor:
    """Stand-in for the input embeddings of the tokens at `positions` (Algorithm 1, step 14): N(0,1) rows,
    a pure function of (request, position)."""
    g = _gen(device, 9_000_000 + w.base_seed + req)
    table = torch.randn(w.ctx_lens[req], blk.hidden, generator=g, device=device, dtype=torch.float32)
    return table[positions.to(device=device, dtype=torch.long)].to(torch.bfloat16)
