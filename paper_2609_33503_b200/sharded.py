"""KV-head-sharded serving layout (tensor parallel over KV heads): plumbing only.

Each rank holds H_kv / N KV heads of the cache and the G query heads of each.  Scoring produces a
partial score over the local heads; the ranks' partial scores are combined by ONE all-reduce of a
[sum T_c] fp32 vector per layer (the only exchange on the path); selection and the repair schedule are
then computed redundantly and deterministically on every rank, and gather / attention / scatter are
local to the rank's heads.  Section 3.2's score is a mean over all H heads: with equal shards it is the
mean over ranks of the local means.

Everything here goes through `binding` (CUDA) and `torch.distributed`; nothing is computed in Python.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch


def head_shard(n_q_heads: int, n_kv_heads: int, world: int, rank: int) -> Tuple[int, int, int, int]:
    """(kv_lo, kv_hi, q_lo, q_hi): the KV heads and query heads rank `rank` of `world` owns.
    KV heads are split evenly (world must divide n_kv_heads); a KV head's whole query group goes with it."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad world/rank")
    if n_kv_heads % world != 0 or n_q_heads % n_kv_heads != 0:
        raise ValueError(f"{world} ranks do not divide {n_kv_heads} KV heads evenly")
    per = n_kv_heads // world
    g = n_q_heads // n_kv_heads
    return rank * per, (rank + 1) * per, rank * per * g, (rank + 1) * per * g


def combine_partial_scores(session, world: int, group=None, stream=None, scale_fn=None) -> torch.Tensor:
    """In place on session.raw: mean over ranks of the local (per-shard mean) scores = the score over all heads.
    One all-reduce(sum) of the [n_layers, sum T_c] fp32 tensor followed by the library's scaling kernel
    (relaxkv_scale_scores, factor 1 / world); identity on a single rank.  Both are enqueued on `stream` (torch's
    current stream if None), so they are ordered after the scoring kernels and before the top-k on that stream.
    `scale_fn(session, factor)` replaces the kernel call where no GPU exists (the CPU rank tests)."""
    raw = session.raw
    if world <= 1:
        return raw
    import torch.distributed as dist
    if raw.is_cuda:
        ctx = torch.cuda.stream(stream) if stream is not None else torch.cuda.stream(torch.cuda.current_stream(raw.device))
        with ctx:
            dist.all_reduce(raw, op=dist.ReduceOp.SUM, group=group)
    else:
        dist.all_reduce(raw, op=dist.ReduceOp.SUM, group=group)
    if scale_fn is not None:
        scale_fn(session, 1.0 / world)
    else:
        from . import binding as B
        B.relaxkv_scale_scores(session.shape, session.n_layers, raw, 1.0 / world, stream=stream)
    return raw


def sharded_score_select(session, q_layers_local: List[torch.Tensor], cache_layers_local, world: int, group=None,
                         row_lse_layers=None, stream=None) -> None:
    """Selection on a head shard: local scoring kernels -> all-reduce of the scores -> scaling -> top-k kernel, all on
    `stream`.  `session` is a pipeline.RepairSession built with the LOCAL head counts; on return session.raw holds the
    global scores and session.anchors the anchors (identical on every rank)."""
    from . import binding as B
    B.relaxkv_score_select(session.shape, q_layers_local, cache_layers_local, session.k, session.raw, None,
                           session.workspace, row_lse_layers=row_lse_layers, stream=stream)
    combine_partial_scores(session, world, group, stream=stream)
    B.relaxkv_select_topk(session.shape, session.n_layers, session.k, session.raw, session.anchors,
                          norm_scores_out=session.norm, stream=stream)
