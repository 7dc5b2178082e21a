"""The N > 1 bench path shards by replica (independent requests, no data-path collective); the only
cross-rank step is the timing reduction: barrier, then the MAX of the ranks' elapsed times.  Checked
here with two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"), world)
    total = bench.whole_job_value(flops_per_rank=2.0e12, world=world, ms_per_step=ms)
    out[rank] = (ms, total)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_timing_is_the_max_and_value_is_the_whole_job():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0][0] == out[1][0] == 15.0
    assert abs(out[0][1] - 2 * 2.0e12 / 15e-3 / 1e12) < 1e-9


def _shard_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import relaxkv_oracle as orc
    from paper_2609_33503_b200 import inputs, sharded
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = inputs.scaled_down(inputs.llama8b_16k(), (384,), (12,), n_layers=1, chunk=64)
    q, k, v = inputs.layer_qkv(w, 0, 0)
    kv_lo, kv_hi, q_lo, q_hi = sharded.head_shard(w.n_q_heads, w.n_kv_heads, world, rank)
    scale = w.head_dim ** -0.5
    # the rank's partial score: the oracle on its own heads only (stands in for the CUDA kernels on a CPU machine)
    local = orc.raw_scores(inputs.bf16_bits(q[:, q_lo:q_hi]), inputs.bf16_bits(k[:, kv_lo:kv_hi]), scale)
    t = torch.from_numpy(local).clone().view(1, -1)

    class HostSession:            # the fields combine_partial_scores reads
        raw, n_layers, shape = t, 1, None

    def scale_on_host(session, factor):   # stands in for relaxkv_scale_scores, like the oracle does for the scoring
        session.raw.mul_(factor)

    sharded.combine_partial_scores(HostSession, world, scale_fn=scale_on_host)
    full = orc.raw_scores(inputs.bf16_bits(q), inputs.bf16_bits(k), scale)
    out[rank] = (float(np.abs(t.numpy()[0] - full).max() / full.max()), orc.topk(t.numpy()[0], 58).tolist() == orc.topk(full, 58).tolist())
    dist.barrier()
    dist.destroy_process_group()


def test_head_sharded_scores_combine_to_the_full_score():
    """Two ranks, each scoring half of the KV heads: one all-reduce of the score vector gives the score over
    all heads, hence the same anchors on every rank (the only exchange step of the sharded path)."""
    from paper_2609_33503_b200 import sharded
    assert sharded.head_shard(40, 8, 4, 1) == (2, 4, 10, 20)
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_shard_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    for r in range(world):
        err, same = out[r]
        assert err < 1e-12 and same


def test_bench_starts_its_own_ranks_when_asked_for_several_gpus():
    """`bench.py --gpus N` without a launcher around it starts N local ranks itself (torch.distributed.run,
    rendezvous on 127.0.0.1).  Driven here with a stand-in job and gloo: the printed line must come from rank 0,
    count two ranks, carry the slowest rank's time and the whole-job value."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selftest-ranks"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["ms_per_step"] == 15.0 and d["backend"] == "gloo"
    assert abs(d["value"] - 2 * 2.0e12 / 15e-3 / 1e12) < 1e-9
