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
