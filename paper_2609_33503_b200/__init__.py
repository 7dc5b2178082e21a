"""RelaxKV selective cache-repair hot path for NVIDIA B200 (sm_100a).

`binding` mirrors the C ABI of include/relaxkv.h one to one; `pipeline.RepairSession` keeps the
device buffers of a request batch and issues the calls in the order of the paper's Algorithm 1;
`inputs` holds the seeded synthetic workloads.  All computation is in librelaxkv.so (CUDA); build
it with `python -m paper_2609_33503_b200.build`.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding", "pipeline", "build"]
