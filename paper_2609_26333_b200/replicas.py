"""Timing bookkeeping for N independent replicas (one process per GPU).

The path has no exchange step: a linear layer's prefill GEMM and decode mat-vec run on one GPU,
so `bench.py --gpus N` runs N replicas of the same workload.  The only communication is the
barrier around the timed region and the max over ranks of the device-measured times."""
from __future__ import annotations

import torch


def max_over_ranks(values, device=None):
    """Element-wise maximum over all ranks of a list of floats (identity without a process group)."""
    import torch.distributed as dist

    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_rate(units_per_rank: float, world: int, slowest_ms: float) -> float:
    """Units all ranks processed per second, on the clock of the slowest rank (weak scaling)."""
    return world * units_per_rank / (slowest_ms * 1e-3)
