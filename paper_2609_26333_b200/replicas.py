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


def spawn_command(n_ranks: int, script_and_args, master_port: int = 0):
    """Command line that runs `script_and_args` as `n_ranks` processes (one per GPU) of one node under
    torch.distributed.run, rendezvous on 127.0.0.1; what `bench.py --gpus N` re-executes itself as when it was not
    started by a launcher."""
    import socket
    import sys

    if master_port == 0:
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            master_port = s.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(n_ranks)}",
            "--master-addr", "127.0.0.1", "--master-port", str(master_port)] + [str(a) for a in script_and_args]
