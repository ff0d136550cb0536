"""The N > 1 path of bench.py on CPU: two gloo ranks, max over ranks of the per-rank times and
the whole-job rate derived from it."""
import os
import socket
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2609_26333_b200 import replicas

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        mine = [10.0 + rank, 5.0 - rank, 0.25 * (rank + 1)]          # per-rank device times (ms)
        got = replicas.max_over_ranks(mine)
        rate = replicas.whole_job_rate(units_per_rank=1.0e12, world=world, slowest_ms=got[0])
        dist.barrier()
        torch.save({"got": got, "rate": rate}, os.path.join(out_dir, f"r{rank}.pt"))
    finally:
        dist.destroy_process_group()


def test_two_rank_max_and_whole_job_rate(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        r = torch.load(os.path.join(str(tmp_path), f"r{rank}.pt"))
        assert r["got"] == [11.0, 5.0, 0.5]                           # same on every rank
        assert r["rate"] == pytest.approx(2 * 1.0e12 / 11.0e-3)


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2609_26333_b200 import replicas

    assert replicas.max_over_ranks([3.0, 1.5]) == [3.0, 1.5]
    assert replicas.whole_job_rate(2.0, 1, 1000.0) == 2.0


def test_bench_starts_its_own_ranks_when_asked_for_several_gpus():
    """`bench.py --gpus 2` outside a launcher re-executes itself as two ranks; the CPU arm prints one line (rank 0)
    that says n_gpus 2, the other rank exits without work."""
    import json
    import subprocess

    sys.path.insert(0, ROOT)
    from paper_2609_26333_b200 import replicas

    cmd = replicas.spawn_command(3, ["x.py", "--a", 1], master_port=1234)
    assert cmd[1:] == ["-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=3", "--master-addr", "127.0.0.1",
                       "--master-port", "1234", "x.py", "--a", "1"]
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--workload", "c1_tiny", "--ref-rows", "16"], capture_output=True, text=True,
                         env=env, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2
