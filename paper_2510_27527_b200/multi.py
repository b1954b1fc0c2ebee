"""Multi-rank bookkeeping of the benchmark (one process per GPU, independent replicas).

The NVFP4 linear-layer path shards by tokens with no collective on the data path (the data-parallel all-reduce of
dW belongs to the trainer, not to this library), so N ranks are N replicas: the job's time is the slowest rank's,
its work the sum over ranks. Only the timing scalar crosses ranks."""
from __future__ import annotations

import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist


def world_info():
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` among all ranks (every rank gets it)."""
    _, world = world_info()
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, seconds_local: float, device="cpu") -> float:
    """Whole-job throughput: units of all ranks divided by the slowest rank's time."""
    _, world = world_info()
    return world * units_per_rank / max_over_ranks(seconds_local, device)


def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def launch_ranks(n: int, script: str, argv: list[str], timeout: float | None = None) -> int:
    """Starts `script argv...` as n ranks of one node (one process per GPU) under torch.distributed.run with a rendezvous
    on 127.0.0.1 and a free port, waits for them, and returns the launcher's exit code. The ranks read RANK / LOCAL_RANK /
    WORLD_SIZE / MASTER_* from the environment; their output goes to this process's stdout / stderr."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), script] + list(argv)
    env = dict(os.environ)
    env.setdefault("OMP_NUM_THREADS", "1")
    return subprocess.run(cmd, env=env, timeout=timeout).returncode
