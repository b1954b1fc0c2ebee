"""World-size-2 check (gloo, CPU) of the benchmark's multi-rank bookkeeping: time = max over ranks, work = sum."""
import os
import socket
import sys

import pytest
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
    import torch.distributed as dist

    from paper_2510_27527_b200 import multi

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_seconds = 0.010 if rank == 0 else 0.025  # rank 1 is the slow one
    slowest = multi.max_over_ranks(local_seconds)
    thr = multi.job_throughput(100.0, local_seconds)
    dist.barrier()
    out[rank] = (multi.world_info(), slowest, thr)
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    with ctx.Manager() as mgr:
        out = mgr.dict()
        port = _free_port()
        procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        for r in range(2):
            (rank, world), slowest, thr = out[r]
            assert (rank, world) == (r, 2)
            assert slowest == pytest.approx(0.025)
            assert thr == pytest.approx(2 * 100.0 / 0.025)


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    from paper_2510_27527_b200 import multi

    assert multi.world_info() == (0, 1)
    assert multi.max_over_ranks(0.5) == 0.5
    assert multi.job_throughput(10.0, 0.5) == 20.0
