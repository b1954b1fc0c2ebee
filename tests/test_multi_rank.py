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


_RANK_SCRIPT = """
import json, os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
from paper_2510_27527_b200 import multi
dist.init_process_group("gloo")
rank, world = multi.world_info()
assert world == int(os.environ["WORLD_SIZE"]) == int(sys.argv[sys.argv.index("--gpus") + 1])
slowest = multi.max_over_ranks(0.010 * (rank + 1))
thr = multi.job_throughput(100.0, 0.010 * (rank + 1))
dist.barrier()
if rank == 0:
    open(sys.argv[sys.argv.index("--out") + 1], "w").write(json.dumps({{"world": world, "slowest": slowest, "thr": thr}}))
dist.destroy_process_group()
"""


def test_launch_ranks_starts_one_process_per_rank(tmp_path):
    """`bench.py --gpus N` without torchrun starts its ranks through multi.launch_ranks: here with two gloo ranks on CPU."""
    import json

    sys.path.insert(0, ROOT)
    from paper_2510_27527_b200 import multi

    script = tmp_path / "rank_script.py"
    script.write_text(_RANK_SCRIPT.format(root=ROOT))
    out = tmp_path / "out.json"
    rc = multi.launch_ranks(2, str(script), ["--gpus", "2", "--out", str(out)], timeout=300)
    assert rc == 0
    got = json.loads(out.read_text())
    assert got["world"] == 2
    assert got["slowest"] == pytest.approx(0.020)
    assert got["thr"] == pytest.approx(2 * 100.0 / 0.020)


def test_bench_parses_gpus_and_would_spawn(monkeypatch):
    """bench.py hands `--gpus N > 1` to launch_ranks when it was not started by torchrun (no WORLD_SIZE in the environment)."""
    import importlib

    sys.path.insert(0, ROOT)
    bench = importlib.import_module("bench")
    from paper_2510_27527_b200 import multi

    calls = []
    monkeypatch.setattr(multi, "launch_ranks", lambda n, script, argv, timeout=None: calls.append((n, script, list(argv))) or 0)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "2"])
    with pytest.raises(SystemExit) as e:
        bench.main()
    assert e.value.code == 0
    assert calls == [(4, os.path.join(ROOT, "bench.py"), ["--gpus", "4", "--steps", "2"])]


def test_module_keys_differ_between_layers_and_calls():
    """Two modules built from the same configuration, and two calls of one module, must not share their stochastic-rounding
    key (the draws of equal-shaped layers would otherwise be identical element for element)."""
    from paper_2510_27527_b200 import module

    keys = {module.call_seed(0, layer, call) for layer in range(24) for call in range(50)}
    assert len(keys) == 24 * 50
    assert all(0 <= k < 1 << 64 for k in keys)
    assert module.call_seed(0, 0, 0) != module.call_seed(1, 0, 0)
    assert module.call_seed(7, 3, 5) == module.call_seed(7, 3, 5)
