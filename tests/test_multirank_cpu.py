"""The N > 1 path of bench.py on CPU: two gloo ranks (replicas, no data-path collective).

The path is not sharded: every rank runs an independent replica and the only exchange is the
max-over-ranks of the device times.  This checks that plumbing with world_size 2 on CPU.
"""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local = [100.0 + 10.0 * rank, 50.0 - rank, 7.0, 3.0 * (rank + 1)]
    got = bench.max_over_ranks(local, dist, torch.device("cpu"))
    dist.barrier()
    out_q.put((rank, got))
    dist.destroy_process_group()


def test_max_over_ranks_and_job_value_world2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == res[1] == [110.0, 50.0, 7.0, 6.0]
    import bench
    # two replicas, each (b + 2) N^2 units, slowest rank 110 ms
    units = 66.0 * 1024 * 1024
    assert bench.job_value(units, 2, 110.0) == pytest.approx(2 * units / 0.110)
    assert bench.max_over_ranks([1.5, 2.5], None, torch.device("cpu")) == [1.5, 2.5]


def test_reference_arm_runs_on_rank0_only(monkeypatch, capsys):
    import bench
    monkeypatch.setenv("RANK", "1")

    class A:
        n, steps, warmup, gpus = 10, 1, 0, 2
    bench.run_reference(A())
    assert capsys.readouterr().out == ""          # other ranks exit without work
