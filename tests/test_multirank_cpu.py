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


# ---------------------------------------------------------------- row-sharded operation: host side on two gloo ranks
def _shard_worker(rank, world, port, out_q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import ctypes

    import numpy as np

    import paper_2609_38198_b200 as fd
    N, b_max = 1000, 8
    sh = fd.Shard(fd.TorchDistTransport(rank, world), N, b_max, "cpu")
    # drive the two callbacks exactly as the library does: raw pointers into the exchange buffer / a host array
    count = 3 * 512                                              # three columns of one 512-row chunk
    send = sh._view(sh._base, count)
    send.copy_(torch.arange(count, dtype=torch.float32) + 1000.0 * rank)
    rc = sh.struct.allgather_dev(None, ctypes.c_void_p(sh._base), ctypes.c_void_p(sh._base + 4 * b_max * 512), count)
    recv = sh._view(sh._base + 4 * b_max * 512, count * world).clone()
    host = np.array([1.5 + rank, -2.0 * (rank + 1), 1e-3], dtype=np.float64)
    rc2 = sh.struct.allreduce_sum_host(None, host.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), 3)
    bad = sh.struct.allgather_dev(None, ctypes.c_void_p(sh._base - 64), ctypes.c_void_p(sh._base), 4)   # outside the buffer
    dist.barrier()
    out_q.put((rank, rc, rc2, bad, recv.numpy().tolist(), host.tolist(), (sh.row_begin, sh.row_end), type(sh.error).__name__))
    dist.destroy_process_group()


def test_shard_callbacks_world2_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = {r[0]: r[1:] for r in (q.get(timeout=180) for _ in range(2))}
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    want = [float(i) for i in range(3 * 512)] + [1000.0 + i for i in range(3 * 512)]
    for r in range(2):
        rc, rc2, bad, recv, host, rows, err = res[r]
        assert rc == 0 and rc2 == 0
        assert bad == 1 and err == "ValueError"                  # a pointer outside the buffer is refused, nothing raised into C
        assert recv == want                                      # ordered by rank, identical on both ranks
        assert host == [1.5 + 2.5, -2.0 - 4.0, 2e-3]
    assert res[0][5] == (0, 512) and res[1][5] == (512, 1000)


def test_shard_rows_partition_every_point_once():
    import paper_2609_38198_b200 as fd
    for N in [1, 100, 255, 256, 257, 1000, 4096, 16384, 131072, 1 << 20, (1 << 20) + 7]:
        for world in [1, 2, 3, 4, 8]:
            ranges = [fd.fd_shard_rows(N, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == N
            for (b0, e0), (b1, e1) in zip(ranges, ranges[1:]):
                assert e0 == b1 and b0 <= e0
            chunk = ranges[0][1] - ranges[0][0]
            assert all(e - b <= chunk for b, e in ranges)
            assert all(b % 256 == 0 for b, e in ranges if e > b)
            # exchange buffer: (world + 1) chunks of the padded block width, no N^2 term
            assert fd.fd_shard_exchange_bytes(N, 64, world) == (world + 1) * 64 * (-(-(-(-N // world)) // 256) * 256) * 4
    with pytest.raises(fd.FdError):
        fd.fd_shard_rows(100, 2, 2)
    assert fd.fd_shard_exchange_bytes(0, 8, 2) == 0
