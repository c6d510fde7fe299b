"""Row-sharded operation on the GPU: `world` in-process ranks (threads) share the one GPU, each with its own context,
stream and row range; the exchange runs on the host side between launches (ThreadTransport), so no kernel ever waits
for another rank.  Every library code path of the sharded mode runs here: owned-row quadratic passes, row gathers,
host sums, the eigensolver on owned rows, the flow.  Gates are the unsharded ones, against the float64 oracle.
"""
import threading

import numpy as np
import pytest
import torch

import workloads
from oracle import dense, flow

pytestmark = pytest.mark.gpu

TOL_APPLY = 1e-5


@pytest.fixture(scope="module")
def fd():
    import __graft_entry__ as g
    g.build()
    import paper_2609_38198_b200 as fd
    assert torch.cuda.is_available()
    return fd


@pytest.fixture(scope="module")
def dev():
    return torch.device("cuda:0")


def relF(a, b):
    a = np.asarray(a, dtype=np.float64)
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def run_ranks(fd, dev, world, X, b_max, m_max, body, path=None):
    """body(ctx, rank) -> result, run once per rank in its own thread on its own stream."""
    hub = fd.ThreadTransport.Hub(world, timeout=300.0)
    Xd = torch.from_numpy(X).to(dev)
    torch.cuda.synchronize()
    results, errors = [None] * world, [None] * world

    def worker(r):
        try:
            torch.cuda.set_device(dev)
            stream = torch.cuda.Stream(device=dev)
            with torch.cuda.stream(stream):
                ctx = fd.Context(Xd, b_max=b_max, m_max=m_max, stream=stream)
                if path is not None:
                    ctx.set_option("path", path)
                ctx.set_shard(fd.Shard(hub.rank(r), X.shape[0], b_max, dev, stream=stream))
                results[r] = body(ctx, r)
                ctx.synchronize()
                ctx.close()
        except BaseException as e:                               # noqa: BLE001
            errors[r] = e
            hub.barrier.abort()

    threads = [threading.Thread(target=worker, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    for e in errors:
        if e is not None and not isinstance(e, threading.BrokenBarrierError):
            raise e
    for e in errors:
        if e is not None:
            raise e
    return results


@pytest.mark.parametrize("world,N,path", [(2, 3000, None), (3, 3000, None), (2, 3000, "tc"), (3, 2304, "tc"), (2, 300, None),
                                          (3, 200, "tc"), (4, 16384, None)])
def test_degree_and_apply_sharded_match_oracle(fd, dev, world, N, path):
    X = workloads.torus6(N, seed=N + world)
    b, beta, alpha = 16, 2.0, 1.0
    V = workloads.block(N, b, seed=3)
    big = N > 8192

    def body(ctx, r):
        q, d, s, so, so2 = ctx.degree(beta, alpha)
        Y = ctx.apply(fd.to_colmajor(V, dev))
        ctx.synchronize()
        return q.cpu().numpy(), d.cpu().numpy(), s.cpu().numpy(), so, so2, Y.cpu().numpy(), ctx.get_option("last_path")

    res = run_ranks(fd, dev, world, X, b, 0, body, path={None: None, "tc": fd.FD_PATH_TC}[path])
    qo, do, s_o, soo, so2o = dense.degree(X, beta, alpha)
    Yo = dense.apply(X, beta, alpha, V)
    for r in range(world):
        q, d, s, so, so2, Y, last = res[r]
        if (path == "tc" or big) and fd.fd_shard_rows(N, world, r)[1] > fd.fd_shard_rows(N, world, r)[0]:
            assert last == fd.FD_PATH_TC                         # (a rank that owns no rows launches no quadratic kernel)
        assert np.abs(q / qo - 1).max() <= 2e-5 and np.abs(d / do - 1).max() <= 4e-5 and np.abs(s / s_o - 1).max() <= 4e-5
        assert abs(so - soo) <= 2e-5 * (soo + N) and abs(so2 - so2o) <= 4e-5 * (so2o + N)
        assert relF(Y, Yo) <= TOL_APPLY
        # complete and identical on every rank: each row was computed by exactly one owner
        assert np.array_equal(Y, res[0][5]) and np.array_equal(q, res[0][0]) and np.array_equal(s, res[0][2])
        assert so == res[0][3] and so2 == res[0][4]


def test_sharded_rows_equal_unsharded_rows(fd, dev):
    # a row's result depends on the other rows of its launch only through the summation order over column splits and
    # flush groups (chosen from the row count): the sharded product reproduces the unsharded one to fp32 rounding
    N, b = 2816, 32
    X = workloads.torus6(N, seed=5)
    V = workloads.block(N, b, seed=6)
    for path, tol in [(fd.FD_PATH_SIMT, 1e-6), (fd.FD_PATH_TC, 2e-6)]:
        ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=b)
        ctx.set_option("path", path)
        ctx.degree(1.5, 0.5)
        Y1 = ctx.apply(fd.to_colmajor(V, dev)).cpu().numpy()
        ctx.close()

        def body(c, r):
            c.degree(1.5, 0.5)
            return c.apply(fd.to_colmajor(V, dev)).cpu().numpy()

        Y2 = run_ranks(fd, dev, 2, X, b, 0, body, path=path)[1]
        assert relF(Y2, Y1.astype(np.float64)) <= tol


@pytest.mark.parametrize("world", [2, 3])
def test_eigs_sharded_match_oracle(fd, dev, world):
    N, beta, alpha, k, b = 2500, 0.6, 1.0, 12, 8
    X = workloads.torus6(N, seed=31)
    lam_o, U_o, d_o = dense.eigs(X, beta, alpha, k + 8)

    def body(ctx, r):
        ctx.degree(beta, alpha)
        lam, U, info = ctx.eigs(k, b)
        return lam, U.cpu().numpy(), (info.applies, info.restarts, info.converged, info.max_residual)

    res = run_ranks(fd, dev, world, X, b, 64, body)
    for r in range(world):
        lam, U, info = res[r]
        assert info[2] == k + 1
        assert np.abs(lam - lam_o[:k + 1]).max() <= 1e-6 * lam_o[0]
        assert np.array_equal(lam, res[0][0]) and info == res[0][2]          # same decisions on every rank
        assert np.array_equal(U, res[0][1])                                  # gathered eigenvectors identical everywhere
        assert np.abs(U.T.astype(np.float64) @ U - np.eye(k + 1)).max() <= 1e-5
        # residual certificate in float64 through the oracle's operator
        R = dense.apply(X, beta, alpha, U.astype(np.float64)) - U * lam[None, :]
        assert np.linalg.norm(R, axis=0).max() <= 5e-6
        # the 13-dimensional leading cluster cut (Perron + 12) is a clean gap on the 6-torus: full angle gate
        ang = dense.principal_angles(U[:, :k + 1], U_o[:, :k + 1])
        gap = lam_o[k] - lam_o[k + 1]
        assert ang.max() <= max(1e-4, 1e-6 / gap) or gap < 1e-3


def test_flow_sharded_matches_oracle_flow(fd, dev):
    N, alpha, k = 1024, 0.5, 3
    X = workloads.torus6_paper(N, seed=42)
    bx_o, status_o, log_o = flow.beta_flow(flow.dense_probe(X, alpha, k), N, flow.beta0(X), 1000.0)

    def body(ctx, r):
        bx, status, lam, U, recs = ctx.beta_flow(k, 8, alpha, beta_start=0.0, beta_max=1000.0)
        return bx, status, lam, [rec["beta"] for rec in recs]

    res = run_ranks(fd, dev, 2, X, 8, 64, body)
    for r in range(2):
        bx, status, lam, betas = res[r]
        assert status == status_o == "VERTEX"
        assert len(betas) == len(log_o)
        assert bx == pytest.approx(bx_o, rel=1e-3)
        assert (bx, betas) == (res[0][0], res[0][3]) and np.array_equal(lam, res[0][2])


def test_exchange_failure_is_reported_not_hung(fd, dev):
    # a transport whose gather raises: the library returns FD_ERR_COMM and the binding re-raises the cause
    class Broken:
        rank, world = 0, 1

        def allreduce_sum_host(self, arr, device, stream):
            pass

        def allgather(self, send, recv, stream):
            raise RuntimeError("link down")

    X = workloads.torus6(600, seed=2)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=8)
    ctx.set_shard(fd.Shard(Broken(), 600, 8, dev))
    with pytest.raises(fd.FdError) as e:
        ctx.degree(1.0, 1.0)
    assert e.value.status == fd.FD_ERR_COMM and isinstance(e.value.__cause__, RuntimeError)
    ctx.set_shard(None)                                           # back to unsharded operation: usable again
    q = ctx.degree(1.0, 1.0)[0].cpu().numpy()
    assert np.abs(q / dense.degree(X, 1.0, 1.0)[0] - 1).max() <= 2e-5
    ctx.close()


def test_torch_distributed_transport_on_a_one_rank_group(fd, dev):
    """The transport a multi-GPU job uses -- NCCL all_gather_into_tensor on the context's stream for the row gathers, a gloo
    group for the small host sums -- on a one-rank group, which needs only this GPU: degree passes, block product and
    eigensolver through fd_set_shard against the oracle."""
    import socket

    import torch.distributed as dist
    if dist.is_initialized():
        pytest.skip("a process group already exists in this process")
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1, device_id=dev)
    try:
        host_group = dist.new_group(backend="gloo")
        N, b, beta, alpha, k = 3000, 16, 1.0, 1.0, 6
        X = workloads.torus6(N, seed=77)
        V = workloads.block(N, b, seed=5)
        for path in (fd.FD_PATH_SIMT, fd.FD_PATH_TC):
            ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=b, m_max=64)
            ctx.set_option("path", path)
            ctx.set_shard(fd.Shard(fd.TorchDistTransport(0, 1, group=None, host_group=host_group), N, b, dev))
            q, d, s, so, so2 = ctx.degree(beta, alpha)
            Y = ctx.apply(fd.to_colmajor(V, dev))
            lam, U, info = ctx.eigs(k, 8)
            ctx.synchronize()
            qo, do, s_o, soo, so2o = dense.degree(X, beta, alpha)
            assert np.abs(q.cpu().numpy() / qo - 1).max() <= 2e-5 and abs(so - soo) <= 2e-5 * (soo + N)
            assert relF(Y.cpu().numpy(), dense.apply(X, beta, alpha, V)) <= TOL_APPLY
            lam_o, U_o, d_o = dense.eigs(X, beta, alpha, k)
            assert info.converged == k + 1 and np.abs(lam - lam_o).max() <= 1e-6
            ctx.close()
        # without a host group the small sums are staged through the device on the NCCL group
        ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=b, m_max=64)
        ctx.set_shard(fd.Shard(fd.TorchDistTransport(0, 1, group=None, host_group=None), N, b, dev))
        q2 = ctx.degree(beta, alpha)[0]
        assert np.abs(q2.cpu().numpy() / qo - 1).max() <= 2e-5
        ctx.close()
    finally:
        dist.destroy_process_group()


def test_eigs_sharded_with_a_rank_that_owns_no_rows(fd, dev):
    # 500 points on 3 ranks: ranges (0, 256), (256, 500), (500, 500) -- the last rank owns nothing, contributes zeros to every
    # sum and still has to take every decision the others take
    N, beta, alpha, k, b = 500, 0.4, 1.0, 6, 8
    X = workloads.torus6(N, seed=12)
    lam_o, U_o, d_o = dense.eigs(X, beta, alpha, k)
    assert fd.fd_shard_rows(N, 3, 2) == (500, 500)

    def body(ctx, r):
        ctx.degree(beta, alpha)
        lam, U, info = ctx.eigs(k, b)
        return lam, U.cpu().numpy(), info.converged

    res = run_ranks(fd, dev, 3, X, b, 64, body)
    for r in range(3):
        lam, U, conv = res[r]
        assert conv == k + 1 and np.abs(lam - lam_o).max() <= 1e-6
        assert np.array_equal(lam, res[0][0]) and np.array_equal(U, res[0][1])
