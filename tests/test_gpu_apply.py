"""GPU parity of the degree passes and the block product against the float64 oracle.

Every call goes through the C ABI (ctypes binding).  Tolerances: relative Frobenius error of
the block product <= 1e-5 in the fp32 mode (<= 3e-3 in the fast mode); q, d, s to 1e-5
relative entrywise (they are sums of positive terms, so the bound is tight); S_off to 1e-6.
"""
import numpy as np
import pytest
import torch

import workloads
from oracle import blocked, dense

pytestmark = pytest.mark.gpu

TOL_APPLY = 1e-5
TOL_FAST = 3e-3


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


def run_case(fd, dev, X, beta, alpha, b, path, seed=1, prec=0, tol=TOL_APPLY):
    N = X.shape[0]
    V = workloads.block(N, b, seed=seed)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=max(b, 1))
    ctx.set_option("path", path)
    q, d, s, so, so2 = ctx.degree(beta, alpha, prec)
    Y = ctx.apply(fd.to_colmajor(V, dev), prec=prec)
    torch.cuda.synchronize()
    qo, do, s_o, soo, so2o = dense.degree(X, beta, alpha)
    Yo = dense.apply(X, beta, alpha, V)
    assert np.abs(q.cpu().numpy() / qo - 1).max() <= tol
    assert np.abs(d.cpu().numpy() / do - 1).max() <= 2 * tol
    assert np.abs(s.cpu().numpy() / s_o - 1).max() <= 2 * tol
    # S_off = sum(q) - N with q held in fp32: absolute floor of ~1e-7 per row on top of the relative bound
    assert abs(so - soo) <= max(1e-6, tol / 10) * soo + 2e-7 * N
    assert abs(so2 - so2o) <= max(1e-6, tol / 10) * so2o + 2e-7 * N
    err = relF(Y.cpu().numpy(), Yo)
    assert err <= tol, f"apply rel-Frobenius error {err:.3e}"
    ctx.close()
    return err


# ------------------------------------------------------------------ the five configurations, reduced N
@pytest.mark.parametrize("alpha", [1.0, 0.5, 0.0])
def test_c1_circle_full(fd, dev, alpha):
    run_case(fd, dev, workloads.circle(2048), 200.0, alpha, 8, fd.FD_PATH_SIMT)


@pytest.mark.parametrize("beta", [10.0, 30.0, 100.0, 300.0])
def test_c2_torus2_reduced(fd, dev, beta):
    run_case(fd, dev, workloads.torus2(4096), beta, 1.0, 16, fd.FD_PATH_SIMT)


@pytest.mark.parametrize("beta", [0.5, 2.0])
def test_c3_torus6_reduced_ragged(fd, dev, beta):
    run_case(fd, dev, workloads.torus6(3001), beta, 1.0, 32, fd.FD_PATH_SIMT)


def test_c4_latent_torus_reduced(fd, dev):
    run_case(fd, dev, workloads.latent_torus(2500), 2.0, 1.0, 32, fd.FD_PATH_SIMT)


def test_c5_block64_reduced(fd, dev):
    run_case(fd, dev, workloads.torus6(2304), 2.0, 1.0, 64, fd.FD_PATH_SIMT)


# ------------------------------------------------------------------ edge shapes
@pytest.mark.parametrize("N", [1, 2, 127, 128, 129, 1000, 2049])
def test_tail_sizes(fd, dev, N):
    run_case(fd, dev, workloads.gaussian_cloud(N, 3, seed=N), 0.7, 1.0, 8 if N > 1 else 1, fd.FD_PATH_SIMT)


@pytest.mark.parametrize("b", [1, 3, 8, 16, 33, 40, 48, 64, 70, 130])
def test_block_widths(fd, dev, b):
    run_case(fd, dev, workloads.torus6(700, seed=b), 1.0, 1.0, b, fd.FD_PATH_SIMT)


@pytest.mark.parametrize("D", [1, 2, 3, 4, 5, 12, 30, 32])
def test_dimensions(fd, dev, D):
    run_case(fd, dev, workloads.gaussian_cloud(600, D, seed=D, scale=0.8), 0.9 / max(1, D // 4), 0.5, 8, fd.FD_PATH_SIMT)


def test_duplicate_points_and_far_pairs(fd, dev):
    X = workloads.gaussian_cloud(300, 4, seed=3)
    X[10] = X[11]                        # duplicate: K = 1
    X[50] += 100.0                       # far away: K underflows to 0 against everyone else
    run_case(fd, dev, X, 1.0, 1.0, 8, fd.FD_PATH_SIMT)


def test_forced_splits_are_deterministic_and_correct(fd, dev):
    X = workloads.torus2(1500, seed=3)
    V = workloads.block(1500, 16, seed=2)
    Yo = dense.apply(X, 30.0, 1.0, V)
    outs = []
    for splits in (1, 3, 8, 8):
        ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=16)
        ctx.set_option("path", fd.FD_PATH_SIMT)
        ctx.set_option("splits", splits)
        ctx.degree(30.0, 1.0)
        Y = ctx.apply(fd.to_colmajor(V, dev)).cpu().numpy()
        assert relF(Y, Yo) <= TOL_APPLY
        outs.append(Y)
        ctx.close()
    assert np.array_equal(outs[2], outs[3])          # same configuration -> bit-identical


# ------------------------------------------------------------------ the general primitive
def test_apply_general_scalings_ones_and_rectangular(fd, dev):
    X = workloads.torus6(900, seed=5)
    Z = workloads.torus6(333, seed=6)
    N = 900
    rng = np.random.default_rng(0)
    l = rng.uniform(0.5, 2.0, N).astype(np.float32)
    r = rng.uniform(0.5, 2.0, N).astype(np.float32)
    lz = rng.uniform(0.5, 2.0, 333).astype(np.float32)
    V = workloads.block(N, 8, seed=4)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=8)
    ctx.set_option("path", fd.FD_PATH_SIMT)
    t = lambda a: torch.from_numpy(a).to(dev)
    Vd = fd.to_colmajor(V, dev)
    beta = 0.8
    Y = ctx.apply_general(beta, Vd, left=t(l), right=t(r)).cpu().numpy()
    assert relF(Y, dense.apply_general(X, beta, V, left=l, right=r)) <= TOL_APPLY
    Y = ctx.apply_general(beta, Vd).cpu().numpy()
    assert relF(Y, dense.apply_general(X, beta, V)) <= TOL_APPLY
    q1 = ctx.apply_general(beta, None).cpu().numpy()[:, 0]                    # K 1 = q
    assert np.abs(q1 / dense.degree(X, beta, 0.0)[0] - 1).max() <= TOL_APPLY
    Y = ctx.apply_general(beta, Vd, left=t(lz), right=t(r), Xrow=t(Z)).cpu().numpy()
    assert Y.shape == (333, 8)
    assert relF(Y, dense.apply_general(X, beta, V, left=lz, right=r, Xrow=Z)) <= TOL_APPLY
    # more new rows than context points: staged chunk by chunk
    Zb = workloads.torus6(2000, seed=8)
    Y = ctx.apply_general(beta, Vd, right=t(r), Xrow=t(Zb)).cpu().numpy()
    assert relF(Y, dense.apply_general(X, beta, V, right=r, Xrow=Zb)) <= TOL_APPLY
    ctx.close()


def test_matrix_free_identities(fd, dev):
    # hold at any size with no oracle: M sqrt(d) = sqrt(d); U^T (M V) = (M U)^T V; linearity
    X = workloads.torus6(5000, seed=11)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=8)
    ctx.set_option("path", fd.FD_PATH_SIMT)
    q, d, s, _, _ = ctx.degree(1.0, 1.0)
    sd = torch.sqrt(d.double()).float()
    Y = ctx.apply(sd[:, None].t().contiguous().t())
    assert float((Y[:, 0] - sd).abs().max() / sd.abs().max()) <= 1e-5
    U = fd.to_colmajor(workloads.block(5000, 4, seed=1), dev)
    V = fd.to_colmajor(workloads.block(5000, 4, seed=2), dev)
    MU, MV = ctx.apply(U), ctx.apply(V)
    a = (U.double().t() @ MV.double()).cpu().numpy()
    b = (MU.double().t() @ V.double()).cpu().numpy()
    assert np.abs(a - b).max() <= 1e-5 * np.abs(a).max()
    MUV = ctx.apply((U + 2 * V).t().contiguous().t())
    assert float((MUV - (MU + 2 * MV)).abs().max()) <= 1e-5 * float(MUV.abs().max())
    ctx.close()


def test_sampled_rows_medium_size(fd, dev):
    # C2 at full N = 16384: oracle on sampled rows (rows.c), GPU on everything
    X = workloads.torus2(16384)
    N = 16384
    rows = workloads.row_sample(N, 256)
    V = workloads.block(N, 16, seed=9)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=16)
    ctx.set_option("path", fd.FD_PATH_SIMT)
    for beta in (10.0, 300.0):
        q, d, s, so, so2 = ctx.degree(beta, 1.0)
        qo, sq = blocked.rows_apply_general(X, beta, None, rows=rows, want_rowsq=True)
        assert np.abs(q.cpu().numpy()[rows] / qo[:, 0] - 1).max() <= TOL_APPLY
        # d, s and M V on sampled rows, using the oracle's own full q (second pass needs all of q)
        qfull = blocked.rows_apply_general(X, beta, None)[:, 0]
        qa = 1.0 / qfull
        do = blocked.rows_apply_general(X, beta, None, rows=rows, left=qa, right=qa)[:, 0]
        assert np.abs(d.cpu().numpy()[rows] / do - 1).max() <= 2 * TOL_APPLY
        assert abs(so / (qfull.sum() - N) - 1) <= 1e-6
        dfull = blocked.rows_apply_general(X, beta, None, left=qa, right=qa)[:, 0]
        sfull = qa / np.sqrt(dfull)
        Yo = blocked.rows_apply_general(X, beta, V, rows=rows, left=sfull, right=sfull)
        Y = ctx.apply(fd.to_colmajor(V, dev)).cpu().numpy()
        assert relF(Y[rows], Yo) <= TOL_APPLY
    ctx.close()


# ------------------------------------------------------------------ error behaviour on a live context
def test_error_paths(fd, dev):
    X = workloads.torus2(256, seed=1)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=8)
    V = fd.to_colmajor(workloads.block(256, 8), dev)
    with pytest.raises(fd.FdError) as e:
        ctx.apply(V)                                   # before fd_degree
    assert e.value.status == fd.FD_ERR_INVALID
    ctx.degree(10.0, 1.0)
    with pytest.raises(fd.FdError):
        ctx.apply(fd.to_colmajor(workloads.block(256, 9), dev))     # b > b_max
    with pytest.raises(fd.FdError):
        ctx.apply(V, out=V)                            # aliasing
    with pytest.raises(fd.FdError):
        ctx.degree(-1.0, 1.0)
    with pytest.raises(fd.FdError):
        ctx.set_option("no_such_option", 1)
    assert ctx.beta0() == pytest.approx(0.1)           # 1 / (2 * 2) = 0.25 -> capped (Eq. 7)
    # workspace too small
    import ctypes
    h = ctypes.c_void_p()
    ws = torch.empty(1024, dtype=torch.uint8, device=dev)
    Xd = torch.from_numpy(X).to(dev)
    st = fd.lib.fd_create(ctypes.byref(h), ctypes.c_void_p(Xd.data_ptr()), 256, 4, 4, 1, 8, 0,
                          ctypes.c_void_p((ws.data_ptr() + 255) // 256 * 256), 512, None)
    assert st == fd.FD_ERR_WORKSPACE
    ctx.close()


def test_beta0_matches_oracle(fd, dev):
    from oracle import flow
    for X in (workloads.torus6(2000, seed=2), workloads.latent_torus(1500, seed=3),
              workloads.gaussian_cloud(500, 3, seed=1, scale=5.0) + 3.0):
        ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=1)
        assert ctx.beta0() == pytest.approx(flow.beta0(X), rel=1e-6)
        ctx.close()


# ------------------------------------------------------------------ seeded sweep over shapes, both kernel families
@pytest.mark.parametrize("seed", range(20))
def test_seeded_shape_sweep_both_families(fd, dev, seed):
    """Random (N, D, b, alpha, beta) drawn from a seed: ragged sizes around the tile edges, every dimension the kernels
    cover, block widths that straddle the column-tile widths.  Each shape runs on every kernel family that covers it
    (direct differences for D <= 32, Gram form for D <= 60 within its accuracy budget), against the dense oracle."""
    rng = np.random.default_rng(1000 + seed)
    N = int(rng.choice([1, 2, 31, 127, 128, 129, 255, 256, 257, 383, 511, 640, 1000, 1537, 2049, 2600]))
    D = int(rng.integers(1, 61))
    b = int(rng.choice([1, 2, 7, 8, 15, 16, 17, 31, 32, 33, 47, 63, 64, 65, 100]))
    alpha = float(rng.choice([0.0, 0.5, 1.0]))
    X = workloads.gaussian_cloud(N, D, seed=seed, scale=0.6)
    # bandwidth: a few tens of effective neighbours, and an exponent magnitude the Gram form is trusted with
    mu = X.mean(axis=0, keepdims=True)
    max_sq = float(((X - mu) ** 2).sum(axis=1).max()) if N > 1 else 1.0
    beta = float(min(2.0 / (0.36 * D), 40.0 / (1.4427 * max(max_sq, 1e-3))))
    V = workloads.block(N, b, seed=seed + 5)
    qo, do, s_o, soo, so2o = dense.degree(X, beta, alpha)
    Yo = dense.apply(X, beta, alpha, V)
    paths = ([fd.FD_PATH_SIMT] if D <= 32 else []) + [fd.FD_PATH_TC]
    for path in paths:
        tol = 1e-5 if path == fd.FD_PATH_SIMT else 2e-5
        ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=b)
        ctx.set_option("path", path)
        q, d, s, so, so2 = ctx.degree(beta, alpha)
        Y = ctx.apply(fd.to_colmajor(V, dev)) if N > 1 or b == 1 else None
        ctx.synchronize()
        assert ctx.get_option("last_path") == path
        assert np.abs(q.cpu().numpy() / qo - 1).max() <= tol, (N, D, b, path)
        assert np.abs(d.cpu().numpy() / do - 1).max() <= 2 * tol and np.abs(s.cpu().numpy() / s_o - 1).max() <= 2 * tol
        assert abs(so - soo) <= tol * (soo + N) and abs(so2 - so2o) <= 2 * tol * (so2o + N)
        if Y is not None:
            err = relF(Y.cpu().numpy(), Yo)
            assert err <= TOL_APPLY, (N, D, b, alpha, beta, path, err)
        ctx.close()
