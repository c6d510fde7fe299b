"""GPU parity of the tensor-core (tcgen05 / TMEM, Gram-form) kernels against the float64 oracle.

Same gates as the direct-difference kernels for the block product (relative Frobenius error
<= 1e-5 in the fp32 mode, <= 3e-3 in the fast mode).  The degree vectors q, d, s carry a small
systematic relative bias on this path (the Gram tile is accumulated inside the tensor core at the
magnitude of beta' |x|^2 and rounded towards zero there); it is common to all entries, cancels in
M = diag(s) K diag(s), and is gated at 2e-5 entrywise here.
"""
import numpy as np
import pytest
import torch

import workloads
from oracle import blocked, dense

pytestmark = pytest.mark.gpu

TOL_APPLY = 1e-5
TOL_FAST = 3e-3
TOL_DEG = 2e-5


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


def tc_case(fd, dev, X, beta, alpha, b, prec=0, seed=1):
    N = X.shape[0]
    V = workloads.block(N, b, seed=seed)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=b)
    ctx.set_option("path", fd.FD_PATH_TC)
    q, d, s, so, so2 = ctx.degree(beta, alpha, prec)
    assert ctx.get_option("last_path") == fd.FD_PATH_TC
    Y = ctx.apply(fd.to_colmajor(V, dev), prec=prec)
    ctx.synchronize()
    assert ctx.get_option("last_path") == fd.FD_PATH_TC
    qo, do, s_o, soo, so2o = dense.degree(X, beta, alpha)
    Yo = dense.apply(X, beta, alpha, V)
    assert np.abs(q.cpu().numpy() / qo - 1).max() <= TOL_DEG
    assert np.abs(d.cpu().numpy() / do - 1).max() <= 2 * TOL_DEG
    assert np.abs(s.cpu().numpy() / s_o - 1).max() <= 2 * TOL_DEG
    assert abs(so - soo) <= TOL_DEG * (soo + N)
    assert abs(so2 - so2o) <= 2 * TOL_DEG * (so2o + N)
    err = relF(Y.cpu().numpy(), Yo)
    assert err <= (TOL_FAST if prec else TOL_APPLY), f"apply rel-Frobenius error {err:.3e}"
    ctx.close()
    return err


@pytest.mark.parametrize("N", [1, 100, 256, 257, 1000, 2304])
def test_row_and_column_tails(fd, dev, N):
    tc_case(fd, dev, workloads.torus6(N, seed=N), 2.0, 1.0, 64 if N > 1 else 1)


@pytest.mark.parametrize("b", [1, 8, 16, 24, 32, 40, 48, 64, 70, 128])
def test_block_widths(fd, dev, b):
    tc_case(fd, dev, workloads.torus6(900, seed=b), 1.0, 1.0, b)


@pytest.mark.parametrize("D,beta", [(2, 3.0), (4, 3.0), (12, 2.0), (13, 1.0), (20, 1.0), (28, 0.5), (30, 1.0), (32, 0.5)])
def test_dimensions_and_k_slabs(fd, dev, D, beta):
    X = workloads.latent_torus(1200, seed=D, D=D) if D >= 13 else workloads.gaussian_cloud(1200, D, seed=D, scale=0.7)
    tc_case(fd, dev, X, beta, 1.0, 32)


@pytest.mark.parametrize("D,b", [(30, 64), (32, 48), (40, 64), (50, 40), (60, 64)])
def test_wide_blocks_at_large_dimension_are_served_in_narrower_chunks(fd, dev, D, b):
    # the stages of a 64-column chunk do not fit in shared memory beyond D = 28 (fp32-grade kernel): the product is then
    # swept in 32- or 16-column chunks; the reduced-precision kernel keeps 64
    X = workloads.latent_torus(1500, seed=D, D=D)
    beta = 0.3
    err = tc_case(fd, dev, X, beta, 1.0, b)
    assert err <= TOL_APPLY
    tc_case(fd, dev, X, beta, 1.0, b, prec=1)


def test_dimensions_33_to_60_take_the_gram_form_path_at_any_size(fd, dev):
    # 32 < D <= 60 is covered by the tensor-core family alone: the automatic choice must pick it even for a small point
    # set, and a bandwidth beyond its accuracy budget is refused instead of silently served by nothing
    X = workloads.latent_torus(2000, seed=40, D=40)
    V = workloads.block(2000, 16, seed=4)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=16)            # path: automatic
    q, d, s, so, so2 = ctx.degree(0.5, 1.0)
    Y = ctx.apply(fd.to_colmajor(V, dev))
    ctx.synchronize()
    assert ctx.get_option("last_path") == fd.FD_PATH_TC
    assert relF(Y.cpu().numpy(), dense.apply(X, 0.5, 1.0, V)) <= TOL_APPLY
    with pytest.raises(fd.FdError) as e:
        ctx.degree(500.0, 1.0)
    assert e.value.status == fd.FD_ERR_UNSUPPORTED
    ctx.close()
    assert fd.fd_workspace_bytes(64, 61, 8, 32) == 0                   # D > FD_MAX_D: no workspace size, no context
    with pytest.raises(fd.FdError):
        fd.Context(torch.zeros((64, 61), dtype=torch.float32, device=dev), b_max=8)


def test_non_finite_points_are_refused(fd, dev):
    X = workloads.torus6(500, seed=1)
    X[123, 4] = np.nan
    with pytest.raises(fd.FdError) as e:
        fd.Context(torch.from_numpy(X).to(dev), b_max=8)
    assert e.value.status == fd.FD_ERR_NONFINITE
    X[123, 4] = np.inf
    with pytest.raises(fd.FdError) as e:
        fd.Context(torch.from_numpy(X).to(dev), b_max=8)
    assert e.value.status == fd.FD_ERR_NONFINITE


@pytest.mark.parametrize("N", [1, 100, 256, 257, 600, 1000, 2304, 5000])
@pytest.mark.parametrize("alpha", [0.0, 1.0])
def test_symmetric_half_work_degree_passes(fd, dev, N, alpha):
    """K = K^T (Sec. 2.1): the degree passes evaluate only the tiles on or above the diagonal and take the mirrored half
    from column sums.  Same gates against the oracle as the full evaluation, agreement with it to fp32 rounding, identical
    bits from run to run (fixed-point sums), odd and even numbers of row pairs, padding inside the last tiles."""
    X = workloads.torus6(N, seed=N + 7)
    beta = 2.0
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=8)
    ctx.set_option("path", fd.FD_PATH_TC)
    out = {}
    for sym in (1, 0, 1):
        ctx.set_option("sym", sym)
        q, d, s, so, so2 = ctx.degree(beta, alpha)
        assert ctx.get_option("last_path") == fd.FD_PATH_TC
        res = (q.cpu().numpy(), d.cpu().numpy(), s.cpu().numpy(), so, so2)
        if sym == 1 and 1 in out:
            for a, b in zip(res[:3], out[1][:3]):
                assert np.array_equal(a, b)
            assert res[3:] == out[1][3:]
        out[sym] = res
    qo, do, s_o, soo, so2o = dense.degree(X, beta, alpha)
    for sym in (1, 0):
        q, d, s, so, so2 = out[sym]
        assert np.abs(q / qo - 1).max() <= TOL_DEG
        assert np.abs(d / do - 1).max() <= 2 * TOL_DEG and np.abs(s / s_o - 1).max() <= 2 * TOL_DEG
        assert abs(so - soo) <= TOL_DEG * (soo + N) and abs(so2 - so2o) <= 2 * TOL_DEG * (so2o + N)
    assert np.abs(out[1][0] / out[0][0] - 1).max() <= 2e-6 and np.abs(out[1][1] / out[0][1] - 1).max() <= 4e-6
    # the block product with the half-work scale vector
    V = workloads.block(N, 8 if N > 1 else 1, seed=2)
    ctx.set_option("sym", 1)
    ctx.degree(beta, alpha)
    Y = ctx.apply(fd.to_colmajor(V, dev))
    ctx.synchronize()
    assert relF(Y.cpu().numpy(), dense.apply(X, beta, alpha, V)) <= TOL_APPLY
    ctx.close()


@pytest.mark.parametrize("alpha", [0.0, 0.5, 1.0])
def test_alpha(fd, dev, alpha):
    tc_case(fd, dev, workloads.torus6(1500, seed=4), 1.5, alpha, 32)


def test_fast_mode(fd, dev):
    err = tc_case(fd, dev, workloads.torus6(2000, seed=5), 2.0, 1.0, 64, prec=1)
    assert err > 1e-6            # it really is the reduced-precision path


# The reduced-precision mode has a kernel of its own (one row tile per CTA, three exponent buffers, tiles alternating
# between two pairs of warpgroups): the same edge shapes as the fp32-grade kernel, against the oracle at its 3e-3 bound.
@pytest.mark.parametrize("N", [1, 100, 128, 129, 257, 1000, 2304])
def test_fast_mode_row_and_column_tails(fd, dev, N):
    tc_case(fd, dev, workloads.torus6(N, seed=N), 2.0, 1.0, 64 if N > 1 else 1, prec=1)


@pytest.mark.parametrize("b", [1, 8, 16, 24, 32, 40, 64, 70, 128])
def test_fast_mode_block_widths(fd, dev, b):
    tc_case(fd, dev, workloads.torus6(900, seed=b), 1.0, 1.0, b, prec=1)


@pytest.mark.parametrize("D,beta", [(2, 3.0), (12, 2.0), (20, 1.0), (30, 1.0)])
def test_fast_mode_dimensions_and_k_slabs(fd, dev, D, beta):
    X = workloads.latent_torus(1200, seed=D, D=D) if D >= 13 else workloads.gaussian_cloud(1200, D, seed=D, scale=0.7)
    tc_case(fd, dev, X, beta, 1.0, 32, prec=1)


@pytest.mark.parametrize("opts", [{"flush": 1}, {"flush": 3}, {"flush": 64}, {"jt_chunk": 1}, {"jt_chunk": 2}, {"jt_chunk": 5, "flush": 2}])
def test_fast_mode_flush_groups_and_column_chunks(fd, dev, opts):
    # 3000 points = 24 column tiles: group and chunk tails, odd tile counts per chunk (the running tile index carries the
    # buffer and warpgroup rotation across work items), and run-to-run bit-reproducibility
    X = workloads.torus6(3000, seed=9)
    V = workloads.block(3000, 64, seed=2)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=64)
    ctx.set_option("path", fd.FD_PATH_TC)
    for k, v in opts.items():
        ctx.set_option(k, v)
    ctx.degree(2.0, 1.0)
    Vd = fd.to_colmajor(V, dev)
    Y1 = ctx.apply(Vd, prec=fd.FD_PREC_FAST).clone()
    Y2 = ctx.apply(Vd, prec=fd.FD_PREC_FAST)
    ctx.synchronize()
    assert torch.equal(Y1, Y2)
    assert relF(Y1.cpu().numpy(), dense.apply(X, 2.0, 1.0, V)) <= TOL_FAST
    ctx.close()


def test_c4_shape_reduced(fd, dev):
    tc_case(fd, dev, workloads.latent_torus(3000), 2.0, 1.0, 32)


@pytest.mark.parametrize("flush", [1, 2, 4, 8])
def test_flush_interval(fd, dev, flush):
    X = workloads.torus6(2304, seed=7)
    V = workloads.block(2304, 64, seed=2)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=64)
    ctx.set_option("path", fd.FD_PATH_TC)
    ctx.set_option("flush", flush)
    ctx.degree(2.0, 1.0)
    Y = ctx.apply(fd.to_colmajor(V, dev))
    ctx.synchronize()
    assert relF(Y.cpu().numpy(), dense.apply(X, 2.0, 1.0, V)) <= TOL_APPLY
    ctx.close()


def test_general_scalings_and_rectangular(fd, dev):
    X = workloads.torus6(1100, seed=5)
    Z = workloads.torus6(700, seed=6)
    N = 1100
    rng = np.random.default_rng(0)
    l = rng.uniform(0.5, 2.0, N).astype(np.float32)
    r = (rng.uniform(0.5, 2.0, N) * np.where(rng.uniform(size=N) < 0.3, -1, 1)).astype(np.float32)   # signs allowed
    lz = rng.uniform(0.5, 2.0, 700).astype(np.float32)
    V = workloads.block(N, 16, seed=4)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=16)
    ctx.set_option("path", fd.FD_PATH_TC)
    t = lambda a: torch.from_numpy(a).to(dev)
    Vd = fd.to_colmajor(V, dev)
    beta = 1.2
    Y = ctx.apply_general(beta, Vd, left=t(l), right=t(r)).cpu().numpy()
    assert relF(Y, dense.apply_general(X, beta, V, left=l, right=r)) <= TOL_APPLY
    Y = ctx.apply_general(beta, Vd, left=t(lz), right=t(r), Xrow=t(Z)).cpu().numpy()
    assert relF(Y, dense.apply_general(X, beta, V, left=lz, right=r, Xrow=Z)) <= TOL_APPLY
    q1 = ctx.apply_general(beta, None).cpu().numpy()[:, 0]
    assert np.abs(q1 / dense.degree(X, beta, 0.0)[0] - 1).max() <= TOL_DEG
    ctx.synchronize()
    # a zero column and a huge column in the same block (per-column scaling)
    V2 = V.copy(); V2[:, 3] = 0.0; V2[:, 5] *= 1e6; V2[:, 7] *= 1e-6
    Y = ctx.apply_general(beta, fd.to_colmajor(V2, dev)).cpu().numpy()
    Yo = dense.apply_general(X, beta, V2)
    for c in range(16):
        if c == 3:
            assert np.all(Y[:, c] == 0)
        else:
            assert relF(Y[:, c], Yo[:, c]) <= TOL_APPLY
    ctx.close()


def test_run_to_run_bit_reproducible(fd, dev):
    X = workloads.torus6(3000, seed=9)
    V = fd.to_colmajor(workloads.block(3000, 32, seed=1), dev)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=32)
    ctx.set_option("path", fd.FD_PATH_TC)
    ctx.degree(1.0, 1.0)
    a = ctx.apply(V).clone()
    b = ctx.apply(V).clone()
    ctx.synchronize()
    assert torch.equal(a, b)
    ctx.close()


def test_eigs_on_tensor_core_path(fd, dev):
    # same gates as the direct-difference path: eigenvalues 1e-6, residual certificate 5e-6
    from test_gpu_eigs import check_eigs, default_m_max
    X = workloads.torus6(3000)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=32, m_max=default_m_max(64, 32))
    ctx.set_option("path", fd.FD_PATH_TC)
    ctx.degree(0.5, 1.0)
    lam, U, info = ctx.eigs(64, 32, tol=1e-6, max_applies=600)
    check_eigs(lam, U.cpu().numpy(), X, 0.5, 1.0, 64)
    ctx.close()


def test_auto_path_selection(fd, dev):
    # small problems and shapes the Gram form cannot carry accurately are served by the direct-difference kernels
    Xs = workloads.torus6(2000, seed=1)
    ctx = fd.Context(torch.from_numpy(Xs).to(dev), b_max=16)
    ctx.degree(1.0, 1.0)
    ctx.apply(fd.to_colmajor(workloads.block(2000, 16), dev))
    assert ctx.get_option("last_path") == fd.FD_PATH_SIMT
    ctx.close()
    Xl = workloads.torus2(20000, seed=1)
    ctx = fd.Context(torch.from_numpy(Xl).to(dev), b_max=16)
    V = fd.to_colmajor(workloads.block(20000, 16), dev)
    ctx.degree(300.0, 1.0)                 # beta' max|x|^2 = 866: beyond the Gram-form budget
    ctx.apply(V)
    assert ctx.get_option("last_path") == fd.FD_PATH_SIMT
    ctx.degree(10.0, 1.0)
    ctx.apply(V)
    ctx.synchronize()
    assert ctx.get_option("last_path") == fd.FD_PATH_TC
    ctx.close()


def test_full_size_sampled_rows_and_identities(fd, dev):
    """Headline configuration (N = 2^20, D = 12, b = 64, beta = 2), the launch bench.py times: sampled rows against
    the oracle, plus properties that hold at any size (Perron identity, symmetry)."""
    N, b, beta = 1 << 20, 64, 2.0
    X = workloads.torus6(N, seed=42)
    V = workloads.block(N, b, seed=1)
    rows = workloads.row_sample(N, 96, seed=3)
    rng = np.random.default_rng(5)
    l = rng.uniform(0.5, 1.5, N).astype(np.float32) * 1e-3
    r = rng.uniform(0.5, 1.5, N).astype(np.float32) * 1e-3
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=b)
    q, d, s, so, so2 = ctx.degree(beta, 1.0)
    assert ctx.get_option("last_path") == fd.FD_PATH_TC
    qo, sq = blocked.rows_apply_general(X, beta, None, rows=rows, want_rowsq=True)
    assert np.abs(q.cpu().numpy()[rows] / qo[:, 0] - 1).max() <= TOL_DEG
    t = lambda a: torch.from_numpy(a).to(dev)
    Vd = fd.to_colmajor(V, dev)
    Y = ctx.apply_general(beta, Vd, left=t(l), right=t(r))
    ctx.synchronize()
    Yo = blocked.rows_apply_general(X, beta, V, rows=rows, left=l, right=r)
    assert relF(Y.cpu().numpy()[rows], Yo) <= TOL_APPLY
    # M sqrt(d) = sqrt(d)
    sd = torch.sqrt(d.double()).float()
    W = torch.empty((b, N), dtype=torch.float32, device=dev).t()
    W[:, 0] = sd
    W[:, 1:] = Vd[:, 1:]
    MW = ctx.apply(W)
    ctx.synchronize()
    assert float((MW[:, 0] - sd).abs().max() / sd.abs().max()) <= 2e-5
    # U^T (M V) = (M U)^T V on two column pairs
    MV = ctx.apply(Vd)
    ctx.synchronize()
    a = float((Vd[:, 2].double() * MV[:, 3].double()).sum())
    bb = float((MV[:, 2].double() * Vd[:, 3].double()).sum())
    scale = float(MV[:, 2].double().norm() * Vd[:, 3].double().norm())
    assert abs(a - bb) <= 1e-5 * scale
    ctx.close()


def test_bounded_wait_expires_cleanly_and_context_survives(fd, dev):
    # a wait on a barrier that nothing completes, with a 1 ms limit: the kernel returns, the status word reports it
    X = workloads.torus6(1024, seed=2)
    V = workloads.block(1024, 16, seed=1)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=16)
    ctx.set_option("path", fd.FD_PATH_TC)
    ctx.degree(1.0, 1.0)
    ctx.set_option("wait_selftest", 2.0e6)
    with pytest.raises(fd.FdError) as e:
        ctx.synchronize()
    assert e.value.status == fd.FD_ERR_TIMEOUT and "0x17f" in str(e.value)
    ctx.synchronize()                                  # reported once, then cleared
    Y = ctx.apply(fd.to_colmajor(V, dev))              # the context (and the GPU) are still fine
    ctx.synchronize()
    assert relF(Y.cpu().numpy(), dense.apply(X, 1.0, 1.0, V)) <= TOL_APPLY
    ctx.close()


def test_c4_full_size_sampled_rows(fd, dev):
    """C4 at full size (N = 262144, D = 30: three 16-wide K slabs): sampled rows of q and of the general product against
    the oracle; Perron identity of the normalised operator."""
    N, b, beta = 262144, 32, 2.0
    X = workloads.latent_torus(N, seed=42)
    V = workloads.block(N, b, seed=1)
    rows = workloads.row_sample(N, 64, seed=4)
    rng = np.random.default_rng(6)
    l = rng.uniform(0.5, 1.5, N).astype(np.float32) * 1e-3
    r = rng.uniform(0.5, 1.5, N).astype(np.float32) * 1e-3
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=b)
    q, d, s, so, so2 = ctx.degree(beta, 1.0)
    assert ctx.get_option("last_path") == fd.FD_PATH_TC
    qo = blocked.rows_apply_general(X, beta, None, rows=rows)
    assert np.abs(q.cpu().numpy()[rows] / qo[:, 0] - 1).max() <= TOL_DEG
    t = lambda a: torch.from_numpy(a).to(dev)
    Vd = fd.to_colmajor(V, dev)
    Y = ctx.apply_general(beta, Vd, left=t(l), right=t(r))
    ctx.synchronize()
    Yo = blocked.rows_apply_general(X, beta, V, rows=rows, left=l, right=r)
    assert relF(Y.cpu().numpy()[rows], Yo) <= TOL_APPLY
    sd = torch.sqrt(d.double()).float()
    W = torch.empty((b, N), dtype=torch.float32, device=dev).t()
    W[:, 0] = sd
    W[:, 1:] = Vd[:, 1:]
    MW = ctx.apply(W)
    ctx.synchronize()
    assert float((MW[:, 0] - sd).abs().max() / sd.abs().max()) <= 2e-5
    ctx.close()


def full_size_certificate(fd, dev, X, beta, k, b, m_max, min_converged, max_applies=400, sample=256):
    """Eigensolve at a benchmark configuration's full size, certified against the float64 oracle on sampled rows.

    No dense oracle is affordable at these sizes, so the gates are (a) the properties that hold at any size -- lambda_0 = 1
    (Perron pair, M sqrt(d) = sqrt(d)), eigenvalues in (0, 1] and descending, orthonormal vectors -- and (b) the residual
    certificate of every returned pair from the ORACLE: rows.c evaluates (M v - theta v)_i in float64, one pair at a time,
    on a seeded sample of rows, for all k + 1 vectors; |r| is estimated as sqrt(N / sample) |r_sample|.  For a symmetric
    operator an eigenvalue lies within the residual norm of theta, so a pair that passes IS an eigenpair to that accuracy.
    The scale vector s that defines M enters the oracle rows as computed on the GPU (all N values of it are needed; an
    exact s costs two full float64 N^2 passes); it is itself checked against oracle rows here, on the same sample."""
    from oracle import blocked
    N = X.shape[0]
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=b, m_max=m_max)
    q, d, s, so, so2 = ctx.degree(beta, 1.0)
    lam, U, info = ctx.eigs(k, b, tol=1e-6, max_applies=max_applies, allow_not_converged=True)
    print(f"N={N} k={k} b={b}: converged {info.converged}/{k + 1} after {info.applies} applies, max residual {info.max_residual:.2e}")
    assert info.converged >= min_converged
    assert info.max_residual <= 2.5e-6
    assert abs(lam[0] - 1.0) <= 1e-6
    assert np.all(np.diff(lam) <= 1e-9) and lam[-1] > 0 and lam[0] <= 1.0 + 1e-6
    G = (U.double().t() @ U.double()).cpu().numpy()
    assert np.abs(G - np.eye(k + 1)).max() <= 1e-5
    sd = torch.sqrt(d.double())
    sd = sd / sd.norm()
    assert float((U[:, 0].double().abs() - sd).abs().max()) <= 1e-4 * float(sd.max())
    # ---- oracle rows
    rows = workloads.row_sample(N, sample, seed=23)
    X64 = X.astype(np.float64)
    q64 = q.cpu().numpy().astype(np.float64)
    s64 = s.cpu().numpy().astype(np.float64)
    # s on the sampled rows from oracle rows of q and d (alpha = 1: d_i = q_i^-1 sum_j K_ij q_j^-1, s_i = q_i^-1 d_i^-1/2);
    # the column vector q^-1 is the GPU's, its sampled entries are checked against the oracle first
    q_rows = blocked.rows_apply_general(X64, beta, None, rows=rows)[:, 0]
    assert np.abs(q64[rows] / q_rows - 1).max() <= TOL_DEG
    d_rows = blocked.rows_apply_general(X64, beta, None, rows=rows, left=1.0 / q64, right=1.0 / q64)[:, 0]
    s_rows = 1.0 / (q_rows * np.sqrt(d_rows))
    assert np.abs(s64[rows] / s_rows - 1).max() <= TOL_DEG
    U64 = np.ascontiguousarray(U.cpu().numpy().astype(np.float64))
    MU = blocked.rows_apply_general(X64, beta, U64, rows=rows, left=s64, right=s64)
    R = MU - U64[rows] * lam[None, :]
    est = np.sqrt(N / float(sample)) * np.linalg.norm(R, axis=0)
    print(f"   oracle-row residual estimates: max {est.max():.2e}, median {np.median(est):.2e}")
    assert est.max() <= 7.5e-6, est.max()          # the 5e-6 certificate with room for the sampling error of 256 rows
    ctx.close()
    return lam, info


def test_c3_full_size_eigs_certificate(fd, dev):
    """C3 at full size: N = 131072, b = 32, k = 64, beta = 2."""
    full_size_certificate(fd, dev, workloads.torus6(131072, seed=42), 2.0, 64, 32, 192, min_converged=65)


def test_c4_full_size_eigs_certificate(fd, dev):
    """C4 at full size: N = 262144, D = 30 (tensor-core distance), b = 32, k = 32, beta = 2."""
    full_size_certificate(fd, dev, workloads.latent_torus(262144, seed=42), 2.0, 32, 32, 128, min_converged=33)


def test_c5_full_size_eigs_certificate(fd, dev):
    """C5 at full size: N = 2^20, b = 64, k = 128, beta = 2.  k = 128 cuts the third cluster of the 6-torus spectrum
    (multiplicities 1 + 12 + 60 = 73, then 160).  With the basis capacity the benchmark uses (3 (k + 1) + 2 b, rounded up to a
    multiple of b: the thick restart then keeps the rest of the cut cluster) all 129 pairs converge to tol = 1e-6 and pass
    the oracle-row certificate."""
    lam, info = full_size_certificate(fd, dev, workloads.torus6(1 << 20, seed=42), 2.0, 128, 64, 576, min_converged=129, sample=128)
    assert info.applies <= 80


def test_c5_full_size_minimum_capacity_is_a_reported_stall(fd, dev):
    """The same solve with the smallest capacity fd_eigs accepts (2 (k + 1) + b -> 384): the pairs inside the cut cluster
    stall just above tol at the fp32 operator's residual floor -- FD_ERR_NOT_CONVERGED is a reported outcome, and every
    returned pair still passes the oracle-row certificate (N = 2^18 level of the same draw keeps the test short).  The
    count the solver reports is the number of LEADING pairs below tol: the Perron pair and the first 12-fold cluster at
    least."""
    X = workloads.torus6(1 << 18, seed=42)
    lam, info = full_size_certificate(fd, dev, X, 2.0, 128, 64, 384, min_converged=13, sample=128, max_applies=200)
    assert info.converged < 129


@pytest.mark.parametrize("beta", [10.0, 30.0])
def test_c2_full_size_eigs_certificate(fd, dev, beta):
    """C2 at full size: N = 16384, D = 4, b = 16, k = 32; beta = 10 runs on the Gram-form kernels, beta = 30 on the
    direct-difference kernels (automatic choice)."""
    full_size_certificate(fd, dev, workloads.torus2(16384, seed=42), beta, 32, 16, 144, min_converged=33)
