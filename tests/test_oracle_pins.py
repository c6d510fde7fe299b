"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test names the statement it checks; together they are chosen so that a dropped
term, wrong sign, wrong exponent of q or d, or a transposed operand fails one of them.
"""
import csv
import math
import os

import numpy as np
import pytest
from scipy.special import ive

import workloads
from oracle import blocked, dense, flow, nystrom


# ----------------------------------------------------------------------------- Eq. 1
def test_kernel_symmetric_unit_diagonal_psd():
    X = workloads.gaussian_cloud(60, 3, seed=3)
    K = dense.kernel(X, 0.7)
    assert np.array_equal(K, K.T)
    assert np.all(np.diag(K) == 1.0)
    w = np.linalg.eigvalsh(K)
    assert w.min() >= -1e-12 * len(X)          # a Gaussian Gram matrix is PSD (App. A)
    assert np.all((K > 0) & (K <= 1))


def test_kernel_entry_brute_force_and_rectangular_orientation():
    X = workloads.gaussian_cloud(7, 5, seed=1).astype(np.float64)
    Z = workloads.gaussian_cloud(4, 5, seed=2).astype(np.float64)
    K = dense.kernel(Z, 1.3, X)                # rows index Z, columns index X
    assert K.shape == (4, 7)
    for i in range(4):
        for j in range(7):
            h = sum((Z[i, k] - X[j, k]) ** 2 for k in range(5))
            assert K[i, j] == pytest.approx(math.exp(-1.3 * h), rel=1e-14)


def test_kernel_doubling_identity():
    # K(2 beta) = K(beta) squared elementwise (Sec. 2.3)
    X = workloads.torus2(50, seed=5)
    assert np.allclose(dense.kernel(X, 2 * 3.1), dense.kernel(X, 3.1) ** 2, rtol=1e-13, atol=0)
    q, d, s, so, so2 = dense.degree(X, 3.1, 1.0)
    K = dense.kernel(X, 3.1)
    assert so == pytest.approx(K.sum() - len(X), rel=1e-13)
    assert so2 == pytest.approx((K * K).sum() - len(X), rel=1e-12)


# ----------------------------------------------------------------------------- Eq. 2
@pytest.mark.parametrize("alpha", [0.0, 0.5, 1.0])
def test_markov_and_symmetric_operator(alpha):
    X = workloads.latent_torus(80, seed=4)
    K = dense.kernel(X, 0.9)
    q, d, s = dense.normalisation(K, alpha)
    P = dense.markov(K, alpha)
    M = dense.symmetric_operator(K, alpha)
    assert np.allclose(P.sum(axis=1), 1.0, atol=1e-13)              # row-stochastic
    assert np.allclose(M, M.T, atol=1e-15)
    # M = D^1/2 P D^-1/2 (Eq. 2), entry by entry
    assert np.allclose(M, np.sqrt(d)[:, None] * P / np.sqrt(d)[None, :], atol=1e-14)
    # same spectrum, Perron value 1 with known vector sqrt(d)
    wP = np.sort(np.linalg.eigvals(P).real)
    wM = np.linalg.eigvalsh(M)
    assert np.allclose(wP, wM, atol=1e-10)
    assert np.allclose(M @ np.sqrt(d), np.sqrt(d), atol=1e-13)
    assert wM.max() == pytest.approx(1.0, abs=1e-12) and wM.min() >= -1e-12
    if alpha == 0.0:
        assert np.allclose(d, q)


def test_normalisation_three_points_by_hand():
    # scalar arithmetic, no arrays: catches a wrong power of q or d
    x = np.array([[0.0], [1.0], [3.0]], dtype=np.float32)
    beta, alpha = 0.25, 1.0
    a, b, c = math.exp(-beta * 1), math.exp(-beta * 9), math.exp(-beta * 4)
    q = [1 + a + b, a + 1 + c, b + c + 1]
    Ka = [[1 / q[0] ** 2, a / (q[0] * q[1]), b / (q[0] * q[2])],
          [a / (q[1] * q[0]), 1 / q[1] ** 2, c / (q[1] * q[2])],
          [b / (q[2] * q[0]), c / (q[2] * q[1]), 1 / q[2] ** 2]]
    d = [sum(r) for r in Ka]
    s = [1 / (q[i] * math.sqrt(d[i])) for i in range(3)]
    qo, do, so, _, _ = dense.degree(x, beta, alpha)
    assert np.allclose(qo, q, rtol=1e-14) and np.allclose(do, d, rtol=1e-14) and np.allclose(so, s, rtol=1e-14)
    # alpha = 1/2 changes d: d_i = q_i^-1/2 sum_j K_ij q_j^-1/2
    _, dh, sh, _, _ = dense.degree(x, beta, 0.5)
    Kmat = [[1, a, b], [a, 1, c], [b, c, 1]]
    d_half = [sum(Kmat[i][j] / math.sqrt(q[i] * q[j]) for j in range(3)) for i in range(3)]
    assert np.allclose(dh, d_half, rtol=1e-14)
    assert np.allclose(sh, [q[i] ** -0.5 * d_half[i] ** -0.5 for i in range(3)], rtol=1e-14)


def test_rank_one_limit():
    # beta -> 0: K -> 1 1^T, M -> (1/N) 1 1^T, nontrivial spectrum collapses, V_bias -> infinity (Sec. 2.3)
    X = workloads.torus2(40, seed=2)
    lam, U, d = dense.eigs(X, 1e-9, 1.0, 5)
    assert lam[0] == pytest.approx(1.0, abs=1e-12)
    assert np.all(np.abs(lam[1:]) < 1e-7)
    M = dense.symmetric_operator(dense.kernel(X, 1e-9), 1.0)
    assert np.allclose(M, 1.0 / 40, atol=1e-8)
    big = dense.eigs(X, 1e-3, 1.0, 5)[0]
    small = dense.eigs(X, 1e-5, 1.0, 5)[0]
    assert flow.v_bias(small) > flow.v_bias(big) > 5.0


# ----------------------------------------------------------------------------- closed forms
@pytest.mark.parametrize("alpha", [0.0, 0.5, 1.0])
def test_two_points_and_simplex(alpha):
    beta, ell = 0.8, 1.7
    e = math.exp(-beta * ell * ell)
    X2 = np.array([[0.0, 0.0], [ell, 0.0]], dtype=np.float64)
    lam, _, _ = dense.eigs(X2, beta, alpha, 1)
    assert lam[0] == pytest.approx(1.0, abs=1e-14)
    assert lam[1] == pytest.approx((1 - e) / (1 + e), rel=1e-13)
    n = 6                                           # regular simplex: scaled unit vectors in R^6
    Xs = np.eye(n) * (ell / math.sqrt(2.0))
    lam, _, _ = dense.eigs(Xs, beta, alpha, n - 1)
    assert lam[0] == pytest.approx(1.0, abs=1e-14)
    assert np.allclose(lam[1:], (1 - e) / (1 + (n - 1) * e), rtol=1e-12)


def _circle_closed_form(N, beta, m_max):
    j = np.arange(N)
    c = np.exp(-4.0 * beta * np.sin(np.pi * j / N) ** 2)      # chord^2 = 4 sin^2(pi j / N)
    f = np.fft.fft(c).real
    return f[: m_max + 1] / f[0], f[0]


@pytest.mark.parametrize("alpha", [0.0, 0.5, 1.0])
def test_circle_closed_form(alpha):
    # Config C1 at reduced N for the dense solve; K is circulant, q is constant, M = K / q_0 for every alpha.
    N, beta, k = 512, 200.0, 8
    X = workloads.circle(N)
    lam, U, d = dense.eigs(X, beta, alpha, k)
    dft, q0 = _circle_closed_form(N, beta, 4)
    expect = np.array([dft[0]] + [dft[m] for m in (1, 1, 2, 2, 3, 3, 4, 4)])
    assert np.allclose(lam, expect, rtol=0, atol=2e-7)         # float32-rounded coordinates move lambda by ~1e-8
    q = dense.degree(X, beta, alpha)[0]
    assert np.allclose(q, q0, rtol=1e-6)
    # Bessel-ratio form I_m(2 beta) / I_0(2 beta) (aliasing is negligible at this N, beta)
    bessel = np.array([ive(m, 2 * beta) / ive(0, 2 * beta) for m in range(5)])
    assert np.allclose(dft, bessel, rtol=0, atol=1e-12)
    # eigenvectors: doublet m spans {cos m theta, sin m theta}
    th = 2 * np.pi * np.arange(N) / N
    for m in (1, 2, 3, 4):
        span = np.stack([np.cos(m * th), np.sin(m * th)], axis=1)
        ang = dense.principal_angles(U[:, 2 * m - 1: 2 * m + 1], span)
        assert ang.max() < 1e-5


def test_circle_full_size_values():
    # C1 itself (N = 2048, beta = 200): closed form only (the dense solve is covered at N = 512).
    dft, q0 = _circle_closed_form(2048, 200.0, 5)
    bessel = np.array([ive(m, 400.0) / ive(0, 400.0) for m in range(6)])
    assert np.allclose(dft, bessel, atol=1e-13)
    assert q0 == pytest.approx(2048 * ive(0, 400.0), rel=1e-12)       # q_0 = sum_j exp(-2b(1-cos)) ~ N e^-2b I_0(2b)
    X = workloads.circle(2048)
    q, sq = blocked.rows_apply_general(X, 200.0, None, rows=[0, 5, 1000], want_rowsq=True)
    assert np.allclose(q[:, 0], q0, rtol=1e-6)


def test_lattice_torus_kronecker_spectrum():
    # equispaced N1 x N2 lattice: K = K1 (x) K2, eigenvalues are products of circle eigenvalues
    N1, N2, beta = 24, 20, 10.0
    X = workloads.torus_grid(N1, N2)
    lam, _, _ = dense.eigs(X, beta, 1.0, 40)
    l1, _ = _circle_closed_form(N1, beta, N1 - 1)
    l2, _ = _circle_closed_form(N2, beta, N2 - 1)
    full = np.sort(np.outer(np.fft.fft(np.exp(-4 * beta * np.sin(np.pi * np.arange(N1) / N1) ** 2)).real,
                            np.fft.fft(np.exp(-4 * beta * np.sin(np.pi * np.arange(N2) / N2) ** 2)).real).ravel())[::-1]
    full = full / full[0]
    assert np.allclose(lam, full[:41], atol=3e-7)
    assert l1[0] == 1.0 and l2[0] == 1.0


# ----------------------------------------------------------------------------- Eq. 3, blocked path
def test_apply_matches_brute_force_loops():
    X = workloads.gaussian_cloud(9, 3, seed=8).astype(np.float64)
    V = np.asarray(workloads.block(9, 2, seed=3), dtype=np.float64)
    beta, alpha = 0.6, 0.5
    q, d, s, _, _ = dense.degree(X, beta, alpha)
    Y = dense.apply(X, beta, alpha, V)
    for i in range(9):
        for c in range(2):
            acc = 0.0
            for j in range(9):
                h = sum((X[i, k] - X[j, k]) ** 2 for k in range(3))
                acc += s[i] * math.exp(-beta * h) * s[j] * V[j, c]
            assert Y[i, c] == pytest.approx(acc, rel=1e-12, abs=1e-15)


def test_blocked_and_rows_c_match_dense():
    X = workloads.torus6(700, seed=9)
    V = workloads.block(700, 5, seed=2)
    beta, alpha = 1.5, 1.0
    qd, dd, sd, so, so2 = dense.degree(X, beta, alpha)
    qb, db, sb, sob, so2b = blocked.degree(X, beta, alpha)
    assert np.allclose(qb, qd, rtol=1e-12) and np.allclose(db, dd, rtol=1e-12) and np.allclose(sb, sd, rtol=1e-12)
    assert sob == pytest.approx(so, rel=1e-12) and so2b == pytest.approx(so2, rel=1e-12)
    Yd = dense.apply(X, beta, alpha, V)
    assert np.allclose(blocked.apply(X, beta, alpha, V, s=sd), Yd, rtol=1e-11, atol=1e-14)
    rng = np.random.default_rng(0)
    l, r = rng.uniform(0.5, 2, 700), rng.uniform(0.5, 2, 700)
    Yg = dense.apply_general(X, beta, V, left=l, right=r)
    assert np.allclose(blocked.apply_general(X, beta, V, left=l, right=r, block=(96, 130)), Yg, rtol=1e-11, atol=1e-14)
    rows = workloads.row_sample(700, 33)
    assert np.allclose(blocked.rows_apply_general(X, beta, V, rows=rows, left=l, right=r), Yg[rows], rtol=1e-11, atol=1e-14)
    # rectangular: new rows against old columns
    Z = workloads.torus6(50, seed=10)
    Yr = dense.apply_general(X, beta, V, right=r, Xrow=Z)
    assert np.allclose(blocked.rows_apply_general(X, beta, V, right=r, Xrow=Z), Yr, rtol=1e-11, atol=1e-14)


def test_apply_properties():
    X = workloads.torus2(300, seed=6)
    beta, alpha = 8.0, 1.0
    q = dense.degree(X, beta, alpha)[0]
    ones = np.ones((300, 1))
    assert np.allclose(dense.apply_general(X, beta, ones)[:, 0], q, rtol=1e-14)      # K 1 = q
    U = np.asarray(workloads.block(300, 3, seed=4), dtype=np.float64)
    V = np.asarray(workloads.block(300, 3, seed=5), dtype=np.float64)
    assert np.allclose(U.T @ dense.apply(X, beta, alpha, V), dense.apply(X, beta, alpha, U).T @ V, atol=1e-12)
    # rigid motion and permutation invariance
    rot, _ = np.linalg.qr(np.random.default_rng(1).standard_normal((4, 4)))
    X2 = X.astype(np.float64) @ rot + 3.0
    assert np.allclose(dense.apply(X2, beta, alpha, V), dense.apply(X, beta, alpha, V), atol=1e-12)
    p = np.random.default_rng(2).permutation(300)
    assert np.allclose(dense.apply(X[p], beta, alpha, V[p]), dense.apply(X, beta, alpha, V)[p], atol=1e-13)


def test_eigs_certified_matches_dense():
    X = workloads.torus6(900, seed=12)
    lam, U, d = dense.eigs(X, 0.5, 1.0, 12)
    lam2, U2, d2, res = blocked.eigs_certified(X, 0.5, 1.0, 12, tol=1e-11)
    assert res.max() < 1e-8
    assert np.allclose(lam2, lam, atol=1e-9)
    assert np.allclose(d2, d, rtol=1e-12)


# ----------------------------------------------------------------------------- Eqs. 7-14
def test_constants_match_paper(golden_dir):
    rows = {}
    with open(os.path.join(golden_dir, "constants.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, val, _ = line.strip().split(",", 2)
            rows[name] = float(val)
    assert flow.BETA0_CAP == rows["beta0_cap"]
    assert flow.P_EXPONENT == rows["p_exponent"] and flow.KAPPA_P == rows["kappa_P"]
    assert flow.ETA["bf16"] == rows["eta_bf16"] and flow.ETA["tf32"] == rows["eta_tf32"]
    assert flow.ETA["fp32"] == rows["eta_fp32"] and flow.ETA["fp64"] == rows["eta_fp64"]


def test_beta0():
    # identity used by Eq. 7: E_ij |x_i - x_j|^2 = 2 E_i |x_i - mu|^2, so 1/(2 mean|x-mu|^2) = 1/mean pairwise sqdist
    X = workloads.gaussian_cloud(200, 3, seed=5, scale=3.0) + 7.0
    H = dense.sqdist(X)
    assert flow.beta0(X) == pytest.approx(1.0 / H.mean(), rel=1e-9)
    assert flow.beta0(X) < 0.1
    assert flow.beta0(workloads.gaussian_cloud(200, 3, seed=5, scale=0.1)) == 0.1     # cap
    assert flow.beta0(workloads.circle(64)) == 0.1                                    # 1/(2*1) = 0.5 -> capped


def test_neff_equal_weights_and_dhat():
    # k equally weighted interactions per row: S_off(beta) = N k w, S_off(2 beta) = N k w^2 -> n_eff = k (Eq. 9)
    N, k, w = 1000, 17, 0.3
    assert flow.n_eff(N * k * w, N * k * w * w, N) == pytest.approx(k, rel=1e-14)
    # S_off ~ beta^(-d/2) => d_hat = d (Eq. 14)
    assert flow.d_hat(5.0 * 3.0 ** -3.0, 5.0 * 6.0 ** -3.0) == pytest.approx(6.0, rel=1e-12)


def test_potential_terms_by_hand():
    lam = np.array([1.0, 0.9, 0.8, 0.5, 0.25])
    vb = flow.v_bias(lam)
    assert vb == pytest.approx(0.5 * (-math.log(0.8) - math.log(0.5)), rel=1e-14)     # even k: mean of middle two
    assert flow.v_bias(lam[:4]) == pytest.approx(-math.log(0.8), rel=1e-14)
    assert flow.perron_gap(lam) == pytest.approx(0.1, rel=1e-12)
    assert flow.v_mach(0.1) == pytest.approx((10 * 1e-7 / 0.1) ** 6, rel=1e-12)
    assert flow.admissible(1.1e-6) and not flow.admissible(1e-6)
    p = flow.potential(lam, 400.0, 100.0, 10)
    assert p["n_eff"] == pytest.approx(160.0) and p["V_stat"] == pytest.approx(1 / math.sqrt(160.0 * vb))
    assert p["V"] == pytest.approx(p["V_bias"] + p["V_stat"] + p["V_mach"])


def test_flow_bracket_vertex_and_edges():
    # synthetic probe whose potential is an exact parabola in log beta with minimum at beta = 3
    def make(lam1_of_beta, so):
        def probe(beta):
            return np.array([1.0, lam1_of_beta(beta)]), so(beta), so(2 * beta)
        return probe
    so = lambda b: 1e6 * b ** -3.0                       # n_eff = 1e6 * 2^3 / (N b^3)
    probe = make(lambda b: math.exp(-1.0 / b), so)       # V_bias = 1/beta (falls), V_stat rises
    bx, status, log = flow.beta_flow(probe, N=1000, beta_start=0.25, beta_max=1000.0)
    assert status == "VERTEX"
    V = lambda b: 1 / b + 1 / math.sqrt(8e3 * b ** -3.0 / b)      # V_bias + V_stat, V_mach negligible
    grid = [0.25 * 2 ** j for j in range(12)]
    jmin = int(np.argmin([V(b) for b in grid]))
    assert [r["beta"] for r in log[-4:-1]] == grid[jmin - 1: jmin + 2]
    assert grid[jmin - 1] <= bx <= grid[jmin + 1]
    true_min = min(np.exp(np.linspace(np.log(grid[jmin - 1]), np.log(grid[jmin + 1]), 20001)), key=V)
    assert abs(math.log(bx / true_min)) < 0.1
    # Perron wall before a bracket
    so_big = lambda b: 1e9 * b ** -3.0                   # pushes the V_bias + V_stat minimum out to beta ~ 11

    def probe_w(beta):                                   # Perron gap 1e-3 / beta^4 closes at beta = 8 first
        return np.array([1.0, 1.0 - 1e-3 / beta ** 4, math.exp(-1.0 / beta), math.exp(-2.0 / beta)]), \
            so_big(beta), so_big(2 * beta)
    bx, status, log = flow.beta_flow(probe_w, 1000, 1.0, 1000.0)
    assert status == "PERRON_WALL" and log[-1].get("wall") and log[-1]["beta"] == 8.0 and bx == 4.0
    # V rising at once
    bx, status, log = flow.beta_flow(make(lambda b: math.exp(-1.0 / b), so), 1000, 64.0, 1000.0)
    assert status == "LEFT_EDGE" and bx == 64.0
    # grid exhausted while falling
    bx, status, log = flow.beta_flow(probe, 1000, 0.25, 1.0)
    assert status == "RIGHT_EDGE" and bx == 1.0


def test_flow_soft_pin_against_printed_table(golden_dir):
    # Paper's T^6 run at N = 1024 (alpha = 1/2, k = 3): printed beta_x = 0.369 +/- 0.040.  Different RNG, so
    # only the trend is pinned: same order of magnitude and within 3 sigma-ish of the printed value.
    with open(os.path.join(golden_dir, "t6_bandwidth_table.txt")) as f:
        rows = [r for r in csv.reader(l for l in f if not l.startswith("#"))]
    table = {int(r[0]): (float(r[1]), float(r[2])) for r in rows[1:]}
    X = workloads.torus6_paper(1024, seed=42)
    b0 = flow.beta0(X)
    assert b0 == pytest.approx(1.0 / (2.0 * sum(r * r for r in workloads.PAPER_T6_RADII)), rel=0.02)
    bx, status, log = flow.beta_flow(flow.dense_probe(X, 0.5, 3), 1024, b0, 1000.0)
    assert status == "VERTEX"
    mean, std = table[1024]
    assert abs(bx - mean) < 3.0 * std + 0.05 * mean
    dh = [r["d_hat"] for r in log if abs(r["beta"] - bx) < 1e-12][0]
    assert 4.0 < dh < 9.0                     # intrinsic dimension 6, finite-sample estimate


# ----------------------------------------------------------------------------- Nystrom
def test_nystrom_reproduces_sample_values():
    X = workloads.torus6(400, seed=3)
    beta, alpha, k = 0.6, 1.0, 6
    lam, U, d = dense.eigs(X, beta, alpha, k)
    psi = dense.markov_vectors(U, d)
    q = dense.degree(X, beta, alpha)[0]
    ext = nystrom.extend(X, q, alpha, beta, psi, lam, X[:37])
    assert np.allclose(ext, psi[:37], atol=1e-12)
    # a genuinely new point close to a sample point gets a close value
    Z = X[:5].astype(np.float64) + 1e-6
    assert np.allclose(nystrom.extend(X, q, alpha, beta, psi, lam, Z), psi[:5], atol=1e-4)


def test_t6_continuum_clusters_soft():
    # unit 6-torus, continuum estimate: first cluster near I_1(2b)/I_0(2b) (x12), second near its square (x60)
    N, beta = 2500, 0.5
    X = workloads.torus6(N, seed=42, sigma=0.0)
    lam, _, _ = dense.eigs(X, beta, 1.0, 12)
    r1 = ive(1, 2 * beta) / ive(0, 2 * beta)
    assert abs(np.mean(lam[1:13]) / r1 - 1.0) < 0.15


# ------------------------------------------------------------------ the checker behind every angle gate
@pytest.mark.parametrize("t", [1e-6, 1e-3, 0.3, 1.2])
def test_principal_angles_known_single_angle(t):
    # span{e1} against span{cos t e1 + sin t e2}: the one principal angle is t (textbook definition)
    n = 50
    A = np.zeros((n, 1)); A[0, 0] = 1.0
    B = np.zeros((n, 1)); B[0, 0] = np.cos(t); B[1, 0] = np.sin(t)
    ang = dense.principal_angles(A, B)
    assert ang.shape == (1,)
    assert ang[0] == pytest.approx(t, rel=1e-9, abs=1e-15)
    # symmetric in its arguments, and insensitive to column scaling and sign
    assert dense.principal_angles(B, A)[0] == pytest.approx(t, rel=1e-9, abs=1e-15)
    assert dense.principal_angles(-3.0 * A, 0.25 * B)[0] == pytest.approx(t, rel=1e-9, abs=1e-15)


def test_principal_angles_two_distinct_angles_and_nonorthonormal_columns():
    # planes span{e1, e2} and span{c1 e1 + s1 e3, c2 e2 + s2 e4}: principal angles are exactly (t1, t2), ascending
    n, t1, t2 = 12, 2e-4, 0.7
    A = np.zeros((n, 2)); A[0, 0] = 1.0; A[1, 1] = 1.0
    B = np.zeros((n, 2))
    B[0, 0] = np.cos(t1); B[2, 0] = np.sin(t1)
    B[1, 1] = np.cos(t2); B[3, 1] = np.sin(t2)
    ang = dense.principal_angles(A, B)
    assert np.allclose(ang, [t1, t2], rtol=1e-9, atol=1e-15)
    # the same two planes given by skewed, unnormalised bases and after a common rotation of the ambient space
    rng = np.random.default_rng(7)
    Ta = np.array([[2.0, 1.5], [0.3, -0.7]]); Tb = np.array([[0.1, 4.0], [1.0, 1.0]])
    Qrot, _ = np.linalg.qr(rng.standard_normal((n, n)))
    ang2 = dense.principal_angles(Qrot @ (A @ Ta), Qrot @ (B @ Tb))
    assert np.allclose(ang2, [t1, t2], rtol=1e-7, atol=1e-13)
    # identical spans: zero; orthogonal spans: pi / 2
    assert dense.principal_angles(A, A @ Ta).max() < 1e-12
    C = np.zeros((n, 2)); C[4, 0] = 1.0; C[5, 1] = 1.0
    assert np.allclose(dense.principal_angles(A, C), [np.pi / 2, np.pi / 2])


# ------------------------------------------------------------------ the T^6 validation score (Sec. 3, Fig. 1(c))
def test_rv_overlap_closed_forms():
    from oracle import overlap
    rng = np.random.default_rng(3)
    n = 4000
    # three exactly orthonormal, exactly centred directions (discrete Fourier modes on n points)
    t = 2.0 * np.pi * np.arange(n) / n
    c1, s1, c2, s2 = np.cos(t), np.sin(t), np.cos(2 * t), np.sin(2 * t)
    B = np.stack([c1, s1], axis=1)
    # identical span, any basis of it, any offset: 1
    T = np.array([[2.0, -0.7], [0.4, 1.3]])
    assert overlap.rv_overlap(B @ T + 5.0, B) == pytest.approx(1.0, abs=1e-12)
    # orthogonal span: 0
    assert overlap.rv_overlap(np.stack([c2, s2], axis=1), B) == pytest.approx(0.0, abs=1e-12)
    # one shared direction of two: 1/2
    assert overlap.rv_overlap(np.stack([c1, c2], axis=1), B) == pytest.approx(0.5, abs=1e-12)
    # both directions tilted by known angles out of the span: (cos^2 a + cos^2 b) / 2
    a, b = 0.3, 1.1
    A = np.stack([np.cos(a) * c1 + np.sin(a) * c2, np.cos(b) * s1 + np.sin(b) * s2], axis=1)
    assert overlap.rv_overlap(A, B) == pytest.approx((np.cos(a) ** 2 + np.cos(b) ** 2) / 2.0, abs=1e-12)
    # symmetric in its arguments; invariant under a rotation inside the doublet (the degenerate pair may rotate)
    R = np.array([[np.cos(0.9), -np.sin(0.9)], [np.sin(0.9), np.cos(0.9)]])
    assert overlap.rv_overlap(B, A) == pytest.approx(overlap.rv_overlap(A, B @ R), abs=1e-12)
    # random data: strictly between 0 and 1
    v = overlap.rv_overlap(rng.standard_normal((n, 2)), B)
    assert 0.0 <= v < 0.01
    assert np.allclose(overlap.first_harmonic_target(np.stack([t] * 6, axis=1), 5), B)


def test_t6_first_harmonic_overlap_soft_pin(golden_dir):
    # Paper's T^6 run at N = 1024: printed overlap 0.929 (another RNG): the oracle flow's leading doublet must score in the
    # same range (1 - overlap within a factor of three of the printed 0.071) against the largest circle, and far lower
    # against any other circle
    from oracle import overlap
    X, ang = workloads.torus6_paper(1024, seed=42, return_angles=True)
    bx, status, log = flow.beta_flow(flow.dense_probe(X, 0.5, 3), 1024, flow.beta0(X), 1000.0)
    lam, U, d = dense.eigs(X, bx, 0.5, 3)
    psi = dense.markov_vectors(U, d)
    score = overlap.rv_overlap(psi[:, 1:3], overlap.first_harmonic_target(ang, 5))
    assert 0.071 / 3.0 < 1.0 - score < 0.071 * 3.0
    assert overlap.rv_overlap(psi[:, 1:3], overlap.first_harmonic_target(ang, 0)) < 0.2


def test_precision_cascade_by_hand():
    # V_bias = 1 / beta, V_stat as in the bracket test (minimum of V_bias + V_stat near beta = 3), and a Perron gap
    # g_P = 0.05 / beta that the coarse data type (eta = 1e-3: wall at g_P <= 1e-2, Eq. 12) loses at beta = 8 while fp32
    # (eta = 1e-7) never does.  Stage 1 from beta = 0.25: its V_mach = (10 eta / g_P)^6 = (beta / 5)^6 moves the
    # minimum to smaller beta; stage 2 must restart one grid step below stage 1's selection and find the fp32 vertex.
    so = lambda b: 1e6 * b ** -3.0

    def probe(beta):
        return np.array([1.0, 1.0 - 0.05 / beta, math.exp(-1.0 / beta) * (1.0 - 0.05 / beta)]), so(beta), so(2 * beta)
    # single-stage runs with each eta
    bx_c, st_c, log_c = flow.beta_flow(probe, 1000, 0.25, 1000.0, eta=1e-3)
    bx_f, st_f, log_f = flow.beta_flow(probe, 1000, 0.25, 1000.0, eta=1e-7)
    assert st_c == "VERTEX" and st_f == "VERTEX" and bx_c < bx_f
    bx, status, logs = flow.cascade([probe, probe], 1000, 0.25, 1000.0, [1e-3, 1e-7])
    assert len(logs) == 2 and status == "VERTEX"
    assert [r["beta"] for r in logs[0]] == [r["beta"] for r in log_c]                 # stage 1 = the coarse sweep
    assert logs[1][0]["beta"] == bx_c / 2.0                                           # stage 2 restarts one step below it
    assert [r["beta"] for r in logs[1][1:-1]] == [bx_c / 2.0 * 2 ** j for j in range(1, len(logs[1]) - 1)]
    # same potential, same fp32 minimum: the cascade's final vertex agrees with the fp32-only sweep's to the accuracy of
    # the three-point fit (different grid offsets)
    assert abs(math.log(bx / bx_f)) < 0.1
    assert all(r["V_mach"] < 1e-20 for r in logs[1])
    # a first stage that meets the wall hands on its last safe probe
    def probe_w(beta):
        return np.array([1.0, 1.0 - min(0.9, 0.05 / beta ** 3), math.exp(-1.0 / beta) * 0.09]), so(beta), so(2 * beta)
    bx1, st1, log1 = flow.beta_flow(probe_w, 1000, 0.25, 1000.0, eta=1e-3)
    assert st1 == "PERRON_WALL" and bx1 == 1.0 and log1[-1]["beta"] == 2.0           # 0.05 / 8 = 6.25e-3 <= 1e-2
    bx2, st2, logs2 = flow.cascade([probe_w, probe_w], 1000, 0.25, 1000.0, [1e-3, 1e-7])
    assert logs2[1][0]["beta"] == 0.5 and st2 == "VERTEX" and bx2 > 2.0
    # one stage = the plain flow
    bx3, st3, logs3 = flow.cascade([probe], 1000, 0.25, 1000.0, [1e-7])
    assert (bx3, st3) == (bx_f, st_f)
