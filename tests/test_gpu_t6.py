"""T^6 validation sweep on the GPU (Sec. 3, Fig. 1(b) and 1(c)): paper radii, alpha = 1/2, k = 3 nontrivial pairs, the
in-loop bandwidth flow from beta_0 of Eq. 7, and the post-hoc first-harmonic overlap of the leading doublet with the
largest circle.  Exact parity is GPU flow vs oracle flow on the same points (sizes the dense oracle finishes); the
printed table (another RNG, mean and spread over repeats) is a soft pin of trend and range."""
import csv
import os

import numpy as np
import pytest
import torch

import workloads
from oracle import dense, flow, overlap

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "t6_bandwidth_table.txt")


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


def table():
    with open(GOLDEN) as f:
        rows = [r for r in csv.reader(l for l in f if not l.startswith("#"))]
    return {int(r[0]): tuple(float(v) for v in r[1:]) for r in rows[1:]}


def gpu_run(fd, dev, N, seed):
    X, ang = workloads.torus6_paper(N, seed=seed, return_angles=True)
    ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=8, m_max=64)
    bx, status, lam, U, recs = ctx.beta_flow(3, 8, 0.5, beta_start=0.0, beta_max=1000.0)
    psi = ctx.scale_by_degree(U, -0.5).cpu().numpy()              # Markov modes d^-1/2 v (end of Sec. 2.3)
    path = ctx.get_option("last_path")
    ctx.close()
    score = overlap.rv_overlap(psi[:, 1:3], overlap.first_harmonic_target(ang, 5))
    return X, ang, bx, status, lam, psi, recs, score, path


@pytest.mark.parametrize("N", [1024, 2048])
def test_flow_and_overlap_match_oracle(fd, dev, N):
    X, ang, bx, status, lam, psi, recs, score, path = gpu_run(fd, dev, N, 42)
    bx_o, status_o, log_o = flow.beta_flow(flow.dense_probe(X, 0.5, 3), N, flow.beta0(X), 1000.0)
    assert status == status_o == "VERTEX"
    assert [r["beta"] for r in recs] == pytest.approx([r["beta"] for r in log_o], rel=1e-6)
    for r, ro in zip(recs, log_o):
        assert r["V"] == pytest.approx(ro["V"], rel=1e-4)
    assert bx == pytest.approx(bx_o, rel=1e-3)
    lam_o, U_o, d_o = dense.eigs(X, bx_o, 0.5, 3)
    assert np.abs(lam - lam_o).max() <= 2e-6          # (beta_x itself differs by up to 1e-3 relative)
    score_o = overlap.rv_overlap(dense.markov_vectors(U_o, d_o)[:, 1:3], overlap.first_harmonic_target(ang, 5))
    assert score == pytest.approx(score_o, abs=2e-4)


def test_sweep_follows_the_printed_table(fd, dev):
    tab = table()
    sizes = [1 << e for e in range(10, 18)]            # 2^10 ... 2^17 (direct-difference kernels below 2^14, Gram-form above)
    res = {}
    for N in sizes:
        seeds = (42, 43, 44) if N <= 16384 else (42,)
        runs = [gpu_run(fd, dev, N, s) for s in seeds]
        assert all(r[3] == "VERTEX" for r in runs)
        res[N] = (float(np.mean([r[2] for r in runs])), float(np.mean([r[7] for r in runs])), runs[0][8])
    assert res[1024][2] == fd.FD_PATH_SIMT and res[1 << 17][2] == fd.FD_PATH_TC
    for N in sizes:
        bx, score, _ = res[N]
        mean, std, ov, ov_std = tab[N]
        # range: the printed value is a mean over repeats of another RNG; this reading sits 10-20 % below it at small N
        spread = std if std > 0 else 0.25 * mean
        assert abs(bx - mean) <= 3.0 * spread + 0.05 * mean, (N, bx, mean)
        assert (1.0 - ov) / 3.0 <= 1.0 - score <= (1.0 - ov) * 3.0, (N, score, ov)
    # where the paper prints a single run (N = 2^17: no averaging over repeats) the flow lands on its bandwidth to 1 % and on
    # its first-harmonic error to 20 %: the closest thing to a hard pin of the flow's reading that the paper offers
    assert abs(res[1 << 17][0] / tab[1 << 17][0] - 1.0) < 0.01
    assert abs((1.0 - res[1 << 17][1]) / (1.0 - tab[1 << 17][2]) - 1.0) < 0.2
    # trend: the selected bandwidth grows with N up to 2^16, as in the printed table (which then drops at 2^17)
    bxs = [res[N][0] for N in sizes]
    assert all(b1 > b0 for b0, b1 in zip(bxs[:6], bxs[1:7]))
    # trend: the first-harmonic error falls by more than an order of magnitude from 2^10 to 2^17
    assert (1.0 - res[1 << 17][1]) < 0.1 * (1.0 - res[1024][1])


@pytest.mark.parametrize("log2n", [18, 19])
def test_larger_sizes_match_the_printed_single_runs(fd, dev, log2n):
    """N = 2^18 and 2^19: the paper prints one run each (seed 42, another RNG); the selected bandwidth must match to 1 % and the
    first-harmonic error to 30 % (measured: 0.2 % / 0.03 % and 11 % / 12 %)."""
    N = 1 << log2n
    tab = table()
    X, ang, bx, status, lam, psi, recs, score, path = gpu_run(fd, dev, N, 42)
    assert status == "VERTEX" and path == fd.FD_PATH_TC
    assert abs(bx / tab[N][0] - 1.0) < 0.01, (bx, tab[N][0])
    assert abs((1.0 - score) / (1.0 - tab[N][2]) - 1.0) < 0.3, (1.0 - score, 1.0 - tab[N][2])
