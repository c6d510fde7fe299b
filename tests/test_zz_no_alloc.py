"""The entry point for callers that cannot allocate device memory (fd_apply_general_static).

A plug-in that is handed only input and output buffers, or code that runs where its host
forbids allocation, cannot give the library a workspace.  fd_apply_general_static keeps its
scratch in the library's own fixed device array instead.  This test calls it through the C ABI
twice in a row (the array is shared and keeps the previous call's contents, so the second call
must not be disturbed by the first) and checks both results against the float64 oracle
(the dense definition written out; the sizes here are small enough for it) and against the
ordinary entry point fd_apply_general, at the tolerance the other parity tests use for the block
product.  It lives
in a file that pytest collects last so that a failure here cannot hide any other test, and it
passes both alone in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest
import torch

import workloads
from oracle import dense

pytestmark = pytest.mark.gpu

TOL_APPLY = 1e-5


@pytest.fixture(scope="module")
def fd():
    import __graft_entry__ as g
    g.build()
    import paper_2609_38198_b200 as fd
    assert torch.cuda.is_available()
    return fd


def relF(a, b):
    a = a.double(); b = b.double()
    return float((a - b).norm() / b.norm())


def relF_oracle(Y, Yo):
    Yn = Y.cpu().numpy().astype(np.float64)
    return float(np.linalg.norm(Yn - Yo) / np.linalg.norm(Yo))


def test_static_scratch_entry_point_matches_workspace_entry_point(fd):
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(3)
    cases = [(workloads.torus6(3000, seed=21), 1.5, 32), (workloads.torus2(1777, seed=22), 30.0, 16)]
    for X, beta, b in cases:
        N = X.shape[0]
        Xd = torch.from_numpy(X).to(dev)
        lh = rng.uniform(0.5, 2.0, N).astype(np.float32)
        rh = rng.uniform(0.5, 2.0, N).astype(np.float32)
        l = torch.from_numpy(lh).to(dev)
        r = torch.from_numpy(rh).to(dev)
        V1h, V2h = workloads.block(N, b, seed=5), workloads.block(N, b, seed=6)
        V1 = fd.to_colmajor(V1h, dev)
        V2 = fd.to_colmajor(V2h, dev)
        # float64 oracle: Y = diag(l) K diag(r) V with K materialised
        O1 = dense.apply_general(X, beta, V1h, left=lh, right=rh)
        O2 = dense.apply_general(X, beta, V2h, left=lh, right=rh)
        O3 = dense.apply_general(X, beta, V1h)
        # reference results from the existing entry point (caller-provided workspace, same kernel family)
        ctx = fd.Context(Xd, b_max=b)
        ctx.set_option("path", fd.FD_PATH_SIMT)
        R1 = ctx.apply_general(beta, V1, left=l, right=r).clone()
        R2 = ctx.apply_general(beta, V2, left=l, right=r).clone()
        ctx.synchronize()
        ctx.close()
        # two calls in a row through the C ABI; outputs are caller-provided buffers
        Y1 = torch.empty((b, N), dtype=torch.float32, device=dev).t()
        Y2 = torch.empty((b, N), dtype=torch.float32, device=dev).t()
        launches = fd.fd_launch_count()
        fd.fd_apply_general_static(Xd, beta, V1, left=l, right=r, out=Y1)
        fd.fd_apply_general_static(Xd, beta, V2, left=l, right=r, out=Y2)
        torch.cuda.synchronize(dev)
        assert fd.fd_launch_count() > launches
        assert relF_oracle(Y1, O1) <= TOL_APPLY
        assert relF_oracle(Y2, O2) <= TOL_APPLY
        assert relF(Y1, R1) <= TOL_APPLY
        assert relF(Y2, R2) <= TOL_APPLY
        # optional scalings absent
        Y3 = fd.fd_apply_general_static(Xd, beta, V1)
        ctx = fd.Context(Xd, b_max=b)
        ctx.set_option("path", fd.FD_PATH_SIMT)
        R3 = ctx.apply_general(beta, V1)
        ctx.synchronize()
        assert relF_oracle(Y3, O3) <= TOL_APPLY
        assert relF(Y3, R3) <= TOL_APPLY
        ctx.close()


def test_static_scratch_entry_point_rejects_oversize(fd):
    dev = torch.device("cuda:0")
    X = torch.zeros((fd.FD_STATIC_MAX_N + 1, 4), dtype=torch.float32, device=dev)
    V = torch.zeros((1, fd.FD_STATIC_MAX_N + 1), dtype=torch.float32, device=dev).t()
    with pytest.raises(fd.FdError) as e:
        fd.fd_apply_general_static(X, 1.0, V)
    assert e.value.status == fd.FD_ERR_UNSUPPORTED and "FD_STATIC_MAX_N" in str(e.value)
    Xs = torch.zeros((64, fd.FD_STATIC_MAX_D + 1), dtype=torch.float32, device=dev)
    Vs = torch.zeros((1, 64), dtype=torch.float32, device=dev).t()
    with pytest.raises(fd.FdError) as e:
        fd.fd_apply_general_static(Xs, 1.0, Vs)
    assert e.value.status == fd.FD_ERR_UNSUPPORTED
    Xb = torch.zeros((64, 4), dtype=torch.float32, device=dev)
    Vb = torch.zeros((fd.FD_STATIC_MAX_B + 1, 64), dtype=torch.float32, device=dev).t()
    with pytest.raises(fd.FdError) as e:
        fd.fd_apply_general_static(Xb, 1.0, Vb)
    assert e.value.status == fd.FD_ERR_UNSUPPORTED
