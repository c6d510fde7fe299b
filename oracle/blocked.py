"""Large-N forms of the same float64 definitions.  Test infrastructure only.

``apply_general`` / ``degree`` evaluate Eqs. 1-3 block by block (each K block is
formed and thrown away: plain, just not stored).  ``rows_*`` evaluate a sample of
rows through the plain-C routine in ``rows.c`` (one pair at a time), which is what
full-size spot checks and the timed CPU baseline use.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = os.path.join(_HERE, "liboracle_rows.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile rows.c with gcc (OpenMP) into liboracle_rows.so next to it."""
    src = os.path.join(_HERE, "rows.c")
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, src, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        dp = ctypes.POINTER(ctypes.c_double)
        lib.fd_oracle_rows.argtypes = [dp, ctypes.c_int64, dp, ctypes.c_int64, ctypes.c_int32,
                                       ctypes.c_double, dp, dp, dp, ctypes.c_int32, dp, dp]
        lib.fd_oracle_rows.restype = None
        lib.fd_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Number of host threads the C routine uses."""
    return int(_load().fd_oracle_threads())


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def rows_apply_general(X, beta, V, rows=None, left=None, right=None, Xrow=None, want_rowsq=False):
    """Rows ``rows`` of Y = diag(left) K(Xrow, X) diag(right) V in float64 via rows.c.

    ``rows`` indexes Xrow (default X).  ``left`` is indexed like Xrow, ``right`` like X.
    V = None means the ones vector.  Returns Y[len(rows), b] (and sum_j K^2 per row).
    """
    X = _f64(X)
    Xr = X if Xrow is None else _f64(Xrow)
    if rows is None:
        rows = np.arange(Xr.shape[0])
    rows = np.asarray(rows, dtype=np.int64)
    Xs = _f64(Xr[rows])
    l = None if left is None else _f64(np.asarray(left, dtype=np.float64)[rows])
    r = None if right is None else _f64(right)
    if V is None:
        Vc, b = None, 1
    else:
        Vc = _f64(V)
        if Vc.ndim == 1:
            Vc = Vc[:, None]
        Vc = np.ascontiguousarray(Vc)
        b = Vc.shape[1]
    Y = np.empty((len(rows), b), dtype=np.float64)
    sq = np.empty(len(rows), dtype=np.float64) if want_rowsq else None
    _load().fd_oracle_rows(_ptr(Xs), len(rows), _ptr(X), X.shape[0], X.shape[1], float(beta),
                           _ptr(l), _ptr(r), _ptr(Vc), b, _ptr(Y), _ptr(sq))
    return (Y, sq) if want_rowsq else Y


def apply_general(X, beta, V, left=None, right=None, Xrow=None, block=(128, 4096)):
    """Y = diag(left) K(Xrow, X) diag(right) V, all rows, K formed in (rb x cb) blocks in numpy."""
    X = _f64(X)
    Xr = X if Xrow is None else _f64(Xrow)
    V = _f64(V)
    if V.ndim == 1:
        V = V[:, None]
    W = V if right is None else _f64(right)[:, None] * V
    R, N = Xr.shape[0], X.shape[0]
    Y = np.zeros((R, W.shape[1]), dtype=np.float64)
    rb, cb = block
    for i0 in range(0, R, rb):
        xi = Xr[i0:i0 + rb]
        acc = np.zeros((xi.shape[0], W.shape[1]), dtype=np.float64)
        for j0 in range(0, N, cb):
            xj = X[j0:j0 + cb]
            H = np.zeros((xi.shape[0], xj.shape[0]), dtype=np.float64)
            for k in range(X.shape[1]):
                diff = xi[:, k][:, None] - xj[:, k][None, :]
                H += diff * diff
            acc += np.exp(-float(beta) * H) @ W[j0:j0 + cb]
        Y[i0:i0 + rb] = acc
    if left is not None:
        Y *= _f64(left)[:, None]
    return Y


def degree(X, beta, alpha):
    """q, d, s, S_off(beta), S_off(2 beta) without storing K (two or three passes of rows.c)."""
    X = _f64(X)
    N = X.shape[0]
    q, sq = rows_apply_general(X, beta, None, want_rowsq=True)
    q = q[:, 0]
    if alpha == 0.0:
        d = q.copy()
        s = d ** (-0.5)
    else:
        qa = q ** (-float(alpha))
        d = rows_apply_general(X, beta, None, left=qa, right=qa)[:, 0]
        s = qa * d ** (-0.5)
    # Each row's diagonal entry is exp(0) = 1 in both sums.
    return q, d, s, float(q.sum() - N), float(sq.sum() - N)


def apply(X, beta, alpha, V, s=None):
    """Y = M V (Eq. 3) for all rows via rows.c; s is recomputed unless given."""
    if s is None:
        _, _, s, _, _ = degree(X, beta, alpha)
    return rows_apply_general(X, beta, V, left=s, right=s)


def eigs_certified(X, beta, alpha, k, tol=1e-10, seed=0, maxiter=400):
    """Leading k+1 eigenpairs of M over the matrix-free float64 operator (scipy LOBPCG),
    certified by explicit residuals.  Returns (evals, evecs, d, residual_norms)."""
    from scipy.sparse.linalg import LinearOperator, lobpcg

    X = _f64(X)
    N = X.shape[0]
    _, d, s, _, _ = degree(X, beta, alpha)

    def mv(V):
        return rows_apply_general(X, beta, V, left=s, right=s)

    op = LinearOperator((N, N), matvec=lambda v: mv(v[:, None])[:, 0], matmat=mv, dtype=np.float64)
    rng = np.random.default_rng(seed)
    nb = k + 1 + min(8, max(2, k // 4))
    U0 = rng.standard_normal((N, nb))
    U0[:, 0] = np.sqrt(d)
    w, U = lobpcg(op, U0, largest=True, tol=tol, maxiter=maxiter)
    order = np.argsort(w)[::-1][: k + 1]
    w, U = w[order], U[:, order]
    res = np.linalg.norm(mv(U) - U * w[None, :], axis=0)
    return w, U, d, res
