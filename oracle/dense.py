"""Dense float64 definitions (Sec. 2.1, Eqs. 1-3).  Test infrastructure only.

Everything here materialises the N x N kernel, so it is for N up to ~16k.
Inputs are the float32-rounded points upcast to float64.
"""
from __future__ import annotations

import numpy as np


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def sqdist(X, Y=None) -> np.ndarray:
    """H_ij = sum_k (x_ik - y_jk)^2 by direct differences (no Gram trick).

    Eq. 1 takes H as the matrix of pairwise squared Euclidean distances.
    """
    X = _f64(X)
    Y = X if Y is None else _f64(Y)
    H = np.zeros((X.shape[0], Y.shape[0]), dtype=np.float64)
    for k in range(X.shape[1]):
        diff = X[:, k][:, None] - Y[:, k][None, :]
        H += diff * diff
    return H


def kernel(X, beta: float, Y=None) -> np.ndarray:
    """K = exp(-beta * H), elementwise (Eq. 1)."""
    return np.exp(-float(beta) * sqdist(X, Y))


def normalisation(K: np.ndarray, alpha: float):
    """q = K 1; K_alpha = diag(q)^-alpha K diag(q)^-alpha; d = K_alpha 1;
    s = q^-alpha * d^-1/2 (text around Eq. 2).  Returns (q, d, s)."""
    q = K.sum(axis=1)
    qa = q ** (-float(alpha))
    K_alpha = qa[:, None] * K * qa[None, :]
    d = K_alpha.sum(axis=1)
    s = qa * d ** (-0.5)
    return q, d, s


def markov(K: np.ndarray, alpha: float) -> np.ndarray:
    """P = diag(d)^-1 K_alpha, the row-stochastic diffusion operator."""
    q = K.sum(axis=1)
    qa = q ** (-float(alpha))
    K_alpha = qa[:, None] * K * qa[None, :]
    d = K_alpha.sum(axis=1)
    return K_alpha / d[:, None]


def symmetric_operator(K: np.ndarray, alpha: float) -> np.ndarray:
    """M = diag(s) K diag(s) (Eq. 2)."""
    _, _, s = normalisation(K, alpha)
    return s[:, None] * K * s[None, :]


def s_off(K: np.ndarray) -> float:
    """S_off = sum_{i != j} K_ij (text before Eq. 9).  The diagonal is exactly 1."""
    return float(K.sum() - np.trace(K))


def degree(X, beta: float, alpha: float):
    """What the degree pass returns: q, d, s, S_off(beta), S_off(2 beta).

    S_off(2 beta) is evaluated from its definition with the kernel at 2 beta.
    """
    K = kernel(X, beta)
    q, d, s = normalisation(K, alpha)
    K2 = kernel(X, 2.0 * float(beta))
    return q, d, s, s_off(K), s_off(K2)


def apply_general(X, beta: float, V, left=None, right=None, Xrow=None) -> np.ndarray:
    """Y = diag(left) K(Xrow, X) diag(right) V with K_ij = exp(-beta |xrow_i - x_j|^2).

    left/right default to ones; Xrow defaults to X (square product).  This is the
    single primitive W -> K W of Sec. 2.1 with both diagonal scalings written out.
    """
    V = _f64(V)
    if V.ndim == 1:
        V = V[:, None]
    K = kernel(X if Xrow is None else Xrow, beta, X)
    W = V if right is None else _f64(right)[:, None] * V
    Y = K @ W
    if left is not None:
        Y = _f64(left)[:, None] * Y
    return Y


def apply(X, beta: float, alpha: float, V) -> np.ndarray:
    """Y = M V = diag(s) K (diag(s) V) (Eq. 3)."""
    K = kernel(X, beta)
    _, _, s = normalisation(K, alpha)
    V = _f64(V)
    if V.ndim == 1:
        V = V[:, None]
    return s[:, None] * (K @ (s[:, None] * V))


def eigs(X, beta: float, alpha: float, k: int):
    """Perron pair + k nontrivial eigenpairs of M, descending (slot 0 = Perron).

    Returns (evals[k+1], evecs[N, k+1], d).  Markov right eigenvectors follow by
    the diagonal rescale psi = d^-1/2 * v (end of Sec. 2.3).
    """
    K = kernel(X, beta)
    _, d, s = normalisation(K, alpha)
    M = s[:, None] * K * s[None, :]
    M = 0.5 * (M + M.T)
    w, U = np.linalg.eigh(M)
    order = np.argsort(w)[::-1][: k + 1]
    return w[order], U[:, order], d


def markov_vectors(evecs: np.ndarray, d: np.ndarray) -> np.ndarray:
    """psi = d^-1/2 * v: right eigenvectors of P from eigenvectors of M."""
    return evecs / np.sqrt(_f64(d))[:, None]


def principal_angles(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """Principal angles (rad, ascending) between span(A) and span(B); columns need not be orthonormal.

    Uses the sine form for small angles: sin(theta) = singular values of (I - Qa Qa^T) Qb.
    """
    Qa, _ = np.linalg.qr(_f64(A))
    Qb, _ = np.linalg.qr(_f64(B))
    R = Qb - Qa @ (Qa.T @ Qb)
    sv = np.linalg.svd(R, compute_uv=False)
    return np.arcsin(np.clip(np.sort(sv), 0.0, 1.0))
