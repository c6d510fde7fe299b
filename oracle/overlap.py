"""Post-hoc subspace score of the T^6 validation (Sec. 3, Fig. 1(c) and its footnote).  Test infrastructure only.

For A (N x p) and B (N x p) with centred covariance blocks G_AA, G_BB, G_AB the score is
sum_ij C_ij^2 / p with C = G_AA^-1/2 G_AB G_BB^-1/2 (p = 2 in the paper: the leading two nontrivial modes against
(cos theta_s, sin theta_s) of the largest circle).  It is 1 iff the centred column spans coincide and 0 iff they are
orthogonal; it does not change when A or B is multiplied by an invertible p x p matrix.  Everything in float64.
"""
from __future__ import annotations

import numpy as np


def _inv_sqrt(G: np.ndarray) -> np.ndarray:
    w, Q = np.linalg.eigh(G)
    return (Q / np.sqrt(w)) @ Q.T


def rv_overlap(A, B) -> float:
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    A = A - A.mean(axis=0, keepdims=True)
    B = B - B.mean(axis=0, keepdims=True)
    n = A.shape[0]
    Gaa, Gbb, Gab = A.T @ A / n, B.T @ B / n, A.T @ B / n
    C = _inv_sqrt(Gaa) @ Gab @ _inv_sqrt(Gbb)
    return float((C * C).sum() / A.shape[1])


def first_harmonic_target(angles, circle: int) -> np.ndarray:
    """Columns (cos theta_s, sin theta_s) of one circle of the torus."""
    t = np.asarray(angles, dtype=np.float64)[:, circle]
    return np.stack([np.cos(t), np.sin(t)], axis=1)
