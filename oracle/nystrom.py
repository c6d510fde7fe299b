"""Out-of-sample (Nystrom) extension of Markov eigenvectors.  Test infrastructure only.

The ladder of Sec. 1 extends an eigenspace found on n points to more points before
re-solving there.  The paper cites the standard out-of-sample formula without printing
it; this is that formula for the row-stochastic operator P = diag(d)^-1 K_alpha of
Sec. 2.1.  Since P(x, i) = K(x, x_i) q_i^-alpha / sum_l K(x, x_l) q_l^-alpha (the
factor q(x)^-alpha cancels between numerator and row sum),

    psi_j(x) = (1 / lambda_j) * sum_i P(x, i) psi_j(x_i).

Evaluated at a sample point it returns psi_j(x_i) itself because P psi = lambda psi.
"""
from __future__ import annotations

import numpy as np

from . import dense


def extend(X_old, q_old, alpha, beta, psi_old, evals, X_new) -> np.ndarray:
    """psi_old: n x m Markov eigenvectors on X_old with eigenvalues evals[m]; returns N_new x m."""
    K = dense.kernel(X_new, beta, X_old)                       # N_new x n
    w = np.asarray(q_old, dtype=np.float64) ** (-float(alpha))
    num = K @ (w[:, None] * np.asarray(psi_old, dtype=np.float64))
    den = K @ w
    return num / den[:, None] / np.asarray(evals, dtype=np.float64)[None, :]
