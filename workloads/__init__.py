"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws points and test blocks.  It holds none of the method's
arithmetic (no kernel, no normalisation, no eigen-anything), so both the CPU
oracle and the CUDA path may take their inputs from it without sharing any
computation.

Every generator draws in float64 from ``numpy.random.default_rng(seed)``
(PCG64), in the draw order written in its docstring, and rounds ONCE to
float32.  The float32 array is the single source of truth: the oracle upcasts
it to float64, the GPU path uses it as is.

Workloads (the paper's Sec. 3 torus experiment and Sec. 4 molecular experiment
are the models for the shapes; no dataset is read):

* ``circle``      equispaced points on the unit circle in R^2 (closed-form spectrum)
* ``torus2``      flat 2-torus in R^4, uniform angles
* ``torus_grid``  equispaced N1 x N2 lattice on the flat 2-torus (Kronecker spectrum)
* ``torus6``      flat 6-torus in R^12 with isotropic Gaussian noise
* ``torus6_paper``the paper's anisotropic T^6 (radii 1.00 .. 1.50), zero-padded to D = 32
* ``latent_torus``4-component von Mises mixture on (phi, psi) pushed to R^30 by tanh(W u + c)
"""
from __future__ import annotations

import numpy as np

TWO_PI = 2.0 * np.pi

# Radii of the anisotropic six-torus of the paper's Sec. 3.
PAPER_T6_RADII = (1.00, 1.08, 1.17, 1.27, 1.38, 1.50)


def circle(N: int = 2048) -> np.ndarray:
    """x_i = (cos(2 pi i / N), sin(2 pi i / N)), i = 0..N-1.  No randomness."""
    th = TWO_PI * np.arange(N, dtype=np.float64) / N
    return np.stack([np.cos(th), np.sin(th)], axis=1).astype(np.float32)


def torus2(N: int = 16384, seed: int = 42) -> np.ndarray:
    """Draw order: t = uniform(0, 2 pi, (N, 2)).  x = (cos t1, sin t1, cos t2, sin t2)."""
    rng = np.random.default_rng(seed)
    t = rng.uniform(0.0, TWO_PI, (N, 2))
    x = np.stack([np.cos(t[:, 0]), np.sin(t[:, 0]), np.cos(t[:, 1]), np.sin(t[:, 1])], axis=1)
    return x.astype(np.float32)


def torus_grid(N1: int, N2: int) -> np.ndarray:
    """Equispaced N1 x N2 lattice on the flat 2-torus, point index = i1 * N2 + i2."""
    a = TWO_PI * np.arange(N1, dtype=np.float64) / N1
    b = TWO_PI * np.arange(N2, dtype=np.float64) / N2
    A, B = np.meshgrid(a, b, indexing="ij")
    x = np.stack([np.cos(A), np.sin(A), np.cos(B), np.sin(B)], axis=-1).reshape(N1 * N2, 4)
    return x.astype(np.float32)


def torus6(N: int = 131072, seed: int = 42, sigma: float = 0.01,
           radii=(1.0,) * 6, pad_to: int | None = None, return_angles: bool = False):
    """Draw order: t = uniform(0, 2 pi, (N, 6)); noise = standard_normal((N, 12)).

    x = (R_a cos t_a, R_a sin t_a)_{a=1..6} + sigma * noise.  The level-n subsample
    of the continuation ladder is simply the first n rows of the N = 2^20 draw.
    """
    rng = np.random.default_rng(seed)
    t = rng.uniform(0.0, TWO_PI, (N, 6))
    R = np.asarray(radii, dtype=np.float64)
    x = np.empty((N, 12), dtype=np.float64)
    x[:, 0::2] = R * np.cos(t)
    x[:, 1::2] = R * np.sin(t)
    if sigma != 0.0:
        x += sigma * rng.standard_normal((N, 12))
    if pad_to is not None and pad_to > 12:
        x = np.concatenate([x, np.zeros((N, pad_to - 12))], axis=1)
    if return_angles:
        return x.astype(np.float32), t
    return x.astype(np.float32)


def torus6_paper(N: int, seed: int = 42, return_angles: bool = False):
    """The paper's Sec. 3 / App. B shape: anisotropic radii, no noise, D = 32 (12 non-zero).  With return_angles the
    N x 6 angles come back too (they enter only the post-hoc first-harmonic score, never a solve)."""
    return torus6(N, seed=seed, sigma=0.0, radii=PAPER_T6_RADII, pad_to=32, return_angles=return_angles)


_VM_MEANS = np.array([(-1.4, 2.6), (-1.4, -0.7), (1.1, -0.8), (-2.5, 2.9)], dtype=np.float64)
_VM_WEIGHTS = np.array([0.4, 0.3, 0.2, 0.1], dtype=np.float64)


def latent_torus(N: int = 262144, seed: int = 42, kappa: float = 8.0,
                 sigma: float = 0.02, D: int = 30, return_angles: bool = False):
    """Molecule-like latent 2-torus in R^D.

    Draw order: W = standard_normal((D, 4)); c = standard_normal(D);
    comp = choice(4, N, p = weights); phi = vonmises(mu_phi[comp], kappa);
    psi = vonmises(mu_psi[comp], kappa); noise = standard_normal((N, D)).
    x = tanh(W [cos phi, sin phi, cos psi, sin psi] + c) + sigma * noise.
    """
    rng = np.random.default_rng(seed)
    W = rng.standard_normal((D, 4))
    c = rng.standard_normal(D)
    comp = rng.choice(4, N, p=_VM_WEIGHTS)
    phi = rng.vonmises(_VM_MEANS[comp, 0], kappa)
    psi = rng.vonmises(_VM_MEANS[comp, 1], kappa)
    u = np.stack([np.cos(phi), np.sin(phi), np.cos(psi), np.sin(psi)], axis=1)
    x = np.tanh(u @ W.T + c) + sigma * rng.standard_normal((N, D))
    x = x.astype(np.float32)
    if return_angles:
        return x, phi, psi
    return x


def gaussian_cloud(N: int, D: int, seed: int = 0, scale: float = 1.0) -> np.ndarray:
    """Generic i.i.d. N(0, scale^2) cloud for shape / tail-tile edge cases."""
    rng = np.random.default_rng(seed)
    return (scale * rng.standard_normal((N, D))).astype(np.float32)


def block(N: int, b: int, seed: int = 1) -> np.ndarray:
    """Right-hand block V (N x b), i.i.d. N(0, 1), returned column-major (Fortran order).

    Unsmoothed noise is the hardest case for entrywise errors of a kernel product.
    """
    rng = np.random.default_rng(seed)
    V = rng.standard_normal((N, b)).astype(np.float32)
    return np.asfortranarray(V)


def row_sample(N: int, count: int, seed: int = 7) -> np.ndarray:
    """Sorted sample of ``count`` distinct row indices, for sampled full-size parity."""
    rng = np.random.default_rng(seed)
    count = min(count, N)
    return np.sort(rng.choice(N, size=count, replace=False)).astype(np.int64)


# name -> (generator kwargs, run parameters) for the five benchmark configurations.
CONFIGS = {
    "C1": dict(gen="circle", N=2048, D=2, beta=200.0, alpha=1.0, b=8, k=8),
    "C2": dict(gen="torus2", N=16384, D=4, betas=(10.0, 30.0, 100.0, 300.0), alpha=1.0, b=16, k=32),
    "C3": dict(gen="torus6", N=131072, D=12, beta_grid=(1.0, 1000.0), alpha=1.0, b=32, k=64),
    "C4": dict(gen="latent_torus", N=262144, D=30, beta=2.0, alpha=1.0, b=32, k=32),
    "C5": dict(gen="torus6", N=1048576, D=12, beta=2.0, alpha=1.0, b=64, k=128,
               ladder=(65536, 131072, 262144, 524288, 1048576)),
}


def make(name: str, N: int | None = None, seed: int = 42) -> np.ndarray:
    """Points of configuration ``name`` (optionally at a reduced N, same recipe)."""
    cfg = CONFIGS[name]
    n = cfg["N"] if N is None else N
    g = cfg["gen"]
    if g == "circle":
        return circle(n)
    if g == "torus2":
        return torus2(n, seed)
    if g == "torus6":
        return torus6(n, seed)
    if g == "latent_torus":
        return latent_torus(n, seed)
    raise KeyError(g)
