"""CPU float64 oracle for the FlashDiffusion hot path.  TEST INFRASTRUCTURE ONLY.

Plain, slow, obviously-correct restatement of what the paper's method computes,
written from the paper's equations; it shares no code with the CUDA path and
never imports it.  Only the tests, the smoke check and the benchmark's CPU
baseline leg may call anything in this package; the product path must never
route through it.

Modules
-------
dense     Sec. 2.1, Eqs. 1-3: K, q, K_alpha, d, P, s, M materialised on small N;
          dense eigendecomposition (the definition of what the eigensolver returns).
blocked   the same definitions evaluated block by block for large N (nothing stored),
          plus a plain-C row-sampled variant (``rows.c``) for full-size spot checks.
flow      Sec. 2.3, Eqs. 7-14: initial bandwidth, potential terms, bracket / vertex rule,
          intrinsic-dimension diagnostic; the precision cascade (one sweep per data type).
nystrom   out-of-sample extension of Markov eigenvectors used by the (n, beta) ladder (Sec. 1).
overlap   post-hoc first-harmonic score of the T^6 validation (Sec. 3, Fig. 1(c) footnote): squared RV coefficient.

Parity pins (tests marked ``not gpu``): symmetry / PSD / unit diagonal of K; Markov
row sums and the Perron identity M sqrt(d) = sqrt(d); the beta -> 0 rank-one limit;
circulant closed form on the circle (DFT and Bessel-ratio forms); Kronecker spectrum on
a lattice torus; two-point and simplex closed forms; K(2 beta) = K(beta)^2; n_eff = k for
k equal weights; dense eigh vs the blocked path; Nystrom reproduces psi at sample points;
principal angles and the RV score on subspaces with known angles; the cascade on a
hand-built potential.  The beta-flow's bracket rule and the cascade's hand-over rule have
only soft pins against the paper (its printed T^6 table, another RNG): exact beta-flow
parity is "parity unpinned".
"""
from . import dense, blocked, flow, nystrom, overlap  # noqa: F401
