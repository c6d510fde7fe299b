"""Bandwidth flow of Sec. 2.3 (Eqs. 7-14) restated step by step.  Test infrastructure only.

The paper states the quantities and the acceptance rule in prose; the readings taken
where it is silent are listed beside each step.  Float64 throughout.
"""
from __future__ import annotations

import math

import numpy as np

from . import dense

# Constants printed in Sec. 2.3.
BETA0_CAP = 0.1          # Eq. 7
P_EXPONENT = 6           # Eq. 11
KAPPA_P = 10.0           # Eq. 11
ETA = {"bf16": 8e-3, "tf32": 1e-3, "fp32": 1e-7, "fp64": 2.22e-16}   # footnote to Eq. 12


def beta0(X) -> float:
    """Eq. 7: min(0.1, 1 / (2 * mean_i |x_i - mu|^2)) on mean-centred data."""
    X = np.asarray(X, dtype=np.float64)
    Xc = X - X.mean(axis=0, keepdims=True)
    mean_sq = float((Xc * Xc).sum(axis=1).mean())
    return min(BETA0_CAP, 1.0 / (2.0 * mean_sq))


def v_bias(evals) -> float:
    """Eq. 8: median over the k nontrivial modes j = 1..k of -log(lambda_j / lambda_0).
    (Even k: numpy's median = mean of the two middle values.)"""
    lam = np.asarray(evals, dtype=np.float64)
    return float(np.median(-np.log(lam[1:] / lam[0])))


def n_eff(S_off_beta: float, S_off_2beta: float, N: int) -> float:
    """Eq. 9: S_off(beta)^2 / (N * S_off(2 beta))."""
    return S_off_beta * S_off_beta / (N * S_off_2beta)


def v_stat(neff: float, vbias: float) -> float:
    """Eq. 10."""
    return 1.0 / math.sqrt(neff * vbias)


def perron_gap(evals) -> float:
    """g_P = (lambda_0 - lambda_1) / |lambda_0| (text before Eq. 11)."""
    return float((evals[0] - evals[1]) / abs(evals[0]))


def v_mach(gP: float, eta: float = ETA["fp32"], kappa: float = KAPPA_P, p: int = P_EXPONENT) -> float:
    """Eq. 11."""
    return (kappa * eta / gP) ** p


def admissible(gP: float, eta: float = ETA["fp32"], kappa: float = KAPPA_P) -> bool:
    """Eq. 12: g_P > kappa_P * eta."""
    return gP > kappa * eta


def d_hat(S_off_beta: float, S_off_2beta: float) -> float:
    """Eq. 14 across the dyadic pair (beta, 2 beta): -2 * dlog S_off / dlog beta."""
    return -2.0 * (math.log(S_off_2beta) - math.log(S_off_beta)) / math.log(2.0)


def potential(evals, S_off_beta, S_off_2beta, N, eta=ETA["fp32"]):
    """All terms of Eq. 13 for one probe, as a dict."""
    vb = v_bias(evals)
    ne = n_eff(S_off_beta, S_off_2beta, N)
    vs = v_stat(ne, vb)
    gp = perron_gap(evals)
    vm = v_mach(gp, eta) if gp > 0 else math.inf
    return dict(V_bias=vb, n_eff=ne, V_stat=vs, g_P=gp, V_mach=vm, V=vb + vs + vm,
                d_hat=d_hat(S_off_beta, S_off_2beta))


def bracket(p1, p2, p3) -> bool:
    """Acceptance rule (last paragraph before Eq. 14): three consecutive probes bracket a
    stationary point, V_bias falling and V_stat or V_mach rising across the triplet."""
    return (p2["V"] <= min(p1["V"], p3["V"]) and p3["V_bias"] < p1["V_bias"]
            and (p3["V_stat"] > p1["V_stat"] or p3["V_mach"] > p1["V_mach"]))


def vertex(p1, p2, p3) -> float:
    """Vertex of the parabola through (log beta, V) of the triplet, clamped to [beta1, beta3]."""
    x = np.log([p1["beta"], p2["beta"], p3["beta"]])
    y = np.array([p1["V"], p2["V"], p3["V"]])
    c2, c1, _ = np.polyfit(x, y, 2)
    xv = x[1] if c2 <= 0 else -c1 / (2.0 * c2)
    return float(np.exp(min(max(xv, x[0]), x[2])))


def dense_probe(X, alpha, k):
    """Probe callable on materialised K: beta -> (evals[k+1], S_off(beta), S_off(2 beta))."""
    def probe(beta):
        _, _, _, so, so2 = dense.degree(X, beta, alpha)
        lam, _, _ = dense.eigs(X, beta, alpha, k)
        return lam, so, so2
    return probe


def beta_flow(probe, N, beta_start, beta_max, eta=ETA["fp32"], ratio=2.0):
    """Dyadic sweep beta -> 2 beta from beta_start; returns (beta_x, status, log).

    status: "VERTEX" (bracket found, final probe at the vertex), "PERRON_WALL" (Eq. 12 failed
    before a bracket: last safe probe), "LEFT_EDGE" (V already rising at the second probe),
    "RIGHT_EDGE" (grid exhausted while V still falls: last probe).
    """
    log = []
    beta = float(beta_start)
    while beta <= beta_max * (1 + 1e-12):
        lam, so, so2 = probe(beta)
        rec = dict(beta=beta, evals=np.asarray(lam, dtype=np.float64), S_off=so, S_off2=so2)
        rec.update(potential(rec["evals"], so, so2, N, eta))
        if not admissible(rec["g_P"], eta):
            rec["wall"] = True
            log.append(rec)
            safe = [r for r in log if not r.get("wall")]
            return (safe[-1]["beta"] if safe else float("nan")), "PERRON_WALL", log
        log.append(rec)
        if len(log) == 2 and log[1]["V"] > log[0]["V"]:
            return log[0]["beta"], "LEFT_EDGE", log
        if len(log) >= 3 and bracket(log[-3], log[-2], log[-1]):
            bv = vertex(log[-3], log[-2], log[-1])
            lam, so, so2 = probe(bv)
            fin = dict(beta=bv, evals=np.asarray(lam, dtype=np.float64), S_off=so, S_off2=so2, final=True)
            fin.update(potential(fin["evals"], so, so2, N, eta))
            log.append(fin)
            return bv, "VERTEX", log
        beta *= ratio
    return log[-1]["beta"], "RIGHT_EDGE", log


def cascade(probes, N, beta_start, beta_max, etas, ratio=2.0):
    """Precision cascade (Sec. 2.3, last paragraph; eta per data type from the footnote to Eq. 11).

    One sweep per requested data type, in the order given: `probes[s]` evaluates a probe at stage s (its arithmetic)
    and `etas[s]` is that data type's precision scale in Eqs. 11-12.  The paper says only that the selected state of
    one stage initialises the next; the reading taken here: stage s + 1 restarts the dyadic sweep one grid step below
    the bandwidth stage s selected (so that a bracket around it can form) and the final bandwidth and eigenpairs
    are those of the last stage.  Returns (beta_x, status, [log per stage]).
    """
    logs = []
    start = float(beta_start)
    bx, status = float("nan"), "PERRON_WALL"
    for probe, eta in zip(probes, etas):
        bx, status, log = beta_flow(probe, N, start, beta_max, eta=eta, ratio=ratio)
        logs.append(log)
        if not (bx == bx):                       # no safe probe at all in this stage: nothing to hand on
            break
        start = bx / ratio
    return bx, status, logs
