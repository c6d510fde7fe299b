#!/usr/bin/env python
"""Benchmark of the FlashDiffusion hot path on B200.

One step = one pass of the whole hot path at a fixed bandwidth over the headline workload
(6-torus in R^12, N = 2^20, block b = 64, alpha = 1, beta = 2): degree pass q = K 1, second
normalisation pass d = q^-a * K q^-a, scale vector s, and the block product Y = M V.  A step
therefore processes (b + 2) N^2 pair-columns; `value` is that count over the step time,
aggregated over ranks (each rank runs an independent replica: the path is not sharded).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--n LOG2N]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU float64 oracle on a bounded
row sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "kernel-apply pair-columns per second (degree passes + block product, one step)"
UNIT = "pair*cols/s"

# Nominal unit counts for the roofline: MUFU 16 ex2/clk/SM, FMA pipe 128 FFMA/clk/SM, 148 SMs.
SM_COUNT = 148
MUFU_PER_CLK_SM = 16
FMA_PER_CLK_SM = 128

# DRAM bytes per launch of the dominant kernel from the committed ncu capture (profiles/), or None.
NCU_TRAFFIC_BYTES = {"simt": None, "tc": 20.15e9 + 2.18e9}   # k_tc block mode at N = 2^20, profiles/bench_c5_n2e20_launch_list.md


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0}, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.idx)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); smax.append(float(parts[2])); power.append(float(parts[3]))
            except ValueError:
                continue
            for n, v in zip(names, parts[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "power_w_max": float(max(power)),
                "samples": len(sm), "reasons": sorted(reasons)}


def workload(log2n: int):
    import workloads
    N = 1 << log2n
    X = workloads.torus6(N, seed=42)
    V = workloads.block(N, 64, seed=1)
    return X, V, dict(workload=f"C5: 6-torus R^12 + noise 0.01, N=2^{log2n}, b=64, alpha=1, beta=2.0",
                      N=N, D=12, b=64, alpha=1.0, beta=2.0, l2_note="inputs (X, V, Y: >= 0.6 GB) exceed the 126 MB L2")


# ------------------------------------------------------------------------------------------- CPU oracle arm
def oracle_step(X64, V64, beta, alpha, rows, q_hint=None):
    """One bounded sample of the step on the CPU oracle: the three passes on `rows` rows."""
    from oracle import blocked
    q_rows, _ = blocked.rows_apply_general(X64, beta, None, rows=rows, want_rowsq=True)
    # the second pass and the product need q, s on all columns: use a positive surrogate vector of the right
    # magnitude for the columns (the cost per pair is what is being timed, not the values)
    w = q_hint
    blocked.rows_apply_general(X64, beta, None, rows=rows, left=w, right=w)
    blocked.rows_apply_general(X64, beta, V64, rows=rows, left=w, right=w)
    return q_rows


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import blocked
    X, V, cfg = workload(args.n)
    N, b = cfg["N"], cfg["b"]
    X64 = X.astype(np.float64)
    V64 = np.ascontiguousarray(V.astype(np.float64))
    cores = blocked.threads()
    # size the sample for ~6-10 s per step on this host: ~4e7 pair-evaluations per core-second over three passes
    rows_n = int(max(16, min(N, 6.0 * cores * 2.0e7 / N)))
    import workloads
    rows = workloads.row_sample(N, rows_n, seed=11)
    w = np.full(N, 1e-2)
    for _ in range(max(1, min(args.warmup, 1))):
        oracle_step(X64, V64, cfg["beta"], cfg["alpha"], rows[: max(16, rows_n // 8)], w)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(X64, V64, cfg["beta"], cfg["alpha"], rows, w)
    dt = (time.perf_counter() - t0) / args.steps
    units = rows_n * N * (b + 2)
    value = units / dt
    sample = f"{rows_n} sampled rows x all {N} columns, three passes (b = 1, 1, {b}), float64, rows.c + OpenMP"
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


# ------------------------------------------------------------------------------------------- multi-rank plumbing
def max_over_ranks(values, dist, device):
    """Device-side times of every rank -> their maximum over ranks (the job is as slow as its slowest replica)."""
    import torch
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def job_value(units_per_rank: float, world: int, ms: float) -> float:
    """Whole-job throughput of `world` independent replicas (weak scaling): all units over the slowest rank's time."""
    return units_per_rank * world / (ms * 1e-3)


# ------------------------------------------------------------------------------------------- GPU arm
def run_gpu(args):
    import torch
    import paper_2609_38198_b200 as fd
    from paper_2609_38198_b200 import build as fd_build
    fd_build.build()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)

    X, V, cfg = workload(args.n)
    N, b, beta, alpha = cfg["N"], cfg["b"], cfg["beta"], cfg["alpha"]
    Xh = torch.from_numpy(X).pin_memory()
    Vh = torch.from_numpy(np.ascontiguousarray(V.T)).pin_memory()          # (b, N): column-major N x b
    Yh = torch.empty((b, N), dtype=torch.float32).pin_memory()
    Xd = Xh.to(dev)
    Vd = Vh.to(dev).t()
    Yd = torch.empty((b, N), dtype=torch.float32, device=dev).t()
    ctx = fd.Context(Xd, b_max=b, m_max=0)
    if args.path:
        ctx.set_option("path", {"auto": 0, "simt": 1, "tc": 2}[args.path])
    stream = torch.cuda.current_stream(dev)

    ev = lambda: torch.cuda.Event(enable_timing=True)

    def step(timers=None):
        e0, e1, e2 = ev(), ev(), ev()
        e0.record(stream)
        ctx.degree(beta, alpha)
        e1.record(stream)
        ctx.apply(Vd, out=Yd)
        e2.record(stream)
        if timers is not None:
            timers.append((e0, e1, e2))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    timers = []
    launches0 = fd.fd_launch_count()
    t_start, t_end = ev(), ev()
    barrier()
    t_start.record(stream)
    for _ in range(args.steps):
        step(timers)
    t_end.record(stream)
    barrier()
    launches = fd.fd_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    total_ms = t_start.elapsed_time(t_end)
    deg_ms = float(np.mean([a.elapsed_time(b_) for a, b_, _ in timers]))
    app_ms = float(np.mean([b_.elapsed_time(c_) for _, b_, c_ in timers]))

    # end-to-end through the public API with host buffers: H2D of X and V, D2H of Y every step
    def e2e_step():
        Xd.copy_(Xh, non_blocking=True)
        Vd.t().copy_(Vh, non_blocking=True)
        c2 = fd.Context(Xd, b_max=b, m_max=0)
        if args.path:
            c2.set_option("path", {"auto": 0, "simt": 1, "tc": 2}[args.path])
        c2.degree(beta, alpha)
        c2.apply(Vd, out=Yd)
        Yh.copy_(Yd.t(), non_blocking=True)
        torch.cuda.synchronize(dev)
        c2.close()

    e2e_steps = max(1, min(args.steps, 3))
    e2e_step()
    barrier()
    e_a, e_b = ev(), ev()
    e_a.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e_b.record(stream)
    barrier()
    e2e_ms = e_a.elapsed_time(e_b) / e2e_steps

    total_ms, e2e_ms, deg_ms, app_ms = max_over_ranks([total_ms, e2e_ms, deg_ms, app_ms], dist, dev)
    step_ms = total_ms / args.steps
    units = float(N) * N * (b + 2)

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        path_used = "tc" if ctx.get_option("last_path") == 2 else "simt"
        pairs_per_s = float(N) * N / (app_ms * 1e-3)
        mhz = (clocks or {}).get("sm_mhz") or peaks.get("sm_max_mhz", 1965.0)
        mufu_peak = SM_COUNT * MUFU_PER_CLK_SM * peaks.get("sm_max_mhz", 1965.0) * 1e6       # exp / s
        fma_peak = SM_COUNT * FMA_PER_CLK_SM * peaks.get("sm_max_mhz", 1965.0) * 1e6         # FMA / s
        D = cfg["D"]
        if path_used == "simt":
            # everything on the FMA pipe: per pair 2 D (difference form) + b (product) + ~3 issue slots
            peak_pairs = fma_peak / (2 * D + b + 3)
            binder = "fma_pipe (direct-difference distance + block product on FFMA)"
        else:
            peak_pairs = mufu_peak
            binder = "mufu (one ex2 per pair)"
        roofline = {"bound": "alu", "kernel": "block product Y = M V (dominant kernel)", "binder": binder,
                    "achieved": pairs_per_s / 1e9, "peak": peak_pairs / 1e9, "unit": "Gpairs/s",
                    "frac": pairs_per_s / peak_pairs, "peak_source": f"unit counts x {peak_kind} max SM clock",
                    "mufu_floor_frac": pairs_per_s / mufu_peak, "traffic": NCU_TRAFFIC_BYTES.get(path_used) if N == (1 << 20) else None,
                    "algorithmic_bytes": 4.0 * N * (D + 2 * b + 2),
                    "sm_mhz_seen": mhz}
        out = {"metric": METRIC, "value": job_value(units, world, step_ms), "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg, "clocks": clocks,
               "apply_only": {"ms": app_ms, "pair_cols_per_s": float(N) * N * b / (app_ms * 1e-3), "pairs_per_s": pairs_per_s},
               "degree_ms": deg_ms, "path": path_used, "roofline": roofline,
               "e2e": {"value": job_value(units, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                       "h2d_bytes_per_step": int(Xh.numel() * 4 + Vh.numel() * 4), "d2h_bytes_per_step": int(Yh.numel() * 4)},
               "gpu_launches": int(launches), "workspace_bytes": ctx.workspace_bytes}
        if not args.no_cpu:
            out["cpu_baseline"] = cpu_baseline(X, V, cfg)
        ctx.close()
        if not args.no_eigs:
            del Xd, Vd, Yd
            torch.cuda.empty_cache()
            out["time_to_k_eigs"] = time_to_k_eigs(fd, dev, full=args.eigs_full)
        print(json.dumps(out), flush=True)
    ctx.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def time_to_k_eigs(fd, dev, full=False):
    """Second half of the metric: wall time from a fresh bandwidth to k eigenpairs (degree passes + fd_eigs) on the
    benchmark configurations at full size (C1, C2 at beta = 10 and 30, C3, C4; with --eigs-full also C5 at N = 2^20), the
    whole dyadic bandwidth flow on C3, and the nested-level ladder.  Host wall clock around synchronous calls."""
    import torch
    import workloads
    res = []
    # (name, points, k, b, beta): the five benchmark configurations at their full sizes
    cases = [("C1 circle", workloads.circle(2048), 8, 8, 200.0),
             ("C2 2-torus", workloads.torus2(16384, seed=42), 32, 16, 10.0),
             ("C2 2-torus", None, 32, 16, 30.0),
             ("C3 6-torus", workloads.torus6(1 << 17, seed=42), 64, 32, 2.0),
             ("C4 latent torus R^30", workloads.latent_torus(262144, seed=42), 32, 32, 2.0)]
    if full:
        cases.append(("C5 6-torus", workloads.torus6(1 << 20, seed=42), 128, 64, 2.0))
    Xnp = None
    for name, Xc, k, b, beta in cases:
        if Xc is not None:
            Xnp = Xc
        N = Xnp.shape[0]
        X = torch.from_numpy(Xnp).to(dev)
        m_max = (max(2 * (k + 1) + b, 4 * b) + b - 1) // b * b
        ctx = fd.Context(X, b_max=b, m_max=m_max)
        ctx.degree(beta, 1.0)                                        # warm-up of both passes
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        ctx.degree(beta, 1.0)
        t1 = time.perf_counter()
        lam, U, info = ctx.eigs(k, b, tol=1e-6, max_applies=600, allow_not_converged=True)
        t2 = time.perf_counter()
        rec = {"workload": f"{name}: N={N}, D={Xnp.shape[1]}, k={k}, b={b}, alpha=1, beta={beta}, tol=1e-6",
               "path": "tc" if ctx.get_option("last_path") == 2 else "simt", "degree_s": t1 - t0,
               "eigs_s": t2 - t1, "total_s": t2 - t0, "applies": int(info.applies), "restarts": int(info.restarts),
               "converged": int(info.converged), "of": k + 1, "max_residual": float(info.max_residual),
               "seconds_in_apply": float(info.seconds_apply), "lambda_1": float(lam[1]), "lambda_k": float(lam[k])}
        if name.startswith("C3"):
            t3 = time.perf_counter()
            bx, outcome, lam2, U2, recs = ctx.beta_flow(k, b, 1.0, beta_start=1.0, beta_max=1000.0, tol=1e-6, max_applies=400)
            t4 = time.perf_counter()
            rec["flow"] = {"grid": "beta = 1, 2, 4, ... <= 1000 (dyadic), warm-started probes", "seconds": t4 - t3,
                           "beta_x": bx, "outcome": outcome, "probes": len(recs),
                           "applies": int(sum(r["applies"] for r in recs)), "n_eff_at_beta_x": recs[-1]["n_eff"],
                           "d_hat_at_beta_x": recs[-1]["d_hat"]}
        ctx.close()
        del ctx, X
        torch.cuda.empty_cache()
        res.append(rec)
    res.append(ladder(fd, dev, full))
    return res


def ladder(fd, dev, full=False):
    """The (n, beta) continuation of Sec. 1 at fixed beta = 2: nested levels (first n rows of one draw), each level's solve
    warm-started from the previous level's eigenpairs through the out-of-sample extension (fd_ladder_start), with the
    cold-started solve of the same level beside it.  Default: 2^15 -> 2^16 -> 2^17 (k = 64, b = 32); --eigs-full: the
    2^16 ... 2^20 ladder with k = 128, b = 64."""
    import torch
    import workloads
    levels, k, b = ([1 << e for e in range(16, 21)], 128, 64) if full else ([1 << 15, 1 << 16, 1 << 17], 64, 32)
    Xall = torch.from_numpy(workloads.torus6(levels[-1], seed=42)).to(dev)
    m_max = (max(2 * (k + 1) + b, 4 * b) + b - 1) // b * b
    out = {"workload": f"6-torus ladder N = {levels}, k={k}, b={b}, alpha=1, beta=2.0, tol=1e-6", "levels": []}
    prev = None
    t_all = time.perf_counter()
    for n in levels:
        X = Xall[:n]
        ctx = fd.Context(X, b_max=b, m_max=m_max)
        t0 = time.perf_counter()
        ctx.degree(2.0, 1.0)
        rec = {"N": n}
        if prev is not None:
            pctx, plam, pU = prev
            Q0 = ctx.ladder_start(pctx, X, pU, plam)
            t1 = time.perf_counter()
            lam, U, info = ctx.eigs(k, b, tol=1e-6, max_applies=400, Q0=Q0, allow_not_converged=True)
            rec.update(extend_s=t1 - t0, warm_s=time.perf_counter() - t1, warm_applies=int(info.applies),
                       warm_converged=int(info.converged))
            pctx.close()
        t2 = time.perf_counter()
        lam_c, U_c, info_c = ctx.eigs(k, b, tol=1e-6, max_applies=400, allow_not_converged=True)
        rec.update(cold_s=time.perf_counter() - t2, cold_applies=int(info_c.applies), cold_converged=int(info_c.converged))
        if prev is None:
            lam, U = lam_c, U_c
        else:
            rec["max_eval_diff_warm_vs_cold"] = float(abs(lam - lam_c).max())
        out["levels"].append(rec)
        prev = (ctx, lam, U)
    prev[0].close()
    out["seconds"] = time.perf_counter() - t_all
    return out


def cpu_baseline(X, V, cfg):
    from oracle import blocked
    import workloads
    N, b = cfg["N"], cfg["b"]
    cores = blocked.threads()
    rows_n = int(max(16, min(N, 12.0 * cores * 2.0e7 / N)))
    rows = workloads.row_sample(N, rows_n, seed=11)
    X64 = X.astype(np.float64)
    V64 = np.ascontiguousarray(V.astype(np.float64))
    w = np.full(N, 1e-2)
    oracle_step(X64, V64, cfg["beta"], cfg["alpha"], rows[:16], w)
    t0 = time.perf_counter()
    oracle_step(X64, V64, cfg["beta"], cfg["alpha"], rows, w)
    dt = time.perf_counter() - t0
    return {"value": rows_n * float(N) * (b + 2) / dt, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": dt,
            "sample": f"{rows_n} sampled rows x all {N} columns, three passes (b = 1, 1, {b}), float64, rows.c + OpenMP"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--n", type=int, default=20, help="log2 of the number of points (default 20: the headline size)")
    ap.add_argument("--path", default="", choices=["", "auto", "simt", "tc"])
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline leg")
    ap.add_argument("--no-eigs", action="store_true", help="skip the time-to-k-eigenpairs leg")
    ap.add_argument("--eigs-full", action="store_true", help="also time the eigensolve at N = 2^20 (k = 128, b = 64)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
