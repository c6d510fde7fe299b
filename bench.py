#!/usr/bin/env python
"""Benchmark of the FlashDiffusion hot path on B200.

Headline metric: kernel-apply throughput N^2 * b / t_apply (pair-columns per second) of the fp32-grade block product
Y = diag(s) K diag(s) V on the headline workload (6-torus in R^12, N = 2^20, block b = 64, alpha = 1, beta = 2), with
its fraction of the binding roofline (one exponential per pair on the MUFU).  One timed step is one pass of the whole
hot path at a fresh bandwidth -- degree pass q = K 1, second normalisation pass d = q^-a * K q^-a, scale vector s, block
product -- so the step time, the degree passes and the reduced-precision product are reported beside the headline, as
are the end-to-end figure through the C ABI with host buffers, the CPU float64 oracle on the box's own cores, and the
time to k eigenpairs on the five benchmark configurations.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--n LOG2N]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU float64 oracle on a bounded row sample of the same
workload instead.  `--gpus N` without a launcher starts N ranks itself, one per GPU.  With N > 1 the data set is row-
sharded (Sec. 3 of the paper): every rank holds all points and evaluates N / world rows of every quadratic pass, the
rows of each result are gathered over NCCL, so the total work is fixed ("scaling": "strong") and `value` is the one
job's N^2 b over the slowest rank's time.  `--replicas` runs N independent copies instead ("weak").
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "kernel-apply pair-columns per second of the block product Y = M V (N^2 * b / t_apply)"
UNIT = "pair*cols/s"

# DRAM bytes per launch of the timed block-product kernel (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture of this kernel at N = 2^20, single-pass metrics), keyed by the kernel that bench times; None = not captured.
NCU_TRAFFIC_BYTES = {"k_tc<64, block>": 17.139e9 + 2.180e9, "k_simt": None}


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
    return X, V, dict(workload=f"C5: 6-torus R^12 + noise 0.01, N=2^{log2n}, b=64, alpha=1, beta=2.0, fp32-grade mode",
                      N=N, D=12, b=64, alpha=1.0, beta=2.0, l2_note=(f"inputs (X, V, Y: {4.0 * N * (12 + 128) / 1e9:.2f} GB) " +
                               ("exceed the 126 MB L2" if 4.0 * N * (12 + 128) > 126e6 else
                                "FIT in the 126 MB L2: a reduced-size run, not a headline number")))


# ------------------------------------------------------------------------------------------- CPU oracle arm
def oracle_sample(X64, V64, beta, rows, w):
    """A bounded sample of the step on the CPU oracle: the three passes on `rows` rows; returns (seconds of the two
    degree passes, seconds of the block product).  The second pass and the product need q, s on all columns: a positive
    surrogate vector of the right magnitude stands in (the cost per pair is what is timed, not the values)."""
    from oracle import blocked
    t0 = time.perf_counter()
    blocked.rows_apply_general(X64, beta, None, rows=rows, want_rowsq=True)
    blocked.rows_apply_general(X64, beta, None, rows=rows, left=w, right=w)
    t1 = time.perf_counter()
    blocked.rows_apply_general(X64, beta, V64, rows=rows, left=w, right=w)
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1


def oracle_rows_for(N, cores, seconds):
    # ~4e7 pair evaluations per core-second for the b = 64 product on these hosts
    return int(max(16, min(N, seconds * cores * 2.5e7 / N)))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import blocked
    import workloads
    X, V, cfg = workload(args.n)
    N, b = cfg["N"], cfg["b"]
    X64 = X.astype(np.float64)
    V64 = np.ascontiguousarray(V.astype(np.float64))
    cores = blocked.threads()
    rows_n = oracle_rows_for(N, cores, 5.0)
    rows = workloads.row_sample(N, rows_n, seed=11)
    w = np.full(N, 1e-2)
    oracle_sample(X64, V64, cfg["beta"], rows[: max(16, rows_n // 8)], w)
    t_deg = t_app = 0.0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        a, c = oracle_sample(X64, V64, cfg["beta"], rows, w)
        t_deg += a; t_app += c
    dt = (time.perf_counter() - t0) / args.steps
    value = rows_n * float(N) * b / (t_app / args.steps)
    sample = (f"{rows_n} sampled rows x all {N} columns per step: block product (b = {b}) timed for the metric, the two "
              f"degree passes beside it; float64, rows.c + OpenMP")
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "whole_step": {"pair_cols_per_s": rows_n * float(N) * (b + 2) / dt}, "gpu_launches": 0}
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
    """Whole-job throughput: the units all ranks processed over the slowest rank's time.  Independent replicas process
    the full workload each; row-sharded ranks process 1 / world of one workload each."""
    return units_per_rank * world / (ms * 1e-3)


def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def spawn_ranks(args) -> int:
    """`python bench.py --gpus N` without a launcher: start N local ranks (one per GPU) of this same script."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


# ------------------------------------------------------------------------------------------- GPU arm
def run_gpu(args):
    # stdout carries the one JSON line: NCCL prints a version banner there at NCCL_DEBUG=VERSION (and at WARN), so that
    # setting is dropped; the library reads the variable once, so this has to happen before torch loads it
    if os.environ.get("NCCL_DEBUG", "").upper() == "VERSION":
        del os.environ["NCCL_DEBUG"]
    import torch
    import __graft_entry__ as entry
    entry.build()
    import paper_2609_38198_b200 as fd

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1 or args.force_shard:
        import torch.distributed as dist_mod
        dist = dist_mod
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if world == 1:                       # --force-shard on one GPU: a one-rank NCCL group exercises the exchange path
            os.environ.setdefault("MASTER_PORT", str(free_port()))
            os.environ.setdefault("RANK", "0")
            os.environ.setdefault("WORLD_SIZE", "1")
        torch.cuda.set_device(local)
        import datetime
        # generous: in replica mode the other ranks wait at the last barrier while rank 0 runs the eigensolver leg
        dist.init_process_group("nccl", device_id=torch.device("cuda", local), timeout=datetime.timedelta(minutes=60))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    sharded = dist is not None and not args.replicas
    transport = None
    if sharded:
        # rows gathered on the NCCL group, the eigensolver's small host sums on a gloo group
        transport = fd.TorchDistTransport(rank, world, group=None, host_group=dist.new_group(backend="gloo"))

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
    shard = fd.Shard(transport, N, b, dev, stream=stream) if sharded else None
    if sharded:
        ctx.set_shard(shard)
    cfg["parallelism"] = (f"rows sharded over {world} ranks, result rows gathered (NCCL all-gather)" if sharded else
                          f"{world} independent replicas" if world > 1 else "single GPU")

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

    # the clock sampler starts before the warm-up (nvidia-smi's own start-up can stall the GPU for a moment); only the
    # samples taken during the timed region are kept
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    sampler.lines.clear()
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
    path_used = "tc" if ctx.get_option("last_path") == 2 else "simt"

    # SM clock the block-product kernel actually runs at (it draws the board's power limit, so the clock sags): median of
    # nvidia-smi samples over a loop of block products alone, and, as a cross-check from the kernel itself, the SM cycles
    # its first CTA counted over the kernel's duration (a lower bound: the count excludes launch and tail)
    sustained_mhz = cycles_mhz = None
    if path_used == "tc":
        s2 = ClockSampler(local)
        if rank == 0:
            s2.start()
            time.sleep(0.5)
            s2.lines.clear()
        e0, e1 = ev(), ev()
        reps = max(4, int(2000.0 / max(app_ms, 1.0)))
        e0.record(stream)
        for _ in range(min(reps, 50)):
            ctx.apply(Vd, out=Yd)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        if rank == 0:
            c2 = s2.stop()
            sustained_mhz = c2.get("sm_mhz")
        cycles_mhz = ctx.get_option("tc_cycles") / (e0.elapsed_time(e1) / min(reps, 50) * 1e3)
    # the reduced-precision product, reported separately (three repeats)
    fast_ms = None
    if path_used == "tc":
        ts = []
        for _ in range(3):
            e0, e1 = ev(), ev()
            e0.record(stream); ctx.apply(Vd, out=Yd, prec=fd.FD_PREC_FAST); e1.record(stream)
            torch.cuda.synchronize(dev)
            ts.append(e0.elapsed_time(e1))
        fast_ms = float(np.median(ts))

    # end-to-end through the public API with host buffers: H2D of X and V, D2H of Y every step
    def e2e_step():
        Xd.copy_(Xh, non_blocking=True)
        Vd.t().copy_(Vh, non_blocking=True)
        c2 = fd.Context(Xd, b_max=b, m_max=0)
        if args.path:
            c2.set_option("path", {"auto": 0, "simt": 1, "tc": 2}[args.path])
        if sharded:
            c2.set_shard(shard)
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
    # pair-columns one rank processes per block product: all of them as a replica, its rows' share when sharded
    units = float(N) * N * b / (world if sharded else 1)

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        rates = fd.fd_unit_peaks(dev)
        D = cfg["D"]
        sm_max = float(peaks.get("sm_max_mhz", 1965.0))
        pairs_per_s = units / b / (app_ms * 1e-3)                 # per GPU: the roofline is one GPU's
        mufu_peak = rates["sm_count"] * rates["ex2_per_clk_sm"] * sm_max * 1e6         # exp / s at the maximum SM clock
        fma_peak = rates["sm_count"] * rates["ffma_per_clk_sm"] * sm_max * 1e6
        if path_used == "simt":
            # everything on the FMA pipe: per pair 2 D (difference form) + b (product) + ~3 issue slots
            peak_pairs = fma_peak / (2 * D + b + 3)
            binder = "fma_pipe (direct-difference distance + block product on FFMA)"
            kernel_name = "k_simt"
        else:
            peak_pairs = mufu_peak
            binder = "mufu (one ex2 per pair; distance and product on the tensor cores)"
            kernel_name = "k_tc<64, block>"
        roofline = {"bound": "alu", "kernel": f"{kernel_name}: block product Y = M V (dominant kernel)", "binder": binder,
                    "achieved": pairs_per_s / 1e9, "peak": peak_pairs / 1e9, "unit": "Gpairs/s",
                    "frac": pairs_per_s / peak_pairs,
                    "peak_source": (f"measured unit rate ({rates['ex2_per_clk_sm']:.2f} ex2/clk/SM, {rates['sm_count']} SMs; "
                                    f"fd_unit_peaks in this run) x maximum SM clock {sm_max:.0f} MHz ({peak_kind})"),
                    "sustained_sm_mhz": sustained_mhz, "sm_mhz_from_kernel_cycles": cycles_mhz,
                    "frac_at_sustained_clock": (pairs_per_s / (peak_pairs * sustained_mhz / sm_max)) if sustained_mhz else None,
                    "traffic": NCU_TRAFFIC_BYTES.get(kernel_name) if N == (1 << 20) else None,
                    "algorithmic_bytes": 4.0 * N * (D + 2 * b + 2),
                    "tensor_work_per_tile_clk": {"gram_3_mma_ss_n128": 3 * rates["clk_mma_ss_n128"],
                                                 "product_24_mma_ts_n64": 24 * rates["clk_mma_ts_n64"],
                                                 "mufu_128x128_exps": 128 * 128 / rates["ex2_per_clk_sm"]},
                    "unit_rates": rates}
        deg_pairs_per_s = 2.0 * units / b / (deg_ms * 1e-3)       # per GPU: pairs SERVED per second (both passes)
        # exponentials the two passes actually execute: all N^2 per pass, or -- on the Gram-form kernels of an unsharded
        # context, which use K = K^T -- only the 128 x 128 tiles on or above the diagonal: T (T + 1) / 2 tiles, T = ceil(N / 256) * 2
        sym_on = path_used == "tc" and not sharded and ctx.get_option("sym") == 1
        T = -(-N // 256) * 2
        deg_exps = 2.0 * (T * (T + 1) // 2 * 16384 if sym_on else float(N) * N / (world if sharded else 1))
        out = {"metric": METRIC, "value": job_value(units, world, app_ms), "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "strong" if sharded else "weak",
               "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg, "clocks": clocks,
               "apply_ms": app_ms, "path": path_used, "roofline": roofline,
               "whole_step": {"ms": step_ms, "pair_cols_per_s": job_value(units * (b + 2) / b, world, step_ms),
                              "note": "degree pass + second normalisation pass + scale vector + block product"},
               "degree_passes": {"ms_both": deg_ms, "pairs_served_per_s": deg_pairs_per_s, "symmetric_half_work": bool(sym_on),
                                 "executed_exponentials_both_passes": deg_exps,
                                 "frac_of_mufu_peak": deg_exps / (deg_ms * 1e-3) / mufu_peak,
                                 "note": "frac counts the exponentials actually executed (never the pairs served), against the same MUFU peak"},
               "fast_mode_apply": None if fast_ms is None else {
                   "ms": fast_ms, "pair_cols_per_s": units / (fast_ms * 1e-3), "frac_of_mufu_peak": units / b / (fast_ms * 1e-3) / mufu_peak,
                   "note": "FD_PREC_FAST: single fp16 operands, relative Frobenius error ~2e-4 (bound 3e-3); reported separately"},
               "e2e": {"value": job_value(units, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                       "note": "host buffers: H2D of X and V, fd_create, degree passes, block product, D2H of Y",
                       "h2d_bytes_per_step": int(Xh.numel() * 4 + Vh.numel() * 4), "d2h_bytes_per_step": int(Yh.numel() * 4)},
               "gpu_launches": int(launches), "workspace_bytes": ctx.workspace_bytes}
        if world == 1 and not sharded:
            out["sharded_rank_share"] = sharded_rank_share(fd, dev, Xd, Vd, Yd, beta, alpha, b)
        if not args.no_cpu and world == 1:
            out["cpu_baseline"] = cpu_baseline(X, V, cfg)
    ctx.close()
    if not args.no_eigs and (rank == 0 or sharded):
        # one GPU or replicas: rank 0 alone; row-sharded: every rank takes part in the sharded solves
        del Xd, Vd, Yd
        torch.cuda.empty_cache()
        eigs = time_to_k_eigs(fd, dev, args, transport if sharded else None)
        if rank == 0:
            out["time_to_k_eigs"] = eigs
    if rank == 0:
        print(json.dumps(out), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def time_to_k_eigs(fd, dev, args, transport=None):
    """Second half of the metric: wall time from a fresh bandwidth to k eigenpairs (degree passes + fd_eigs) on the five
    benchmark configurations at their full sizes (C2 at all four bandwidths; non-convergence within the apply budget is a
    reported outcome there), the whole dyadic bandwidth flow on C3, and the nested-level ladder with the bandwidth
    re-optimised on every level.  Host wall clock around synchronous calls.  With a transport (row-sharded ranks) every
    rank runs the same solves on its rows; only the large configurations are run then (C3 with its flow, C4, C5)."""
    import torch
    import workloads
    res = []
    # (name, points, k, b, beta, max_applies)
    cases = [("C1 circle", workloads.circle(2048), 8, 8, 200.0, 600),
             ("C2 2-torus", workloads.torus2(16384, seed=42), 32, 16, 10.0, 600),
             ("C2 2-torus", None, 32, 16, 30.0, 600),
             ("C2 2-torus", None, 32, 16, 100.0, 1000),
             ("C2 2-torus", None, 32, 16, 300.0, 1000),
             ("C3 6-torus", workloads.torus6(1 << 17, seed=42), 64, 32, 2.0, 600),
             ("C4 latent torus R^30", workloads.latent_torus(262144, seed=42), 32, 32, 2.0, 600)]
    if not args.no_c5_eigs:
        cases.append(("C5 6-torus", workloads.torus6(1 << 20, seed=42), 128, 64, 2.0, 400))
    if transport is not None:
        cases = [cse for cse in cases if cse[0][:2] in ("C3", "C4", "C5")]
    if args.eigs_case:
        # restrict the leg to one configuration (for profiling a single solve); C2 keeps its four bandwidths
        pts = None
        picked = []
        for cse in cases:
            pts = cse[1] if cse[1] is not None else pts
            if cse[0].startswith(args.eigs_case):
                picked.append((cse[0], pts) + cse[2:])
        cases = picked
    Xnp = None
    for name, Xc, k, b, beta, max_applies in cases:
        if Xc is not None:
            Xnp = Xc
        N = Xnp.shape[0]
        X = torch.from_numpy(Xnp).to(dev)
        m_max = args.m_max if args.m_max > 0 else default_m_max(k, b)
        ctx = fd.Context(X, b_max=b, m_max=m_max)
        if transport is not None:
            ctx.set_shard(fd.Shard(transport, N, b, dev))
        ctx.degree(beta, 1.0)                                        # warm-up of both passes
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        ctx.degree(beta, 1.0)
        t1 = time.perf_counter()
        lam, U, info = ctx.eigs(k, b, tol=1e-6, max_applies=max_applies, allow_not_converged=True)
        t2 = time.perf_counter()
        rec = {"workload": f"{name}: N={N}, D={Xnp.shape[1]}, k={k}, b={b}, alpha=1, beta={beta}, tol=1e-6",
               "path": "tc" if ctx.get_option("last_path") == 2 else "simt", "degree_s": t1 - t0,
               "eigs_s": t2 - t1, "total_s": t2 - t0, "applies": int(info.applies), "restarts": int(info.restarts),
               "converged": int(info.converged), "of": k + 1, "max_residual": float(info.max_residual), "m_max": m_max,
               "seconds_in_apply": float(info.seconds_apply), "lambda_1": float(lam[1]), "lambda_k": float(lam[k])}
        if name.startswith("C3"):
            t3 = time.perf_counter()
            bx, outcome, lam2, U2, recs = ctx.beta_flow(k, b, 1.0, beta_start=1.0, beta_max=1000.0, tol=1e-6, max_applies=400)
            t4 = time.perf_counter()
            rec["flow"] = {"grid": "beta = 1, 2, 4, ... <= 1000 (dyadic), warm-started probes", "seconds": t4 - t3,
                           "beta_x": bx, "outcome": outcome, "probes": len(recs),
                           "applies": int(sum(r["applies"] for r in recs)), "n_eff_at_beta_x": recs[-1]["n_eff"],
                           "d_hat_at_beta_x": recs[-1]["d_hat"]}
            # the same sweep as a precision cascade (Sec. 2.3): reduced-precision kernels explore, fp32-grade kernels resolve
            t5 = time.perf_counter()
            bxc, outc, lam3, U3, stg = ctx.beta_flow_cascade(k, b, 1.0, [(fd.FD_PREC_FAST, 0.0, 0.0), (fd.FD_PREC_FP32, 0.0, 0.0)],
                                                             beta_start=1.0, beta_max=1000.0, max_applies=400)
            t6 = time.perf_counter()
            rec["cascade"] = {"stages": "FD_PREC_FAST (eta 1e-3, tol 1e-3) -> FD_PREC_FP32 (eta 1e-7, tol 1e-6)", "seconds": t6 - t5,
                              "beta_x": bxc, "outcome": outc, "probes_per_stage": [len(x) for x in stg],
                              "applies_per_stage": [int(sum(r["applies"] for r in x)) for x in stg],
                              "max_eval_diff_vs_flow": float(abs(lam3 - lam2).max())}
        ctx.close()
        del ctx, X
        torch.cuda.empty_cache()
        res.append(rec)
    if not args.eigs_case and transport is None:
        res.append(ladder(fd, dev, args.ladder_full))
        res.append({"t6_validation": t6_validation(fd, dev, args.t6_full)})
        res.append({"paper_shape_context": paper_shape_context(fd, dev)})
    return res


def t6_validation(fd, dev, full=False):
    """The paper's T^6 validation sweep (Sec. 3, Fig. 1(b), 1(c)): anisotropic radii, alpha = 1/2, k = 3, seed 42 per N, the
    bandwidth flow from beta_0 of Eq. 7; per N the selected beta_x and the post-hoc squared-RV overlap of the leading two
    nontrivial Markov modes with (cos, sin) of the largest circle, with the printed values beside them (another RNG).
    Default N = 2^10 ... 2^17; --t6-full continues to 2^20."""
    import torch
    import workloads
    printed = {}
    try:
        with open(os.path.join(ROOT, "tests", "golden", "t6_bandwidth_table.txt")) as f:
            for line in f:
                if line[0].isdigit():
                    r = line.strip().split(",")
                    printed[int(r[0])] = (float(r[1]), float(r[3]))
    except OSError:
        pass
    printed_s = {1024: 6.03, 16384: 6.37, 65536: 15.98, 131072: 61.58, 262144: 147.90, 524288: 464.25, 1048576: 2225.04}
    out = []
    for e in range(10, 21 if full else 18):
        N = 1 << e
        X, ang = workloads.torus6_paper(N, seed=42, return_angles=True)
        ctx = fd.Context(torch.from_numpy(X).to(dev), b_max=8, m_max=64)
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        bx, outcome, lam, U, recs = ctx.beta_flow(3, 8, 0.5, beta_start=0.0, beta_max=1000.0)
        dt = time.perf_counter() - t0
        psi = ctx.scale_by_degree(U, -0.5).cpu().numpy().astype(np.float64)[:, 1:3]
        path = "tc" if ctx.get_option("last_path") == 2 else "simt"
        ctx.close()
        # squared RV coefficient of the two centred 2-column blocks (float64, whitened cross-covariance)
        A = psi - psi.mean(axis=0)
        B = np.stack([np.cos(ang[:, 5]), np.sin(ang[:, 5])], axis=1)
        B = B - B.mean(axis=0)

        def inv_sqrt(G):
            w, Q = np.linalg.eigh(G)
            return (Q / np.sqrt(w)) @ Q.T
        C = inv_sqrt(A.T @ A) @ (A.T @ B) @ inv_sqrt(B.T @ B)
        score = float((C * C).sum() / 2.0)
        rec = {"N": N, "beta_x": bx, "outcome": outcome, "probes": len(recs), "applies": int(sum(r["applies"] for r in recs)),
               "flow_s": dt, "path": path, "n_eff": recs[-1]["n_eff"], "d_hat": recs[-1]["d_hat"], "one_minus_overlap": 1.0 - score}
        if N in printed:
            rec["printed_beta_x"], rec["printed_one_minus_overlap"] = printed[N][0], 1.0 - printed[N][1]
        if N in printed_s:
            rec["printed_time_to_solution_s_other_gpu"] = printed_s[N]     # Fig. 1(a): flow + ladder + solver, one RTX PRO 6000
        out.append(rec)
    return out


def paper_shape_context(fd, dev):
    """Context rows: the raw kernel application K V on the paper's own race shape (App. B: anisotropic T^6 zero-padded to
    D = 32, beta = 1, b = 1 and b = 8), fp32-grade mode, with the times the paper prints for its kernel on another GPU
    (RTX PRO 6000) beside them.  Not the metric's configuration and not a target: context."""
    import torch
    import workloads
    printed = {(1 << 17, 1): 0.03901, (1 << 17, 8): 0.04319, (1 << 20, 1): 2.083, (1 << 20, 8): 2.897}
    out = []
    for e in (17, 20):
        N = 1 << e
        X = torch.from_numpy(workloads.torus6_paper(N, seed=42)).to(dev)
        ctx = fd.Context(X, b_max=8, m_max=0)
        for b in (1, 8):
            V = torch.from_numpy(np.ascontiguousarray(workloads.block(N, b, seed=7).T)).to(dev).t()
            Y = torch.empty((b, N), dtype=torch.float32, device=dev).t()
            ctx.apply_general(1.0, V, out=Y)
            torch.cuda.synchronize(dev)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = 3
            e0.record()
            for _ in range(reps):
                ctx.apply_general(1.0, V, out=Y)
            e1.record()
            torch.cuda.synchronize(dev)
            t = e0.elapsed_time(e1) / reps * 1e-3
            out.append({"N": N, "D": 32, "beta": 1.0, "b": b, "seconds": t, "pair_cols_per_s": float(N) * N * b / t,
                        "path": "tc" if ctx.get_option("last_path") == 2 else "simt",
                        "printed_seconds_other_gpu": printed[(N, b)]})
        ctx.close()
    return out


def sharded_rank_share(fd, dev, Xd, Vd, Yd, beta, alpha, b):
    """What ONE rank of a row-sharded job computes, measured on this GPU with the exchange stubbed out (a transport whose
    gathers and sums do nothing): the block product and the degree passes over rank 0's rows of a 2-, 4- and 8-rank
    partition, pack / unpack copies of the gather included, the NCCL transfer itself (N b 4 bytes per product over
    NVLink) not.  The figures say how the work divides; they are not a multi-GPU measurement."""
    import torch
    N = Xd.shape[0]

    class Stub:
        def __init__(self, world):
            self.rank, self.world = 0, world

        def allreduce_sum_host(self, arr, device, stream):
            pass

        def allgather(self, send, recv, stream):
            pass

    out = []
    for world in (2, 4, 8):
        ctx = fd.Context(Xd, b_max=b, m_max=0)
        ctx.set_shard(fd.Shard(Stub(world), N, b, dev))
        ctx.degree(beta, alpha)
        ctx.apply(Vd, out=Yd)
        torch.cuda.synchronize(dev)
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record()
        ctx.degree(beta, alpha)
        e[1].record()
        for _ in range(3):
            ctx.apply(Vd, out=Yd)
        e[2].record()
        torch.cuda.synchronize(dev)
        r0, r1 = fd.fd_shard_rows(N, world, 0)
        out.append({"world": world, "rows_of_rank_0": r1 - r0, "apply_ms": e[1].elapsed_time(e[2]) / 3.0,
                    "degree_passes_ms": e[0].elapsed_time(e[1]), "gather_bytes_per_apply": int(N) * b * 4})
        ctx.close()
    return out


def default_m_max(k, b):
    """Basis capacity for fd_eigs: three times the wanted pairs plus two blocks, at least four blocks and at least 64
    columns.  The thick restart keeps 3/5 of the capacity, so this keeps about twice the wanted pairs: room for the rest
    of an eigenvalue cluster that the request cuts (the 6-torus at k = 128 cuts a 160-fold cluster: with room for it all
    129 pairs converge in 44 block products, with 2 (k + 1) + b columns only 73 do in 125)."""
    return (max(3 * (k + 1) + 2 * b, 4 * b, 64) + b - 1) // b * b


def ladder(fd, dev, full=False):
    """The (n, beta) continuation of Sec. 1: nested levels (first n rows of one draw).  On every level the bandwidth is
    re-optimised by the dyadic flow started one probe below the previous level's beta_x, and every probe's solve is
    warm-started: the first from the previous level's eigenpairs through the out-of-sample extension (fd_ladder_start),
    the others from the previous probe.  A cold-started solve at the level's beta_x stands beside it.
    Default: 2^15 -> 2^16 -> 2^17 (k = 64, b = 32); --ladder-full: config 5 itself, 2^16 ... 2^20 with k = 128, b = 64."""
    import torch
    import workloads
    levels, k, b = ([1 << e for e in range(16, 21)], 128, 64) if full else ([1 << 15, 1 << 16, 1 << 17], 64, 32)
    Xall = torch.from_numpy(workloads.torus6(levels[-1], seed=42)).to(dev)
    m_max = default_m_max(k, b)
    out = {"workload": f"6-torus ladder N = {levels}, k={k}, b={b}, alpha=1, tol=1e-6, beta re-optimised per level", "levels": []}
    prev = None
    t_all = time.perf_counter()
    for n in levels:
        X = Xall[:n]
        ctx = fd.Context(X, b_max=b, m_max=m_max)
        rec = {"N": n}
        t0 = time.perf_counter()
        if prev is None:
            bx, outcome, lam, U, recs = ctx.beta_flow(k, b, 1.0, beta_start=0.5, beta_max=64.0, tol=1e-6, max_applies=400)
        else:
            pctx, plam, pU, pbx = prev
            ctx.degree(pbx, 1.0)                                    # the extension is scaled by this level's degrees
            Q0 = ctx.ladder_start(pctx, X, pU, plam)
            rec["extend_s"] = time.perf_counter() - t0
            bx, outcome, lam, U, recs = ctx.beta_flow(k, b, 1.0, beta_start=pbx / 2.0, beta_max=pbx * 16.0, tol=1e-6,
                                                      max_applies=400, Q0=Q0)
            pctx.close()
        rec.update(flow_s=time.perf_counter() - t0, beta_x=bx, outcome=outcome, probes=len(recs),
                   flow_applies=int(sum(r["applies"] for r in recs)), probe_betas=[r["beta"] for r in recs])
        t2 = time.perf_counter()
        ctx.degree(bx, 1.0)
        lam_c, U_c, info_c = ctx.eigs(k, b, tol=1e-6, max_applies=400, allow_not_converged=True)
        rec.update(cold_at_beta_x_s=time.perf_counter() - t2, cold_applies=int(info_c.applies), cold_converged=int(info_c.converged),
                   max_eval_diff_flow_vs_cold=float(abs(lam - lam_c).max()))
        out["levels"].append(rec)
        prev = (ctx, lam, U, bx)
    prev[0].close()
    out["seconds"] = time.perf_counter() - t_all
    return out


def cpu_baseline(X, V, cfg):
    from oracle import blocked
    import workloads
    N, b = cfg["N"], cfg["b"]
    cores = blocked.threads()
    rows_n = oracle_rows_for(N, cores, 10.0)
    rows = workloads.row_sample(N, rows_n, seed=11)
    X64 = X.astype(np.float64)
    V64 = np.ascontiguousarray(V.astype(np.float64))
    w = np.full(N, 1e-2)
    oracle_sample(X64, V64, cfg["beta"], rows[:16], w)
    t_deg, t_app = oracle_sample(X64, V64, cfg["beta"], rows, w)
    return {"value": rows_n * float(N) * b / t_app, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": t_deg + t_app,
            "whole_step_pair_cols_per_s": rows_n * float(N) * (b + 2) / (t_deg + t_app),
            "sample": (f"{rows_n} sampled rows x all {N} columns: block product (b = {b}) timed for the metric, the two degree "
                       f"passes beside it; float64, rows.c + OpenMP")}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--n", type=int, default=20, help="log2 of the number of points (default 20: the headline size)")
    ap.add_argument("--path", default="", choices=["", "auto", "simt", "tc"])
    ap.add_argument("--replicas", action="store_true", help="with --gpus N > 1: N independent replicas instead of row sharding")
    ap.add_argument("--force-shard", action="store_true", help="one GPU: run the row-sharded code path on a one-rank NCCL group")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline leg")
    ap.add_argument("--no-eigs", action="store_true", help="skip the time-to-k-eigenpairs leg")
    ap.add_argument("--no-c5-eigs", action="store_true", help="skip the eigensolve at N = 2^20 (k = 128, b = 64; about 80 s)")
    ap.add_argument("--eigs-case", default="", choices=["", "C1", "C2", "C3", "C4", "C5"],
                    help="time-to-k-eigenpairs leg: only this configuration (and no ladder)")
    ap.add_argument("--m-max", type=int, default=0, help="basis capacity of the eigensolver legs (0: default_m_max(k, b))")
    ap.add_argument("--t6-full", action="store_true", help="T^6 validation sweep up to N = 2^20 instead of 2^17")
    ap.add_argument("--ladder-full", action="store_true", help="run config 5's own ladder (2^16 ... 2^20, k = 128, b = 64; many minutes)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    run_gpu(args)


if __name__ == "__main__":
    main()
