#!/usr/bin/env python
"""Benchmark of the Sinkhorn hot path: iterations/s at n = 32768, fp32 dense K, one B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 1..5]

A step is one full solve of the configuration (its stated number of iterations: a row pass and a
column pass each) through fs_iterate, on seeded synthetic inputs that are resident in HBM before
the timed region starts.  Rank 0 prints ONE JSON line.  Keys beyond the basic contract:

  roofline      dominant kernel (config 4: the single-read fused iteration kernel): algorithmic bytes
                per launch over its average launch interval against the measured HBM copy rate of this
                pool.  `frac` is SUSTAINED (the timed region itself); `burst` holds the same for a short
                loop of single launches from an idle GPU; both carry the SM clock sampled meanwhile and
                time x clock (SM cycles per launch)
  other_paths   config 4 on the two-pass path (K streamed twice per iteration): the row pass and the
                column pass each timed alone, and whole iterations
                and through the implicit-kernel path (fs_create_points) with its ex2-rate ("alu") roofline
  cpu_baseline  the fp64 CPU checker timed on this machine's host cores on a few iterations, with all
                cores (OpenMP) and on one thread
  e2e           the same metric through fs_solve_host: host buffers in, host buffers out, all
                host<->device copies inside the timed region
  clocks        SM clock and throttle reasons sampled with nvidia-smi during the timed region
  other_configs it/s of configurations 1, 2, 3 and 5 from short runs of the same kind, each with the kernel
                path the library chose and the SM clock sampled during it (N = 1 only)

With --impl reference the CPU checker is what gets timed (same config, metric and unit); under a
multi-process launch only rank 0 runs it.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2502_07021_b200 import distributed as fsdist  # noqa: E402
from paper_2502_07021_b200 import workloads  # noqa: E402

METRIC = "sinkhorn_iterations_per_s"
UNIT = "it/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/
# (kernel name, n) -> bytes; a capture at n = 16384 is scaled by 4 for n = 32768 (traffic is proportional to n*n).
TRAFFIC_BYTES_PER_LAUNCH = {
    ("fused_iteration_kernel", 16384): 1.074029e9 + 1.96e6,
    ("fused_iteration_kernel", 32768): 4 * (1.074029e9 + 1.96e6),
    # the implicit pass reads only the operands of the two clouds from DRAM (n*d-sized, not n*n): captured at n = 16384
    ("implicit_pass_kernel", 16384): 8.51e6,
    ("implicit_pass_kernel", 32768): 2 * 8.51e6,
    ("log_row_pass_kernel", 16384): 1.074043e9 + 3.39e6,
    ("fused_log_iteration_kernel", 16384): 1.073997e9 + 4.36e6,
    ("batched_tc_kernel", 8192): 281.10e6 + 3.51e6,
    # captured on a 200-iteration launch; K is read from DRAM once per launch whatever the iteration count
    ("persistent_iterations_kernel", 4096): 67.26e6 + 1.4e6,
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


class ClockSampler:
    """nvidia-smi sampling in a child process while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except (OSError, ValueError):
            self.proc = None

    def stop(self):
        if self.proc is None:
            return None
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smmax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smmax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smmax), "reasons": sorted(reasons),
                "samples": len(sm)}


class NvmlSampler:
    """SM clock and throttle reasons read through NVML from a thread of this process, every few milliseconds:
    for timed loops too short for the nvidia-smi child process to see (reading only, nothing is set)."""

    def __init__(self, index: int, period_s: float = 0.004):
        self.index, self.period, self.samples, self.reasons = index, period_s, [], 0
        self.thread = None
        self.stop_flag = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
                self.reasons |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv is None:
            return
        import threading
        self.samples, self.reasons, self.stop_flag = [], 0, False
        self.thread = threading.Thread(target=self._loop, daemon=True)
        self.thread.start()

    def stop(self):
        if self.nv is None or self.thread is None:
            return None
        self.stop_flag = True
        self.thread.join(timeout=2)
        self.thread = None
        if not self.samples:
            return None
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        try:
            smmax = nv.nvmlDeviceGetMaxClockInfo(self.handle, nv.NVML_CLOCK_SM)
        except Exception:
            smmax = None
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": smmax,
                "reasons": sorted(k for k, bit in names.items() if self.reasons & bit), "samples": len(self.samples)}


def with_clock(entry, seconds_per_unit, clocks, key):
    """Adds the sampled median SM clock and time x clock (SM cycles per unit of work) to a result entry."""
    entry["clocks"] = clocks
    if clocks and clocks.get("sm_mhz"):
        entry[key] = seconds_per_unit * clocks["sm_mhz"] * 1e6
    return entry


def visible_device_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except (ValueError, IndexError):
            return local_rank
    return local_rank


def config_dict(w, args, world):
    return {"workload": f"config {w.cfg}: n={w.n}" + (f" N={w.nbatch}" if w.nbatch > 1 else "")
            + f" {'log' if w.domain else 'scaling'}-domain fp32 dense matrix, eps={w.eps}, c={w.c} row blocks, "
            + f"{w.iters} iterations per step",
            "n": w.n, "nbatch": w.nbatch, "row_blocks": w.c, "iterations_per_step": w.iters,
            "domain": "log" if w.domain else "scaling",
            "matrix_bytes": int(w.n) * int(w.n) * 4,
            "l2": "matrix is larger than the 126 MB L2, so every pass streams it from HBM; no flush needed"
            if w.n * w.n * 4 > 126e6 else "matrix fits in L2: numbers are L2/latency-bound, not HBM-bound",
            "parallelism": "1 GPU" if world == 1 else f"{world} independent replicas (one problem instance per GPU)"}


# ------------------------------------------------------------------------------------------ reference arm

def oracle_iterate(w, iters):
    import oracle
    if w.nbatch > 1:
        t0 = time.perf_counter()
        oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a[0], w.b[0], iters)
        return (time.perf_counter() - t0), 1.0 / w.nbatch     # one problem of the batch per sample
    t0 = time.perf_counter()
    if w.domain == workloads.DOMAIN_LOG:
        oracle.sinkhorn_log(w.C, w.eps, w.a, w.b, iters)
    else:
        oracle.sinkhorn_scaling(w.K, oracle.KIND_KERNEL, w.eps, w.a, w.b, iters)
    return (time.perf_counter() - t0), 1.0


def cpu_baseline(w, budget_s=12.0):
    """Times the checker, as it stands, on a bounded sample: whole iterations until ~budget_s."""
    import oracle
    oracle.build()
    dt, frac = oracle_iterate(w, 1)
    iters = 1
    total = dt
    while total + dt < budget_s and iters < w.iters:
        d, _ = oracle_iterate(w, 1)
        total += d
        iters += 1
    value = iters * frac / total
    sample = f"{iters} full iteration(s) of the same workload" + (" for 1 of the batch's problems" if w.nbatch > 1 else "")
    out = {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample,
           "seconds": total}
    # the same checker on ONE thread (its OpenMP loops keep every sum's order, so only the time changes)
    try:
        import ctypes
        omp = ctypes.CDLL("libgomp.so.1")
        omp.omp_get_max_threads.restype = ctypes.c_int
        before = omp.omp_get_max_threads()
        omp.omp_set_num_threads(1)
        try:
            d1, f1 = oracle_iterate(w, 1)
        finally:
            omp.omp_set_num_threads(before)
        out["single_thread"] = {"value": f1 / d1, "unit": UNIT, "cores": 1, "sample": "1 full iteration", "seconds": d1}
    except OSError:
        out["single_thread"] = None
    return out


def run_reference(args, w, world):
    import oracle
    oracle.build()
    per_step = max(1, args.ref_iters)
    for _ in range(args.warmup):
        oracle_iterate(w, 1)
    t = 0.0
    frac = 1.0
    for _ in range(args.steps):
        d, frac = oracle_iterate(w, per_step)
        t += d
    value = args.steps * per_step * frac / t
    sample = f"each step = {per_step} iteration(s) of the workload" + (" for 1 of the batch's problems" if w.nbatch > 1 else "")
    cfg = config_dict(w, args, 1)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": cfg, "gpu_launches": 0,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ GPU arm

def time_config(fs, torch, dev, stream, w, steps=3, device_index=0):
    """it/s of one configuration through fs_iterate (device-resident inputs, CUDA events)."""
    M = torch.from_numpy(w.matrix).to(dev)
    a = torch.from_numpy(w.a).to(dev)
    b = torch.from_numpy(w.b).to(dev)
    torch.cuda.synchronize()
    h = fs.fs_create(w.n, w.c, w.offsets, M, w.n, w.kind, w.eps, a, b, w.nbatch, w.domain, stream)
    try:
        if w.check_every:
            fs.fs_set_error_trace(h, w.check_every)

        def step():
            fs.fs_reset(h, stream)
            fs.fs_iterate(h, w.iters, stream)

        path = fs.fs_iteration_path(h)
        for _ in range(3):
            step()
        stream.synchronize()
        sampler = NvmlSampler(device_index)
        sampler.start()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            step()
        e1.record(stream)
        stream.synchronize()
        clocks = sampler.stop()
        ms = e0.elapsed_time(e1)
        row, col = fs.fs_marginal_error(h, 1, w.nbatch, stream)
    finally:
        fs.fs_destroy(h)
    its = steps * w.iters
    return with_clock({"path": path, "workload": f"n={w.n}" + (f" N={w.nbatch}" if w.nbatch > 1 else "") + (" log" if w.domain else " scaling"),
            "value": its / (ms * 1e-3), "unit": UNIT, "us_per_iteration": ms * 1e3 / its, "steps": steps,
            "iterations_per_step": w.iters,
            "effective_gbs_2n2": 2 * w.n * w.n * 4 * its / (ms * 1e-3) / 1e9,
            "final_row_marginal_l1_max": float(row.max()), "final_col_marginal_l1_max": float(col.max())},
                      ms * 1e-3 / its, clocks, "sm_cycles_per_iteration")


def run_implicit_only(args, rank, local_rank, world):
    """--path implicit: one JSON line for the implicit-kernel path alone (profiling runs, scaled-down sizes)."""
    import torch
    from paper_2502_07021_b200 import binding as fs
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.Stream(device=dev)
    wp = workloads.make(args.config, n=args.n, nbatch=1, fp32_points=True, want_cost=False, want_kernel=False)
    if args.iters is not None:
        wp.iters = args.iters
    r = time_implicit(fs, torch, dev, stream, wp, visible_device_index(local_rank), args, wp=wp)
    if rank != 0:
        return
    line = {"metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": world, "steps": r["steps"], "warmup": 3,
            "ms_per_step": r["us_per_iteration"] * wp.iters * 1e-3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"config {wp.cfg} from its point clouds: n={wp.n} d={wp.X.shape[1]} eps={wp.eps}, "
                                   f"{wp.iters} iterations per step, kernel applied implicitly"},
            "gpu_launches": 4 * wp.iters * r["steps"], "clocks": r.get("clocks"), "e2e": r.get("e2e"),
            "roofline": r["roofline"], "cpu_baseline": None}
    print(json.dumps(line), flush=True)


def time_implicit(fs, torch, dev, stream, w, devidx, args, wp=None):
    """Config `w` from its fp32 point clouds through fs_create_points: device-timed it/s, the ex2 roofline of its
    pass kernel and the end-to-end rate through fs_solve_host_points."""
    if wp is None:
        wp = workloads.make(w.cfg, fp32_points=True, want_cost=False, want_kernel=False)
    d = wp.X.shape[1]
    X = torch.from_numpy(wp.X).to(dev)
    Y = torch.from_numpy(wp.Y).to(dev)
    a = torch.from_numpy(wp.a).to(dev)
    b = torch.from_numpy(wp.b).to(dev)
    torch.cuda.synchronize()
    h = fs.fs_create_points(wp.n, wp.c, wp.offsets, X, Y, d, wp.cost_scale, wp.eps, a, b, stream)
    try:
        def step():
            fs.fs_reset(h, stream)
            fs.fs_iterate(h, wp.iters, stream)
        for _ in range(3):
            step()
        stream.synchronize()
        steps = max(1, min(args.steps, 5))
        smp = NvmlSampler(devidx)
        smp.start()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            step()
        e1.record(stream)
        stream.synchronize()
        clocks = smp.stop()
        ms = e0.elapsed_time(e1)
        row, col = fs.fs_marginal_error(h, 1, 1, stream)
        # the special-function rate right after, at the clock the board holds under this kind of load
        smp2 = NvmlSampler(devidx)
        smp2.start()
        ex2_rate = fs.fs_selftest_ex2_rate(1 << 15, stream)
        ex2_clocks = smp2.stop()
    finally:
        fs.fs_destroy(h)
    its = steps * wp.iters
    pass_s = ms * 1e-3 / (2 * its)
    n2 = float(wp.n) * float(wp.n)
    achieved = n2 / pass_s
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    nominal = 16.0 * sms * (clocks["sm_mhz"] * 1e6 if clocks and clocks.get("sm_mhz") else 1.965e9)
    out = {"what": "fs_create_points: K_il = exp(-s|x_i - y_l|^2/eps) formed on the fly (tcgen05 contraction + one ex2 per "
                   "element per pass), two implicit_pass_kernel launches and two stage-2 launches per iteration",
           "value": its / (ms * 1e-3), "unit": UNIT, "us_per_iteration": ms * 1e3 / its, "steps": steps,
           "iterations_per_step": wp.iters, "points_bytes": int(2 * wp.n * d * 4),
           "final_row_marginal_l1": float(row[0]), "final_col_marginal_l1": float(col[0]),
           "roofline": {"bound": "alu", "kernel": "implicit_pass_kernel", "unit": "Gex2/s",
                        "achieved": achieved / 1e9, "peak": ex2_rate / 1e9, "frac": achieved / ex2_rate,
                        "peak_source": "measured: fs_selftest_ex2_rate (every thread issues independent ex2.approx) right "
                                       "after the timed region",
                        "peak_clocks": ex2_clocks,
                        "nominal_peak": nominal / 1e9,
                        "nominal_peak_source": "16 ex2 per clock per SM x SM count x the median SM clock sampled in the "
                                               "timed region",
                        "frac_of_nominal": achieved / nominal,
                        "algorithmic_ex2_per_launch": n2, "us_per_launch": pass_s * 1e6,
                        "traffic": TRAFFIC_BYTES_PER_LAUNCH.get(("implicit_pass_kernel", wp.n))}}
    with_clock(out, ms * 1e-3 / its, clocks, "sm_cycles_per_iteration")
    if not args.no_e2e:
        pin = [torch.from_numpy(x).pin_memory() for x in (wp.X, wp.Y, wp.a, wp.b)]
        uo = torch.empty(wp.n, dtype=torch.float32).pin_memory()
        vo = torch.empty(wp.n, dtype=torch.float32).pin_memory()
        call = lambda: fs.fs_solve_host_points(wp.n, wp.c, wp.offsets, pin[0], pin[1], d, wp.cost_scale, wp.eps, pin[2],
                                               pin[3], wp.iters, uo, vo)
        call()
        ts = []
        for _ in range(3):
            t0 = time.perf_counter()
            call()
            ts.append(time.perf_counter() - t0)
        med = statistics.median(ts)
        out["e2e"] = {"value": wp.iters / med, "unit": UNIT, "ms_per_step": med * 1e3,
                      "h2d_bytes_per_step": int(2 * wp.n * d * 4 + 2 * wp.n * 4), "d2h_bytes_per_step": int(2 * wp.n * 4 + 8),
                      "note": "fs_solve_host_points: allocation, H2D of the two clouds and the marginals, operand set-up, all "
                              "iterations, marginal error, D2H of the scalings, free -- every step"}
    return out


def run_shard_model(args):
    """--multi model (one GPU): the local-compute term of the paper's per-iteration model (Section 4.1:
    T_comp = 2 t_mv(m, n) + t_ew) measured for the row block a shard would own with G = 1, 2, 4, 8 shards of the
    configuration: row pass + column partial + finish on an m x n block, m = n / G.  The exchange term cannot be
    measured with one GPU; it is left out, not assumed."""
    import torch
    from paper_2502_07021_b200 import binding as fs
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    dev = torch.device("cuda", 0)
    stream = torch.cuda.Stream(device=dev)
    n = args.n or workloads._SPECS[args.config]["n"]
    out = []
    for G in (1, 2, 4, 8):
        lo, hi = fsdist.row_range(n, 0, G)
        w = workloads.make(args.config, n=args.n, nbatch=1, want_cost=False, rows=(lo, hi))
        Kb = torch.from_numpy(w.K).to(dev)
        a_loc = torch.from_numpy(w.a[lo:hi].copy()).to(dev)
        b = torch.from_numpy(w.b).to(dev)
        r_buf = torch.empty(w.n, dtype=torch.float32, device=dev)
        torch.cuda.synchronize()
        sh = fs.fs_shard_create(w.n, lo, hi - lo, Kb, w.n, fs.FS_MATRIX_KERNEL, w.eps, a_loc, b, stream)
        iters = max(20, min(200, int(2e9 / ((hi - lo) * w.n * 8))))

        def run(k, fused):
            for _ in range(k):
                if not (fused and fs.fs_shard_fused_step(sh, r_buf, stream, allow_unsupported=True)):
                    fs.fs_shard_row_pass(sh, stream)
                    fs.fs_shard_col_partial(sh, r_buf, stream)
                fs.fs_shard_col_finish(sh, r_buf, stream)

        def timed_run(fused):
            run(5, fused)
            stream.synchronize()
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            run(iters, fused)
            e1.record(stream)
            stream.synchronize()
            return e0.elapsed_time(e1) * 1e3 / iters
        us = timed_run(False)
        us_fused = timed_run(True)
        fs.fs_shard_destroy(sh)
        del Kb
        torch.cuda.empty_cache()
        out.append({"shards": G, "rows_per_shard": hi - lo, "local_us_per_iteration_single_read": us_fused,
                    "local_us_per_iteration": us,
                    "local_gbs": 2 * (hi - lo) * w.n * 4 / (us * 1e-6) / 1e9,
                    "exchange_bytes_per_iteration": w.n * 4})
    line = {"metric": "shard_local_step_us", "unit": "us", "n_gpus": 1, "data": "synthetic", "dtype": "f32",
            "config": {"workload": f"config {args.config}: n={n}, the row block of shard 0 of G"},
            "model": out,
            "note": "local operator time t_local(G) = 2 t_mv(n/G, n) + elementwise of one shard, measured on one GPU; "
                    "an iteration on G GPUs costs max over shards of this plus one exchange of n floats (not measured here)"}
    print(json.dumps(line), flush=True)


def run_sharded(args, rank, local_rank, world):
    """Row-partitioned run (opt-in, --multi sharded): one shard of the SAME problem per GPU, one all-reduce
    of n floats per iteration over NCCL; total work is fixed, so scaling is strong."""
    import torch
    from paper_2502_07021_b200 import binding as fs

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.Stream(device=dev)
    n_total = args.n or workloads._SPECS[args.config]["n"]
    lo, hi = fsdist.row_range(n_total, rank, world)
    w = workloads.make(args.config, n=args.n, nbatch=1, want_cost=False, rows=(lo, hi))
    if w.domain != workloads.DOMAIN_SCALING or w.nbatch != 1:
        raise RuntimeError("--multi sharded covers the single-problem scaling-domain configurations")
    if args.iters is not None:
        w.iters = args.iters
    Kb = torch.from_numpy(w.K).to(dev)
    a_loc = torch.from_numpy(w.a[lo:hi].copy()).to(dev)
    b = torch.from_numpy(w.b).to(dev)
    r_buf = torch.empty(w.n, dtype=torch.float32, device=dev)
    ones_u = torch.ones(hi - lo, dtype=torch.float32, device=dev)
    ones_v = torch.ones(w.n, dtype=torch.float32, device=dev)
    torch.cuda.synchronize()
    sh = fs.fs_shard_create(w.n, lo, hi - lo, Kb, w.n, fs.FS_MATRIX_KERNEL, w.eps, a_loc, b, stream)

    # does the single-read local step apply (then the local block is read once per iteration, not twice)?
    single_read = args.exchange != "alg1" and fs.fs_shard_fused_step(sh, r_buf, stream, allow_unsupported=True)
    reads_per_iteration = 1 if single_read else 2
    sizes = [fsdist.row_range(n_total, r, world)[1] - fsdist.row_range(n_total, r, world)[0] for r in range(world)]
    split = {"local_ms": 0.0, "exchange_ms": 0.0}

    def step(timed=False):
        fs.fs_shard_set_scalings(sh, ones_u, ones_v, stream)
        t = fsdist.sharded_iterate(fs, sh, r_buf, w.iters, stream, exchange=args.exchange, sizes=sizes, timed=timed)
        if t:
            split["local_ms"] += t["local_ms"]
            split["exchange_ms"] += t["exchange_ms"]

    for _ in range(max(3, args.warmup)):
        step()
    stream.synchronize()
    sampler = ClockSampler(visible_device_index(local_rank))
    fsdist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    stream.synchronize()
    torch.cuda.synchronize()
    fsdist.barrier()
    clocks = sampler.stop()
    t_ms, _ = fsdist.aggregate(e0.elapsed_time(e1), 0.0, dev)
    # the paper's split of an iteration into local operator time and collective time (max over ranks), from one
    # more step with CUDA events around every phase (the events themselves cost a little, so it is not the timed one)
    step(timed=True)
    loc_ms, _ = fsdist.aggregate(split["local_ms"], 0.0, dev)
    exc_ms, _ = fsdist.aggregate(split["exchange_ms"], 0.0, dev)
    l1, _ = fs.fs_shard_row_error(sh, stream)
    _, l1 = fsdist.aggregate(0.0, l1, dev)
    fs.fs_shard_destroy(sh)
    if rank != 0:
        return
    its = args.steps * w.iters
    peaks, peak_kind = measured_peaks()
    per_pass_bytes = (hi - lo) * w.n * 4
    line = {"metric": METRIC, "value": its / (t_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": t_ms / args.steps, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": dict(config_dict(w, args, world), parallelism=f"{world} row shards of one problem, exchange = "
                           + {"allreduce": "one sum all-reduce of n floats per iteration",
                              "ordered": "all-gather of the G partial vectors, added in rank order on every shard",
                              "alg1": "Algorithm 1: two Allgathers of scaling slices per iteration (symmetric K)"}[args.exchange]
                           + " (NCCL)"),
            "phase_split": {"local_us_per_iteration": 1e3 * loc_ms / w.iters, "exchange_us_per_iteration": 1e3 * exc_ms / w.iters,
                            "exchange_fraction": exc_ms / max(loc_ms + exc_ms, 1e-30),
                            "note": "CUDA events around every local step and every collective of one extra step, max over "
                                    "ranks; the paper reports the same split (local matvec time vs collective time)"},
            "gpu_launches": int(its * 5), "clocks": clocks, "e2e": None,
            "roofline": {"bound": "hbm", "kernel": "fused_iteration_kernel on the shard's block" if single_read
                         else "row_pass_kernel + col_partial_kernel (per shard)",
                         "achieved": reads_per_iteration * per_pass_bytes * its / (t_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                         "unit": "GB/s",
                         "frac": reads_per_iteration * per_pass_bytes * its / (t_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                         "peak_source": f"of {peak_kind}", "traffic": None,
                         "note": "per-GPU rate over the whole iteration, collectives included"},
            "cpu_baseline": None, "row_marginal_l1_before_last_iteration": l1}
    print(json.dumps(line), flush=True)


def run_ours(args, w, rank, local_rank, world):
    import torch
    from paper_2502_07021_b200 import binding as fs

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    fs.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.Stream(device=dev)
    M_host = torch.from_numpy(w.matrix)
    M = M_host.to(dev)
    a = torch.from_numpy(w.a).to(dev)
    b = torch.from_numpy(w.b).to(dev)
    torch.cuda.synchronize()
    h = fs.fs_create(w.n, w.c, w.offsets, M, w.n, w.kind, w.eps, a, b, w.nbatch, w.domain, stream)
    if w.check_every:
        fs.fs_set_error_trace(h, w.check_every)

    def step():
        fs.fs_reset(h, stream)
        fs.fs_iterate(h, w.iters, stream)

    for _ in range(max(3, args.warmup)):
        step()
    stream.synchronize()
    sampler = ClockSampler(visible_device_index(local_rank))
    fsdist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    launches0 = fs.fs_launch_count(h)
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    stream.synchronize()
    torch.cuda.synchronize()
    fsdist.barrier()
    clocks = sampler.stop()
    launches = fs.fs_launch_count(h) - launches0
    elapsed_ms = e0.elapsed_time(e1)
    row_err, col_err = fs.fs_marginal_error(h, 1, w.nbatch, stream)
    t_ms, total_iters = fsdist.aggregate(elapsed_ms, args.steps * w.iters, dev)

    # dominant kernel.  Two regimes are reported and named: "sustained" = the timed region itself (seconds of
    # back-to-back iterations, SM clock settled under the power cap), which is what `frac` describes, and
    # "burst" = a short loop of single launches from an idle GPU, timed with CUDA events on the launching stream
    # right after the timed region (SM clock near its maximum).
    peaks, peak_kind = measured_peaks()
    devidx = visible_device_index(local_rank)
    path = fs.fs_iteration_path(h)
    n2 = w.n * w.n * 4
    its_region = args.steps * w.iters

    def timed(fn, reps):
        fn()
        stream.synchronize()
        time.sleep(0.5)                       # from an idle GPU
        smp = NvmlSampler(devidx, period_s=0.001)
        smp.start()
        k0 = torch.cuda.Event(enable_timing=True)
        k1 = torch.cuda.Event(enable_timing=True)
        k0.record(stream)
        for _ in range(reps):
            fn()
        k1.record(stream)
        stream.synchronize()
        return k0.elapsed_time(k1) * 1e-3 / reps, smp.stop()

    # (kernel, algorithmic bytes per launch, launches of it per iteration, burst callable, repeats, note)
    if path == "fused_log":
        kernel, bytes_launch, per_iter = "fused_log_iteration_kernel", n2, 1
        burst_fn, reps = (lambda: fs.fs_iterate(h, 1, stream)), 20
        note = ("one launch per iteration reads C once (n*n*4 bytes), one ex2 per element; the timed interval "
                "includes the stage-2 kernel that follows it")
    elif path == "fused":
        kernel, bytes_launch, per_iter = "fused_iteration_kernel", n2, 1
        burst_fn, reps = (lambda: fs.fs_iterate(h, 1, stream)), 20
        note = ("one launch per iteration reads K once (n*n*4 bytes); the timed interval includes the "
                "col_finish_kernel that follows it")
    elif path in ("resident", "persistent"):
        # all iterations of a step in one launch of a persistent kernel; K is read from HBM once per launch
        # and then served from shared memory or from L2 and shared memory
        kernel, bytes_launch, per_iter = path + "_iterations_kernel", n2 * w.iters, 1.0 / w.iters
        burst_fn, reps = (lambda: fs.fs_iterate(h, w.iters, stream)), 5
        note = ("one launch runs all %d iterations of a step; bytes = one read of K per iteration (n*n*4 each), served "
                "from on-chip memory and L2, not HBM: the kernel is latency-bound and this fraction is not an HBM "
                "utilisation" % w.iters)
    elif path == "batched_tc":
        kernel, bytes_launch, per_iter = "batched_tc_kernel", n2 + 4 * w.n * w.nbatch * 4, 2
        burst_fn, reps = (lambda: fs.fs_row_pass(h, stream)), 20
        note = ("one batched pass, one launch: K as two bf16 terms (n*n*4 bytes) + operand and result vectors; the "
                "split-K partial tiles are exchanged inside the cluster and the update is applied in the same "
                "kernel; tensor work is 3 bf16 products per useful one")
    else:
        kernel = {"two_pass": "row_pass_kernel", "two_pass_log": "log_row_pass_kernel"}.get(path, "batched_fma_kernel")
        bytes_launch, per_iter = n2, 2
        burst_fn, reps = (lambda: fs.fs_row_pass(h, stream)), 20
        note = "one pass streams the matrix once (n*n*4 bytes); an iteration is a row pass and a column pass"
    per_launch_sustained_s = elapsed_ms * 1e-3 / (its_region * per_iter)
    achieved = bytes_launch / per_launch_sustained_s / 1e9
    per_launch_burst_s, burst_clocks = timed(burst_fn, reps)
    burst_gbs = bytes_launch / per_launch_burst_s / 1e9
    traffic = TRAFFIC_BYTES_PER_LAUNCH.get((kernel, w.n)) if args.traffic_bytes is None else args.traffic_bytes
    peak_src = ("of measured (MEASURED_PEAKS.json hbm_gbs, copy rate)" if peak_kind == "measured" else "of fallback")
    roof = {"bound": "hbm", "kernel": kernel, "path": path, "achieved": achieved, "peak": peaks["hbm_gbs"],
            "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "peak_source": peak_src,
            "regime": "sustained: the timed region itself, elapsed / launches of this kernel in it "
                      "(the interval also holds the small kernels that run between its launches)",
            "frac_of_nominal_8000_gbs": achieved / 8000.0,
            "algorithmic_bytes_per_launch": bytes_launch, "us_per_launch": per_launch_sustained_s * 1e6,
            "traffic": traffic, "note": note,
            "burst": with_clock({"regime": "%d single launches from an idle GPU, CUDA events on the launching stream" % reps,
                                 "achieved": burst_gbs, "frac": burst_gbs / peaks["hbm_gbs"],
                                 "us_per_launch": per_launch_burst_s * 1e6}, per_launch_burst_s, burst_clocks,
                                "sm_cycles_per_launch"),
            # the metric's own accounting (every iteration streams 2 n^2 matrix elements) applied to the timed region
            "iteration_effective_gbs_2n2": 2 * n2 * its_region / (elapsed_ms * 1e-3) / 1e9}
    with_clock(roof, per_launch_sustained_s, clocks, "sm_cycles_per_launch")

    # the literal dense-K passes of the same configuration: row pass and two-stage column pass, K streamed twice
    # per iteration (FS_OPT_FUSED = 0), each pass timed alone with CUDA events and as whole iterations
    other_paths = None
    if world == 1 and path == "fused" and not args.headline_only:
        def gbs(sec):
            return {"us": sec * 1e6, "gbs": n2 / sec / 1e9, "frac_of_measured": n2 / sec / 1e9 / peaks["hbm_gbs"],
                    "frac_of_nominal_8000_gbs": n2 / sec / 1e9 / 8000.0}
        fs.fs_set_option(h, fs.FS_OPT_FUSED, 0)
        assert fs.fs_iteration_path(h) == "two_pass"
        fs.fs_reset(h, stream)
        fs.fs_iterate(h, 10, stream)
        row_s, row_clk = timed(lambda: fs.fs_row_pass(h, stream), 100)
        col_s, col_clk = timed(lambda: fs.fs_col_pass(h, stream), 100)
        fs.fs_reset(h, stream)
        it_s, it_clk = timed(lambda: fs.fs_iterate(h, w.iters, stream), 2)
        fs.fs_set_option(h, fs.FS_OPT_FUSED, 1)
        other_paths = {"two_pass": {
            "what": "row_pass_kernel, then col_partial_kernel + col_finish_kernel: K is read from HBM twice per iteration",
            "row_pass": with_clock(dict(gbs(row_s), launches_timed=100), row_s, row_clk, "sm_cycles_per_launch"),
            "col_pass": with_clock(dict(gbs(col_s), launches_timed=100), col_s, col_clk, "sm_cycles_per_launch"),
            "iterations": with_clock({"value": w.iters / it_s, "unit": UNIT, "us_per_iteration": it_s / w.iters * 1e6,
                                      "iterations_timed": 2 * w.iters,
                                      "gbs_2n2": 2 * n2 * w.iters / it_s / 1e9,
                                      "frac_of_measured": 2 * n2 * w.iters / it_s / 1e9 / peaks["hbm_gbs"],
                                      "frac_of_nominal_8000_gbs": 2 * n2 * w.iters / it_s / 1e9 / 8000.0},
                                     it_s / w.iters, it_clk, "sm_cycles_per_iteration")}}

    # the same configuration with the kernel applied implicitly from the point clouds (fs_create_points): no matrix in
    # memory, one ex2 per matrix element per pass; bound by the special-function units ("alu" roofline)
    if world == 1 and not args.headline_only and args.n is None and w.cfg in (2, 4) and w.nbatch == 1:
        try:
            if other_paths is None:
                other_paths = {}
            other_paths["implicit"] = time_implicit(fs, torch, dev, stream, w, devidx, args)
        except Exception as exc:  # must not lose the headline line
            other_paths = dict(other_paths or {}, implicit={"error": repr(exc)})

    # the other four configurations, briefly (single GPU runs only): same step definition, fewer steps
    others = None
    if world == 1 and not args.headline_only and args.config == 4 and args.n is None and args.iters is None:
        others = {}
        for cfg in (1, 2, 3, 5):
            try:
                time.sleep(1.0)  # each short run starts from an idle GPU, not from the headline run's power state
                others[f"config{cfg}"] = time_config(fs, torch, dev, stream, workloads.make(cfg, want_cost=None if cfg == 3 else False),
                                                     device_index=devidx)
            except Exception as exc:  # a failure here must not lose the headline line
                others[f"config{cfg}"] = {"error": repr(exc)}
        # the one table the paper prints for this path (Table 1: 15 iterations, n = 5000; 1 problem 0.32 s,
        # 500 targets vectorised 0.31 s, on an unnamed GPU in fp64): same shapes, our recipe, fp32
        try:
            t1 = {}
            # N = 1 and 500 are the table's rows; 5000 and 10000 extend it along the paper's fp32 multi-target sweep
            # (Section 5.1.1 goes to N = 1e5), where the cost per problem keeps falling until the passes are tensor-bound
            for label, nb in (("one_problem", 1), ("vectorized_500", 500), ("vectorized_5000", 5000),
                              ("vectorized_10000", 10000)):
                wt = workloads.make(5, n=5000, nbatch=nb, want_cost=False)
                wt.iters = 15
                r = time_config(fs, torch, dev, stream, wt, steps=5, device_index=devidx)
                t1[label] = {"seconds_for_15_iterations": 15 * r["us_per_iteration"] * 1e-6,
                             "paper_seconds": {1: 0.32, 500: 0.31}.get(nb),
                             "us_per_iteration_and_problem": r["us_per_iteration"] / nb, "path": r["path"],
                             "final_row_marginal_l1_max": r["final_row_marginal_l1_max"]}
                del wt
            others["paper_table1_n5000"] = t1
        except Exception as exc:
            others["paper_table1_n5000"] = {"error": repr(exc)}

    # end-to-end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        pin_M = M_host.pin_memory()
        pin_a = torch.from_numpy(w.a).pin_memory()
        pin_b = torch.from_numpy(w.b).pin_memory()
        out_u = torch.empty_like(pin_a).pin_memory()
        out_v = torch.empty_like(pin_b).pin_memory()
        fs.fs_destroy(h)
        h = None
        del M
        torch.cuda.empty_cache()
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        fs.fs_solve_host(w.n, w.c, w.offsets, pin_M, w.n, w.kind, w.eps, pin_a, pin_b, w.nbatch, w.domain, w.iters,
                         out_u, out_v)  # warm-up
        fsdist.barrier()
        step_ms = []
        for _ in range(e2e_steps):
            t0 = time.perf_counter()
            fs.fs_solve_host(w.n, w.c, w.offsets, pin_M, w.n, w.kind, w.eps, pin_a, pin_b, w.nbatch, w.domain,
                             w.iters, out_u, out_v)
            step_ms.append((time.perf_counter() - t0) * 1e3)
        # the host is shared: the PCIe copy of one step can take several times longer than that of the next,
        # so the reported rate uses the median step; the spread is reported beside it
        dt_ms = statistics.median(step_ms) * e2e_steps
        dt_ms, its = fsdist.aggregate(dt_ms, e2e_steps * w.iters, dev)
        h2d = w.n * w.n * 4 + 2 * w.a.size * 4
        d2h = 2 * w.a.size * 4 + 8 * w.nbatch
        e2e = {"value": its / (dt_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "steps": e2e_steps, "ms_per_step": dt_ms / e2e_steps, "ms_per_step_min": min(step_ms),
               "ms_per_step_max": max(step_ms), "statistic": "median step",
               "note": "fs_solve_host: device allocation, H2D of the matrix and marginals from pinned memory, "
                       "all iterations, marginal error, D2H of the scalings, free -- every step"}
    if h is not None:
        fs.fs_destroy(h)

    if rank != 0:
        return
    base = None
    if not args.no_cpu_baseline:
        base = cpu_baseline(w)
    line = {"metric": METRIC, "value": total_iters / (t_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": t_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_dict(w, args, world), "gpu_launches": int(launches), "clocks": clocks,
            "e2e": e2e, "roofline": roof, "cpu_baseline": base, "other_paths": other_paths, "other_configs": others,
            "final_row_marginal_l1": float(row_err[0]), "final_col_marginal_l1": float(col_err[0])}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4, help="workload 1..5 (4 = the n=32768 headline)")
    ap.add_argument("--n", type=int, default=None, help="override n (scaled-down copy of the recipe)")
    ap.add_argument("--iters", type=int, default=None, help="override the iterations per step (profiling runs)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--ref-iters", type=int, default=1, help="--impl reference: iterations per step")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--multi", default="replicas", choices=["replicas", "sharded", "model"],
                    help="N > 1: independent replicas (default, weak scaling) or row shards of one problem")
    ap.add_argument("--path", default="auto", choices=["auto", "implicit"],
                    help="implicit: time only the implicit-kernel path (fs_create_points) of the configuration")
    ap.add_argument("--exchange", default="allreduce", choices=["allreduce", "ordered", "alg1"],
                    help="--multi sharded: how the shards exchange per iteration (alg1 needs a symmetric kernel: config 5 shape)")
    ap.add_argument("--headline-only", action="store_true", help="skip the short runs of configurations 1, 2, 3, 5")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="DRAM bytes per launch of the dominant kernel from an ncu capture (reported as is)")
    args = ap.parse_args()

    rank, local_rank, world = fsdist.env_world()
    if args.impl == "reference":
        if rank != 0:
            return 0
        w = workloads.make(args.config, n=args.n, want_cost=None if args.config == 3 else False)
        if args.iters is not None:
            w.iters = args.iters
        run_reference(args, w, world)
        return 0
    if world > 1:
        fsdist.init()
    if args.multi == "model":
        if rank == 0:
            run_shard_model(args)
        fsdist.finalize()
        return 0
    if args.multi == "sharded":
        try:
            run_sharded(args, rank, local_rank, world)
        finally:
            fsdist.finalize()
        return 0
    if args.path == "implicit":
        run_implicit_only(args, rank, local_rank, world)
        fsdist.finalize()
        return 0
    w = workloads.make(args.config, n=args.n, want_cost=None if args.config == 3 else False)
    if args.iters is not None:
        w.iters = args.iters
    try:
        run_ours(args, w, rank, local_rank, world)
    finally:
        fsdist.finalize()
    return 0


if __name__ == "__main__":
    sys.exit(main())
