#!/usr/bin/env python
"""Benchmark of the triangle-block SYRK library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c1|c2|c3|c4|c5|lbc]
                    [--impl ours|reference]

A step is one pass of the whole hot path (work-list lookup, TMA streaming, tensor-core update,
epilogue) over one seeded synthetic workload: one SYRK call for configurations 1-4, the 64 calls of
the trailing-update sweep for configuration 5.  Prints ONE JSON line (rank 0).

Without --workload the headline (top-level `value`, `roofline`, `e2e`, `cpu_baseline`) is the largest
configuration, the sweep, and the same line carries a `per_config` object with every configuration
(c1..c5, and the Cholesky driver built on the sweep's call) timed in the same process by the same
protocol.  With --workload only that one is run.  Every record has two legs:

  burst      K steps, each bracketed by CUDA events on the launching stream, a 256 MiB buffer written
             between steps to flush L2 (the sweep's operands exceed L2 by themselves);
  sustained  calls enqueued back to back for at least two seconds, no flush, one event pair around
             all of them, with the SM clock and power sampled meanwhile.

With N > 1 every rank runs an independent replica of the headline on its own GPU (the path has no
exchange step); the value is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2202_10217_b200 import inputs as I

METRIC = "syrk_tflops_N(N+1)M"
UNIT = "TFLOP/s"
DTYPE_NAME = {I.DTYPE_F64: "f64", I.DTYPE_BF16_F32: "bf16_in_f32_acc", I.DTYPE_TF32_F32: "tf32_in_f32_acc",
              I.DTYPE_E4M3_F32: "fp8_e4m3_in_f32_acc", I.DTYPE_F16_F32: "f16_in_f32_acc"}
ELEM_A = {I.DTYPE_F64: 8, I.DTYPE_BF16_F32: 2, I.DTYPE_TF32_F32: 4, I.DTYPE_E4M3_F32: 1, I.DTYPE_F16_F32: 2}
ELEM_C = {I.DTYPE_F64: 8, I.DTYPE_BF16_F32: 4, I.DTYPE_TF32_F32: 4, I.DTYPE_E4M3_F32: 4, I.DTYPE_F16_F32: 4}
SWEEP_NAME = "c5_f64_sweep_32768..512_x512"
SWEEP_N, SWEEP_STEP = 32768, 512
ALL_WORKLOADS = ["c1", "c2", "c3", "c4", "c5", "lbc"]
HEADLINE = "c5"
L2_FLUSH = "256 MiB buffer written between timed steps (L2 flush)"
L2_LARGE = "operands larger than L2 (C view 8.6 GB .. 2 MB, read and written once per call)"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


def sweep_flops() -> int:
    return sum(n * (n + 1) * I.SWEEP_K for n in I.sweep_sizes(SWEEP_N, SWEEP_STEP))


def config_of(key: str, shape: I.Workload | None = None, world: int = 1) -> dict:
    """What a workload is, in words both arms print identically (no measured or device-side facts)."""
    par = {"parallelism": "replicas only" if world > 1 else "1 gpu"}
    if key == "c5":
        return dict({"workload": SWEEP_NAME, "calls_per_step": len(I.sweep_sizes(SWEEP_N, SWEEP_STEP)), "N": SWEEP_N,
                     "M": I.SWEEP_K, "alpha": -1.0, "beta": 1.0, "ldc": SWEEP_N, "l2": L2_LARGE}, **par)
    if key == "lbc":
        return dict({"workload": "lbc_f64_%d" % SWEEP_N, "N": SWEEP_N, "l2": L2_LARGE}, **par)
    wl = shape or I.CONFIGS[key]
    return dict({"workload": wl.name, "N": wl.N, "M": wl.M, "alpha": wl.alpha, "beta": wl.beta, "l2": L2_FLUSH}, **par)


class ClockSampler:
    """Samples SM clock, power and throttle reasons (one `nvidia-smi -lms` process) while a timed
    region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, period_ms: int = 10):
        self.cmd = ["nvidia-smi", "-i", str(index), "--query-gpu=" + self.QUERY,
                    "--format=csv,noheader,nounits", "-lms", str(period_ms)]
        self.proc = None
        self.rows = []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(self.cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            time.sleep(0.4)                       # let the first samples arrive before the load starts
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is None:
            return
        time.sleep(0.05)                          # one more sampling period, so that a short region is seen
        self.proc.terminate()                     # the exact process started above
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        self.rows = [[x.strip() for x in line.split(",")] for line in out.splitlines() if line.strip()]

    def summary(self):
        sm, mx, power, reasons = [], 0.0, [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                c, m, w = float(r[0]), float(r[1]), float(r[2])
            except Exception:
                continue
            sm.append(c)
            mx = max(mx, m)
            power.append(w)
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        # "under load": samples drawing more than half of the way from the lowest to the largest power seen
        # (the sampler also sees the idle time before and after the region)
        top, low = (max(power), min(power)) if power else (0.0, 0.0)
        load = [(c, w) for c, w in zip(sm, power) if w >= low + 0.5 * (top - low)]
        return {"sm_mhz": float(np.median([c for c, _ in load])) if load else None, "sm_max_mhz": mx or None,
                "reasons": sorted(reasons), "samples": len(sm), "samples_under_load": len(load),
                "power_w_median": float(np.median([w for _, w in load])) if load else None,
                "power_w_max": top or None}


# ---- the CPU reference as a timed baseline -----------------------------------------------------------------

def oracle_sample(key: str, shape: I.Workload | None = None, target_macs: float = 6.0e9):
    """The bounded sample of a workload the CPU reference is timed on: (A rows, C_in or None, alpha, beta,
    dtype, flops, words).  Single calls: the first R rows of the lower triangle, R chosen for about
    `target_macs` multiply-adds.  The sweep (and the factorisation built on it): its call n = 4096
    (alpha = -1, beta = 1, inner dimension 512), first R rows."""
    if key in ("c5", "lbc"):
        n = 4096
        wl = I.Workload("c5_call_n4096", n, I.SWEEP_K, I.DTYPE_F64, -1.0, 1.0, I.SWEEP_SEED, "normal", std=I.SWEEP_K ** -0.5)
        A = I.sweep_panel(n, SWEEP_N)
    else:
        wl = shape or I.CONFIGS[key]
        A = None
    R = int(min(wl.N, max(64, math.sqrt(2.0 * target_macs / max(wl.M, 1)))))
    if A is None:
        A = I.Workload(wl.name, R, wl.M, wl.dtype, wl.alpha, wl.beta, wl.seed, wl.dist, wl.std).make_A() \
            if R < wl.N and wl.N * wl.M > (1 << 28) else wl.make_A()
    sub = np.ascontiguousarray(A[:R])
    Cin = I.random_c(R, 17, wl.dtype) if wl.beta != 0.0 else None
    words = "first %d of %d rows of the lower triangle of %s" % (R, wl.N, wl.name)
    return sub, Cin, wl.alpha, wl.beta, wl.dtype, R * (R + 1) * wl.M, words


def time_oracle(sample, min_seconds: float, max_reps: int = 1000):
    """Runs the reference, as it stands, on `sample` until `min_seconds` have passed (at least once)."""
    from oracle import syrk as O
    sub, Cin, alpha, beta, dtype, flops, words = sample
    reps, t0 = 0, time.perf_counter()
    while True:
        O.syrk_lower(sub, Cin, alpha, beta, dtype)
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds or reps >= max_reps:
            break
    return {"value": reps * flops / dt * 1e-12, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
            "sample": "%s, %d time%s (%.3g flops, %.1f s)" % (words, reps, "" if reps == 1 else "s", reps * flops, dt)}


def run_reference(args, key: str, shape, rank: int):
    """--impl reference: the CPU oracle on host cores, rank 0 only; a step is one pass over the sample."""
    if rank != 0:
        return
    from oracle import syrk as O
    sample = oracle_sample(key, shape)
    sub, Cin, alpha, beta, dtype, flops, words = sample
    for _ in range(args.warmup):
        O.syrk_lower(sub, Cin, alpha, beta, dtype)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        O.syrk_lower(sub, Cin, alpha, beta, dtype)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = flops / dt * 1e-12
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": DTYPE_NAME[dtype], "data": "synthetic",
        "config": config_of(key, shape, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
                         "sample": "%s, once per step (%.3g flops)" % (words, flops)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ---- measured DRAM traffic -------------------------------------------------------------------------------

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures
# summarised under profiles/.  Valid only for the kernel source it was taken on: keyed by its SHA-256.
NCU_TRAFFIC = {
    # workload: (bytes per launch, kernel source file, sha256 of that file at capture time, square-schedule bytes or None)
    "c2_f64_4096x4096": (822_442_496, "syrk_f64.cu", "b7220ccfcf5f6537b1b742a9ff9c2f3bd738d45ad98f75423b3ab2b781f45979", 809_468_160),
    "c3_bf16_16384x4096": (1_898_579_968, "syrk_bf16.cu", "527f2140d892d840fb605c824d4e19c4706e87355a46c48bb934fb71b3a9a97b", 3_150_107_648),
    "c4_bf16_2048x262144": (1_308_831_488, "syrk_bf16_pair.cu", "1f007b0ed5552de540c0cf0f25685f828321404cc4f842d0dbfcbbdcc303fc01", 2_332_056_832),
    "c5_call_n16384": (2_697_048_064, "syrk_f64.cu", "b7220ccfcf5f6537b1b742a9ff9c2f3bd738d45ad98f75423b3ab2b781f45979", 2_507_285_760),
}


def source_hash(name: str) -> str:
    import hashlib
    with open(os.path.join(ROOT, "paper_2202_10217_b200", "csrc", name), "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()


def traffic_of(workload_name: str):
    """(bytes per launch or None, the same for the square schedule or None)."""
    rec = NCU_TRAFFIC.get(workload_name)
    if rec is None or source_hash(rec[1]) != rec[2]:
        return None, None
    return rec[0], rec[3]


# ---- timing ------------------------------------------------------------------------------------------------

class Timer:
    """The two legs of a record.  `call` enqueues one step on torch's current stream."""

    def __init__(self, torch, local_rank: int, dist):
        self.torch, self.local_rank, self.dist = torch, local_rank, dist
        self.flush_buf = None

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def max_over_ranks(self, value: float) -> float:
        """Slowest rank's time (every rank gets it); the identity without a process group."""
        return max_over_ranks(value, self.dist, "cuda")

    def flush(self):
        if self.flush_buf is None:
            self.flush_buf = self.torch.empty(256 << 20, dtype=self.torch.uint8, device="cuda")     # > L2 (126 MB)
        self.flush_buf.zero_()

    def burst(self, call, steps: int, warmup: int, flush: bool):
        torch = self.torch
        for _ in range(warmup):
            call()
        torch.cuda.synchronize()
        ev0 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        ev1 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        self.barrier()
        with ClockSampler(self.local_rank) as clocks:
            for i in range(steps):
                if flush:
                    self.flush()                           # evict A and C from L2 (not timed)
                ev0[i].record()
                call()
                ev1[i].record()
            self.barrier()
        times = [a.elapsed_time(b) for a, b in zip(ev0, ev1)]
        total_ms = self.max_over_ranks(float(sum(times)))
        return total_ms / steps, float(np.mean(times)), clocks.summary()

    def sustained(self, call, est_ms: float, seconds: float = 2.2, max_calls: int = 60000):
        torch = self.torch
        n = int(max(3, min(max_calls, math.ceil(seconds * 1e3 / max(est_ms, 1e-3)))))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        with ClockSampler(self.local_rank) as clocks:
            e0.record()
            for _ in range(n):
                call()
            e1.record()
            self.barrier()
        ms = self.max_over_ranks(e0.elapsed_time(e1)) / n
        return ms, n, clocks.summary()


def max_over_ranks(value: float, dist, device) -> float:
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(flops_per_replica: float, world: int, seconds: float) -> float:
    """Replicas only: every rank does the same work, the job lasts as long as its slowest rank."""
    return world * flops_per_replica / seconds * 1e-12


def peak_for(B, dtype: int, cache: dict):
    """(burst peak, sustained peak or None, where they come from) for the tensor-core type of `dtype`."""
    peaks, kind = measured_peaks()
    if dtype == I.DTYPE_F64:
        if "f64" not in cache:
            cache["f64"] = B.syrk_probe_f64_mma_peak(20000)
        note = ("FP64 tensor-core (DMMA) rate measured in this run by the library's register-only mma.sync "
                "probe; MEASURED_PEAKS.json has no FP64 figure (bf16 %s %.1f x 40/2250 = %.1f)"
                % (kind, peaks["bf16_tflops"], peaks["bf16_tflops"] * 40.0 / 2250.0))
        return cache["f64"], cache["f64"], note
    ratio, words = 1.0, ""
    if dtype == I.DTYPE_E4M3_F32:
        ratio, words = 2.0, " x nominal fp8/bf16 ratio 2"
    elif dtype == I.DTYPE_TF32_F32:
        ratio, words = 1.1 / 2.25, " x nominal tf32/bf16 ratio 1.1/2.25"
    sus = peaks.get("bf16_tflops_sustained")
    return (float(peaks["bf16_tflops"]) * ratio, float(sus) * ratio if sus else None,
            "cuBLAS bf16 burst / sustained, MEASURED_PEAKS.json (%s)%s" % (kind, words))


def roofline_record(flops_per_launch: float, kernel_ms: float, sustained_ms, peak, peak_sus, note, traffic, traffic_sq, extra=None):
    achieved = flops_per_launch / (kernel_ms * 1e-3) * 1e-12
    r = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": UNIT, "frac": achieved / peak,
         "traffic": traffic, "peak_source": note, "algorithmic_flops_per_launch": flops_per_launch}
    if traffic_sq is not None:
        r["traffic_square"] = traffic_sq
    if sustained_ms:
        r["achieved_sustained"] = flops_per_launch / (sustained_ms * 1e-3) * 1e-12
        if peak_sus:
            r["peak_sustained"] = peak_sus
            r["frac_sustained"] = r["achieved_sustained"] / peak_sus
    if extra:
        r.update(extra)
    return r


# ---- one record per workload ---------------------------------------------------------------------------------

def to_device(torch, A_host, dtype):
    """(pinned host tensor, device tensor) of an operand in its storage type."""
    if dtype in (I.DTYPE_BF16_F32, I.DTYPE_F16_F32):
        pinned = torch.from_numpy(A_host.view(np.int16)).pin_memory()
        return pinned, pinned.cuda().view(torch.float16 if dtype == I.DTYPE_F16_F32 else torch.bfloat16)
    pinned = torch.from_numpy(A_host).pin_memory()
    return pinned, pinned.cuda()


def record_single(key, shape, args, T: Timer, B, torch, world, want_e2e: bool, peak_cache: dict):
    """Configurations 1-4 (or a --shape): one syrk_lower call per step."""
    wl = shape or I.CONFIGS[key]
    N, M, dtype = wl.N, wl.M, wl.dtype
    A_host = wl.make_A()
    A_pinned, dA = to_device(torch, A_host, dtype)
    cdt = torch.float64 if dtype == I.DTYPE_F64 else torch.float32
    dC = torch.zeros((N, N), dtype=cdt, device="cuda")
    B.syrk_plan_prepare_stream(N, M, dtype)
    stats = B.syrk_get_schedule_stats(N, M, dtype)
    ran = stats["effective_schedule"]
    call = lambda: B.syrk_lower(N, M, dA, M, dC, N, wl.alpha, wl.beta, dtype)
    ms_step, kernel_ms, clocks = T.burst(call, args.steps, max(args.warmup, 3), flush=True)
    assert B.syrk_last_status() == 0
    sus_ms, sus_calls, sus_clocks = T.sustained(call, kernel_ms)
    assert B.syrk_last_status() == 0
    peak, peak_sus, note = peak_for(B, dtype, peak_cache)
    traffic, traffic_sq = traffic_of(wl.name)
    rec = {
        "workload": wl.name, "metric": METRIC, "unit": UNIT, "value": whole_job_tflops(wl.flops, world, ms_step * 1e-3),
        "ms_per_step": ms_step, "steps": args.steps, "dtype": DTYPE_NAME[dtype], "config": config_of(key, shape),
        "schedule": {"ran": B.SCHEDULE_NAME[ran], "k_slices": stats["split_k"], "tile": stats["tile"], "k": stats["k"],
                     "tbs_items": stats["items"],
                     "tbs_tri_items": stats["tri_items"], "tbs_model_a_bytes": stats["a_loads"] * ELEM_A[dtype],
                     "s_acc": stats["s_acc"], "s_total": stats["s_total"]},
        "clocks": clocks,
        "value_sustained": whole_job_tflops(wl.flops, world, sus_ms * 1e-3),
        "sustained": {"ms_per_step": sus_ms, "calls": sus_calls, "l2": "no flush, calls back to back", "clocks": sus_clocks},
        "gpu_launches": args.steps * stats["launches"],
        "roofline": roofline_record(wl.flops, kernel_ms, sus_ms, peak, peak_sus, note, traffic, traffic_sq),
    }
    if want_e2e:
        rec.update(e2e_single(wl, A_pinned, B, torch, T, world))
    del dA, dC
    torch.cuda.empty_cache()
    return rec, A_host


def e2e_single(wl, A_pinned, B, torch, T: Timer, world):
    """The same metric through syrk_lower_host from page-locked host buffers: the upload of A and the
    download of the lower triangle of C are inside the timed region.  Two figures: the pipeline the call
    takes by itself, and the column-block pipeline, the one that runs the device call's schedule."""
    N, M, dtype = wl.N, wl.M, wl.dtype
    C_pinned = torch.zeros((N, N), dtype=torch.float64 if dtype == I.DTYPE_F64 else torch.float32).pin_memory()
    out = {}
    for name, mode in (("e2e", B.HOST_AUTO), ("e2e_tbs", B.HOST_COLUMN_BLOCKS)):
        try:
            B.syrk_set_host_pipeline(mode)
            path = B.syrk_host_pipeline_for(N, M, True)
            if name == "e2e_tbs" and out["e2e"]["pipeline"].startswith("column"):
                out[name] = dict(out["e2e"])                   # the call took this pipeline by itself
                continue
            B.syrk_lower_host(N, M, A_pinned, M, C_pinned, N, wl.alpha, wl.beta, dtype)      # warm-up (allocates staging)
            T.barrier()
            steps = 3
            t0 = time.perf_counter()
            for _ in range(steps):
                B.syrk_lower_host(N, M, A_pinned, M, C_pinned, N, wl.alpha, wl.beta, dtype)
            sec = T.max_over_ranks((time.perf_counter() - t0) / steps)
        finally:
            B.syrk_set_host_pipeline(B.HOST_AUTO)
        if path == B.HOST_ROW_BANDS:
            words, sched = "row bands (upload, compute and download overlap band by band)", "square"
        else:
            words = "column blocks (upload overlaps compute; C downloaded after the last block)"
            sched = B.SCHEDULE_NAME[B.syrk_effective_schedule(N, M, dtype)]
        out[name] = {"value": whole_job_tflops(wl.flops, world, sec), "unit": UNIT, "ms_per_step": sec * 1e3,
                     "h2d_bytes_per_step": N * M * ELEM_A[dtype] + (N * N * ELEM_C[dtype] if wl.beta != 0 else 0),
                     "d2h_bytes_per_step": N * (N + 1) // 2 * ELEM_C[dtype], "api": "syrk_lower_host",
                     "pipeline": words, "schedule": sched}
    return out


def record_sweep(args, T: Timer, B, torch, world, want_e2e: bool, peak_cache: dict):
    """Configuration 5: C_n <- C_n - A_n A_n^T on the trailing n x n view of one 32768^2 FP64 matrix,
    n = 32768, 32256, ..., 512 (64 calls, inner dimension 512, ldc = 32768).  One step = the whole sweep."""
    n_max, M = SWEEP_N, I.SWEEP_K
    sizes = I.sweep_sizes(n_max, SWEEP_STEP)
    flops = sweep_flops()
    # A_n = the trailing n rows of one seeded n_max x 512 panel (same shapes, pitches and value
    # distribution as a fresh panel per step); C = n_max * I + G G^T / 512 prepared with torch.
    A_pinned = torch.from_numpy(I.sweep_panel(n_max, n_max)).pin_memory()
    dA = A_pinned.cuda()
    G = torch.from_numpy(I.sweep_factor(n_max)).cuda()
    C = torch.matmul(G, G.T) / float(M)
    C.diagonal().add_(float(n_max))
    del G
    for n in sizes:
        B.syrk_plan_prepare_stream(n, M, I.DTYPE_F64)

    def sweep(src=dA):
        for n in sizes:
            off = n_max - n
            B.syrk_lower(n, M, src.data_ptr() + off * M * 8, M, C.data_ptr() + (off * n_max + off) * 8, n_max,
                         -1.0, 1.0, I.DTYPE_F64)

    ms_step, kernel_ms, clocks = T.burst(sweep, args.steps, max(args.warmup, 3), flush=False)
    assert B.syrk_last_status() == 0
    sus_ms, sus_calls, sus_clocks = T.sustained(sweep, kernel_ms)
    assert B.syrk_last_status() == 0
    peak, peak_sus, note = peak_for(B, I.DTYPE_F64, peak_cache)
    stats = B.syrk_get_schedule_stats(n_max, M, I.DTYPE_F64)
    # DRAM traffic: one launch (n = 16384) was captured; the average launch of the sweep does flops / 64,
    # and both the old and new C bytes and the re-read A bytes of a launch grow like n^2, as its flops do.
    traffic, _ = traffic_of("c5_call_n16384")
    if traffic is not None:
        traffic = int(traffic * (flops / len(sizes)) / (16384 * 16385 * M))
    rec = {
        "workload": SWEEP_NAME, "metric": METRIC, "unit": UNIT, "value": whole_job_tflops(flops, world, ms_step * 1e-3),
        "ms_per_step": ms_step, "steps": args.steps, "dtype": "f64", "config": config_of("c5"),
        "schedule": {"ran": "tbs", "tile": stats["tile"], "k": stats["k"], "s_acc": stats["s_acc"], "s_total": stats["s_total"]},
        "clocks": clocks,
        "value_sustained": whole_job_tflops(flops, world, sus_ms * 1e-3),
        "sustained": {"ms_per_step": sus_ms, "calls": sus_calls * len(sizes), "l2": "no flush, sweeps back to back",
                      "clocks": sus_clocks},
        # one kernel per call, plus the reduction kernel of the few smallest calls that run in K-slices
        "gpu_launches": args.steps * sum(B.syrk_get_schedule_stats(n, M, I.DTYPE_F64)["launches"] for n in sizes),
        "roofline": roofline_record(flops / len(sizes), kernel_ms / len(sizes), sus_ms / len(sizes), peak, peak_sus, note,
                                    traffic, None, {"launches_per_step": len(sizes)}),
    }
    if want_e2e:
        # end to end: the matrix stays on the device across the 64 calls (as in the factorisation the sweep
        # imitates); every call's panel is copied from page-locked host memory before it, and the diagonal of
        # the result is read back
        bufs = [torch.empty_like(dA), torch.empty_like(dA)]
        diag_host = torch.empty(n_max, dtype=torch.float64).pin_memory()
        copy_stream = torch.cuda.Stream()
        landed = [torch.cuda.Event(), torch.cuda.Event()]
        consumed = [torch.cuda.Event(), torch.cuda.Event()]

        def e2e_sweep():
            # two panel buffers: the panel of call i + 1 travels on a copy stream while call i computes
            cur = torch.cuda.current_stream()
            for ev in consumed:
                ev.record(cur)
            for i, n in enumerate(sizes):
                off, b = n_max - n, i % 2
                with torch.cuda.stream(copy_stream):
                    copy_stream.wait_event(consumed[b])          # the call that last read this buffer has finished
                    bufs[b][off:].copy_(A_pinned[off:], non_blocking=True)
                    landed[b].record(copy_stream)
                cur.wait_event(landed[b])
                B.syrk_lower(n, M, bufs[b].data_ptr() + off * M * 8, M, C.data_ptr() + (off * n_max + off) * 8, n_max,
                             -1.0, 1.0, I.DTYPE_F64)
                consumed[b].record(cur)
            diag_host.copy_(C.diagonal(), non_blocking=True)
            torch.cuda.synchronize()

        e2e_sweep()
        T.barrier()
        steps = 3
        t0 = time.perf_counter()
        for _ in range(steps):
            e2e_sweep()
        sec = T.max_over_ranks((time.perf_counter() - t0) / steps)
        rec["e2e"] = {"value": whole_job_tflops(flops, world, sec), "unit": UNIT, "ms_per_step": sec * 1e3,
                      "h2d_bytes_per_step": sum(n * M * 8 for n in sizes), "d2h_bytes_per_step": n_max * 8,
                      "api": "syrk_lower", "schedule": "tbs",
                      "pipeline": "C resident on the device across the 64 calls; each call's panel uploaded from "
                                  "page-locked host memory on a copy stream while the previous call computes (two "
                                  "buffers); the diagonal read back"}
    del dA, C
    torch.cuda.empty_cache()
    return rec


def record_cholesky(args, T: Timer, B, torch, peak_cache: dict, n: int, block: int):
    """Large Block Cholesky of a seeded n^2 FP64 matrix (n*I + G G^T / 512); a step is one factorisation
    (the matrix is restored from a device copy between steps, outside the timing)."""
    M = I.SWEEP_K
    G = torch.from_numpy(I.sweep_factor(n)).cuda()
    A0 = torch.matmul(G, G.T) / float(M)
    A0.diagonal().add_(float(n))
    del G
    A = A0.clone()
    flops = n ** 3 / 3.0
    steps = max(1, min(args.steps, 3))
    times = []
    with ClockSampler(T.local_rank) as clocks:
        for i in range(steps + 1):                       # first pass is the warm-up (allocates work lists)
            A.copy_(A0)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.cholesky_lower(n, A, n, block)
            e1.record()
            torch.cuda.synchronize()
            assert B.syrk_last_status() == 0 and B.cholesky_last_info() == 0
            if i > 0:
                times.append(e0.elapsed_time(e1))
    ms = float(np.mean(times))
    # residual on sampled entries: (L L^T)_ij against A0_ij
    idx = torch.randint(0, n, (4096,), device="cuda")
    jdx = (torch.rand(4096, device="cuda") * (idx + 1)).long()
    L = torch.tril(A)
    rec_ij = (L[idx] * L[jdx]).sum(dim=1)
    err = float((rec_ij - A0[idx, jdx]).abs().max() / A0.abs().max())
    peak, _, note = peak_for(B, I.DTYPE_F64, peak_cache)
    out = {"workload": "lbc_f64_%d" % n, "metric": "cholesky_tflops_N^3/3", "unit": UNIT, "value": flops / (ms * 1e-3) * 1e-12,
           "ms_per_step": ms, "steps": steps, "dtype": "f64", "config": dict(config_of("lbc"), N=n, block=block or "library default"),
           "clocks": clocks.summary(), "sampled_relative_residual": err,
           "roofline": {"bound": "tensor", "achieved": flops / (ms * 1e-3) * 1e-12, "peak": peak, "unit": UNIT,
                        "frac": flops / (ms * 1e-3) * 1e-12 / peak, "traffic": None, "peak_source": note}}
    del A, A0, L
    torch.cuda.empty_cache()
    return out


def run_ours(args, keys, headline, shape, rank: int, world: int, local_rank: int):
    import torch
    from paper_2202_10217_b200 import binding as B

    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        keys = [headline]                                    # replicas time the headline only
    T = Timer(torch, local_rank, dist)
    peak_cache: dict = {}
    records = {}
    for key in keys:
        if key == "c5":
            records[key] = record_sweep(args, T, B, torch, world, want_e2e=True, peak_cache=peak_cache)
        elif key == "lbc":
            records[key] = record_cholesky(args, T, B, torch, peak_cache, args.lbc_n, args.block)
        else:
            records[key], _ = record_single(key, shape if key == headline else None, args, T, B, torch, world,
                                            want_e2e=True, peak_cache=peak_cache)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    head = records[headline]
    line = {
        "metric": head["metric"], "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": head["steps"],
        "warmup": max(args.warmup, 3), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": head["dtype"], "data": "synthetic",
        "config": config_of(headline, shape, world),
        "schedule": head.get("schedule"),
        "clocks": head["clocks"],
        "value_sustained": head.get("value_sustained"), "sustained": head.get("sustained"),
        "e2e": head.get("e2e"), "gpu_launches": head.get("gpu_launches"),
        "roofline": head["roofline"],
    }
    if "e2e_tbs" in head:
        line["e2e_tbs"] = head["e2e_tbs"]
    if world == 1:
        line["cpu_baseline"] = time_oracle(oracle_sample(headline, shape), min_seconds=12.0)
        if len(records) > 1:
            line["per_config"] = records
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ---- K-sharded update over the ranks (strong scaling; the default N > 1 run is replicas) ----------------------------

def run_kshard(args, key, shape, rank: int, world: int, local_rank: int):
    """--kshard: one update of the workload with the inner dimension split over the ranks (every rank a
    block of columns of A, one reduce-scatter of the packed lower triangles); a step is the whole
    exchange-and-update, the value is the whole problem's flops over the slowest rank's time."""
    import torch
    import torch.distributed as dist
    from paper_2202_10217_b200 import binding as B
    from paper_2202_10217_b200 import distributed as D

    torch.cuda.set_device(local_rank)
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29555")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", local_rank))
    T = Timer(torch, local_rank, dist if world > 1 else None)
    wl = shape or I.CONFIGS[key]
    N, M, dtype = wl.N, wl.M, wl.dtype
    k0, k1 = D.column_block(M, world, rank, dtype)
    A_host = wl.make_A()                                      # every rank draws the same seeded matrix and keeps its block
    _, dA = to_device(torch, np.ascontiguousarray(A_host[:, k0:k1]), dtype)
    del A_host
    cdt = torch.float64 if dtype == I.DTYPE_F64 else torch.float32
    dC = torch.zeros((N, N), dtype=cdt, device="cuda")
    chunk = D.packed_share(N, world, rank)[2]
    ws = (torch.empty((N, N), dtype=cdt, device="cuda"), torch.zeros(world * chunk, dtype=cdt, device="cuda"))
    call = lambda: D.syrk_lower_ksharded(N, k1 - k0, dA, max(k1 - k0, 1), dC, N, wl.alpha, wl.beta, dtype, workspace=ws)
    ms_step, _, clocks = T.burst(call, args.steps, max(args.warmup, 3), flush=True)
    assert B.syrk_last_status() == 0
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": wl.flops / (ms_step * 1e-3) * 1e-12, "unit": UNIT, "n_gpus": world,
                          "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
                          "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": DTYPE_NAME[dtype],
                          "data": "synthetic", "config": dict(config_of(key, shape), parallelism="k-sharded x%d" % world),
                          "clocks": clocks, "exchange": {"collective": "reduce_scatter of the packed lower triangle",
                                                         "bytes_per_rank": world * chunk * (8 if dtype == I.DTYPE_F64 else 4)}}))
    dist.destroy_process_group()


# ---- short device-timed runs for the profiler ------------------------------------------------------------------------

def run_kernel_only(args, key, shape, rank: int, world: int, local_rank: int):
    """--kernel-only: device-timed steps of one workload, nothing else (for ncu and for sweeps of sizes)."""
    import torch
    from paper_2202_10217_b200 import binding as B

    torch.cuda.set_device(local_rank)
    T = Timer(torch, local_rank, None)
    if args.schedule != "default":
        B.syrk_set_schedule({"tbs": B.SCHEDULE_TBS, "square": B.SCHEDULE_SQUARE, "pair": B.SCHEDULE_PAIR_SQUARE,
                             "auto": B.SCHEDULE_AUTO}[args.schedule])
    if key == "c5" and shape is None:
        n_max, M = SWEEP_N, I.SWEEP_K
        sizes = I.sweep_sizes(n_max, SWEEP_STEP)
        dA = torch.from_numpy(I.sweep_panel(n_max, n_max)).cuda()
        C = torch.zeros((n_max, n_max), dtype=torch.float64, device="cuda")
        C.diagonal().add_(float(n_max))

        def call():
            for n in sizes:
                off = n_max - n
                B.syrk_lower(n, M, dA.data_ptr() + off * M * 8, M, C.data_ptr() + (off * n_max + off) * 8, n_max,
                             -1.0, 1.0, I.DTYPE_F64)
        flops, name, flush = sweep_flops(), SWEEP_NAME, False
    else:
        wl = shape or I.CONFIGS[key]
        N, M, dtype = wl.N, wl.M, wl.dtype
        if args.batch > 0:
            return run_batched(args, wl)
        if args.syr2k:
            return run_syr2k(args, wl)
        if args.herk:
            return run_herk(args, wl)
        _, dA = to_device(torch, wl.make_A(), dtype)
        dC = torch.zeros((N, N), dtype=torch.float64 if dtype == I.DTYPE_F64 else torch.float32, device="cuda")
        if args.gram:                                          # same operand stored M x N: C = A^T A
            dA = dA.t().contiguous()
            call = lambda: B.syrk_lower_tn(N, M, dA, N, dC, N, wl.alpha, wl.beta, dtype)
        else:
            call = lambda: B.syrk_lower(N, M, dA, M, dC, N, wl.alpha, wl.beta, dtype)
        flops, name, flush = wl.flops, wl.name, True
    ms_step, _, _ = T.burst(call, args.steps, args.warmup, flush=flush)
    assert B.syrk_last_status() == 0
    out = {"metric": METRIC, "value": whole_job_tflops(flops, 1, ms_step * 1e-3), "unit": UNIT, "n_gpus": 1,
           "steps": args.steps, "ms_per_step": ms_step, "kernel_only": True,
           "config": {"workload": name, "schedule": args.schedule,
                      "operand": "M x N (Gram form)" if args.gram else "N x M"}}
    if args.sustained:
        sus_ms, n, clocks = T.sustained(call, ms_step)
        out["value_sustained"] = whole_job_tflops(flops, 1, sus_ms * 1e-3)
        out["sustained"] = {"ms_per_step": sus_ms, "calls": n, "clocks": clocks}
    print(json.dumps(out))


def run_batched(args, wl):
    """--kernel-only --batch B: B seeded problems of the workload's shape through syrk_lower_batched,
    beside the same B problems enqueued one by one with syrk_lower (device-timed, L2 flushed)."""
    import torch
    from paper_2202_10217_b200 import binding as B

    N, M, dtype, nb = wl.N, wl.M, wl.dtype, args.batch
    tall = I.Workload(wl.name, nb * N, M, dtype, wl.alpha, wl.beta, wl.seed, wl.dist, wl.std).make_A()
    dA = torch.from_numpy(tall.view(np.int16) if tall.dtype == np.uint16 else tall).cuda()   # nb matrices, stride N * M
    dC = torch.zeros((nb, N, N), dtype=torch.float64 if dtype == I.DTYPE_F64 else torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    ea, ec = dA.element_size(), dC.element_size()

    def batched():
        B.syrk_lower_batched(nb, N, M, dA, M, N * M, dC, N, N * N, wl.alpha, wl.beta, dtype)

    def one_by_one():
        for b in range(nb):
            B.syrk_lower(N, M, dA.data_ptr() + b * N * M * ea, M, dC.data_ptr() + b * N * N * ec, N,
                         wl.alpha, wl.beta, dtype)

    out = {}
    for name, call in (("batched", batched), ("one_by_one", one_by_one)):
        for _ in range(max(args.warmup, 1)):
            call()
        torch.cuda.synchronize()
        assert B.syrk_last_status() == 0
        times = []
        for _ in range(args.steps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            call()
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        out[name] = float(np.mean(times))
    assert B.syrk_last_status() == 0
    print(json.dumps({"metric": METRIC, "value": nb * wl.flops / (out["batched"] * 1e-3) * 1e-12, "unit": UNIT,
                      "n_gpus": 1, "steps": args.steps, "ms_per_step": out["batched"], "kernel_only": True,
                      "one_by_one_ms": out["one_by_one"],
                      "one_by_one_value": nb * wl.flops / (out["one_by_one"] * 1e-3) * 1e-12,
                      "config": {"workload": wl.name, "N": N, "M": M, "batch": nb}}))


def run_syr2k(args, wl):
    """--kernel-only --syr2k: the rank-2k update alpha (A B^T + B A^T) + beta C of the workload's shape and type
    (B drawn like A from the next seed); 2 N (N+1) M flops."""
    import torch
    from paper_2202_10217_b200 import binding as B

    N, M, dtype = wl.N, wl.M, wl.dtype
    _, dA = to_device(torch, wl.make_A(), dtype)
    _, dB = to_device(torch, I.Workload(wl.name, N, M, dtype, wl.alpha, wl.beta, wl.seed + 1, wl.dist, wl.std).make_A(), dtype)
    dC = torch.zeros((N, N), dtype=torch.float64 if dtype == I.DTYPE_F64 else torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    call = lambda: B.syr2k_lower_ex(N, M, dA, M, dB, M, dC, N, wl.alpha, wl.beta, dtype)
    for _ in range(max(args.warmup, 1)):
        call()
    torch.cuda.synchronize()
    times = []
    for _ in range(args.steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        call()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    assert B.syrk_last_status() == 0
    ms = float(np.mean(times))
    print(json.dumps({"metric": "syr2k_tflops_2N(N+1)M", "value": 2 * wl.flops / (ms * 1e-3) * 1e-12, "unit": UNIT,
                      "n_gpus": 1, "steps": args.steps, "ms_per_step": ms, "kernel_only": True,
                      "config": {"workload": wl.name, "N": N, "M": M, "op": "syr2k", "dtype": DTYPE_NAME[dtype]}}))


def run_herk(args, wl):
    """--kernel-only --herk: the Hermitian rank-k update alpha A A^H + beta C of the workload's N x M with complex128
    entries (both parts drawn N(0, 1)); 4 N (N+1) M real flops (a complex multiply-add counted as 8)."""
    import torch
    from paper_2202_10217_b200 import binding as B

    N, M = wl.N, wl.M
    if wl.dtype != I.DTYPE_F64:
        raise SystemExit("--herk is a binary64 path: give an f64 workload or --shape N,M,f64,alpha,beta")
    gen = torch.Generator(device="cuda").manual_seed(wl.seed)
    dA = torch.view_as_complex(torch.randn((N, M, 2), dtype=torch.float64, device="cuda", generator=gen))
    dC = torch.zeros((N, N), dtype=torch.complex128, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    call = lambda: B.herk_lower(N, M, dA, M, dC, N, wl.alpha, wl.beta)
    for _ in range(max(args.warmup, 1)):
        call()
    torch.cuda.synchronize()
    times = []
    for _ in range(args.steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        call()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    assert B.syrk_last_status() == 0
    ms = float(np.mean(times))
    print(json.dumps({"metric": "herk_tflops_4N(N+1)M", "value": 4 * wl.flops / (ms * 1e-3) * 1e-12, "unit": UNIT,
                      "n_gpus": 1, "steps": args.steps, "ms_per_step": ms, "kernel_only": True,
                      "config": {"workload": wl.name, "N": N, "M": M, "op": "herk", "dtype": "c128"}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=None, choices=ALL_WORKLOADS,
                    help="run this workload only (default: the sweep c5 as the headline and every workload in per_config)")
    ap.add_argument("--lbc-n", type=int, default=SWEEP_N, help="matrix size of the lbc workload")
    ap.add_argument("--block", type=int, default=0, help="panel width of the lbc workload (0 = library default)")
    ap.add_argument("--shape", default=None,
                    help="N,M,dtype,alpha,beta (dtype f64|bf16|tf32|e4m3|f16): a custom seeded N(0,1) workload")
    ap.add_argument("--kernel-only", action="store_true",
                    help="device-timed kernel steps only (no end-to-end leg, CPU baseline or peak probe); "
                         "for short profiler runs")
    ap.add_argument("--sustained", action="store_true", help="with --kernel-only: add the back-to-back leg")
    ap.add_argument("--gram", action="store_true",
                    help="with --kernel-only: hand the operand over stored M x N and time syrk_lower_tn (C = A^T A)")
    ap.add_argument("--batch", type=int, default=0,
                    help="with --kernel-only: that many problems of the workload's shape through syrk_lower_batched")
    ap.add_argument("--schedule", default="default", choices=["default", "tbs", "square", "pair", "auto"],
                    help="with --kernel-only: the library's default rule, triangle blocks at every size, the "
                         "square-block comparison schedule, or square blocks on CTA pairs")
    ap.add_argument("--syr2k", action="store_true",
                    help="with --kernel-only: time syr2k_lower_ex (rank-2k update of the workload's type) instead")
    ap.add_argument("--herk", action="store_true",
                    help="with --kernel-only: time herk_lower (Hermitian rank-k update, complex128, of the workload's N x M)")
    ap.add_argument("--kshard", action="store_true",
                    help="split the inner dimension of the workload (default c4) over the ranks: K-sharded update with "
                         "one reduce-scatter (strong scaling) instead of independent replicas")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    args = ap.parse_args()
    for flag, on in (("--schedule", args.schedule != "default"), ("--syr2k", args.syr2k), ("--herk", args.herk),
                     ("--batch", args.batch > 0), ("--gram", args.gram), ("--sustained", args.sustained)):
        if on and not args.kernel_only:
            ap.error(flag + " needs --kernel-only")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    shape = None
    if args.shape:
        n, m, dt, al, be = args.shape.split(",")
        dtype = {"f64": I.DTYPE_F64, "bf16": I.DTYPE_BF16_F32, "tf32": I.DTYPE_TF32_F32, "e4m3": I.DTYPE_E4M3_F32,
                 "f16": I.DTYPE_F16_F32}[dt]
        shape = I.Workload("custom_%s_%sx%s" % (dt, n, m), int(n), int(m), dtype, float(al), float(be), 99, "normal")
    headline = "custom" if shape is not None else (args.workload or HEADLINE)
    if args.impl == "reference":
        if headline == "lbc":
            print(json.dumps({"impl": "reference", "unavailable": "the factorisation has no oracle timing leg; use --workload c5"}))
            return
        run_reference(args, headline, shape, rank)
        return
    if args.kshard:
        key = "custom" if shape is not None else (args.workload or "c4")
        if key in ("c5", "lbc"):
            ap.error("--kshard takes a single-call workload")
        run_kshard(args, key, shape, rank, world, local_rank)
        return
    if args.kernel_only:
        if rank == 0:
            run_kernel_only(args, headline, shape, rank, world, local_rank)
        return
    keys = [headline] if (args.workload or shape is not None) else list(ALL_WORKLOADS)
    run_ours(args, keys, headline, shape, rank, world, local_rank)


if __name__ == "__main__":
    main()
