#!/usr/bin/env python
"""Benchmark of the triangle-block SYRK library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c1|c5]
                    [--impl ours|reference]

A step is one SYRK call (the whole hot path: work-list lookup, TMA streaming, tensor-core
update, epilogue) on one seeded synthetic workload.  Prints ONE JSON line (rank 0).
With N > 1 every rank runs an independent replica on its own GPU (the path has no
exchange step); the value is the sum over ranks divided by the slowest rank's time.
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

import numpy as np

from paper_2202_10217_b200 import inputs as I

METRIC = "syrk_tflops_N(N+1)M"
UNIT = "TFLOP/s"
DTYPE_NAME = {I.DTYPE_F64: "f64", I.DTYPE_BF16_F32: "bf16_in_f32_acc", I.DTYPE_TF32_F32: "tf32_in_f32_acc",
              I.DTYPE_E4M3_F32: "fp8_e4m3_in_f32_acc", I.DTYPE_F16_F32: "f16_in_f32_acc"}
ELEM_A = {I.DTYPE_F64: 8, I.DTYPE_BF16_F32: 2, I.DTYPE_TF32_F32: 4, I.DTYPE_E4M3_F32: 1, I.DTYPE_F16_F32: 2}
ELEM_C = {I.DTYPE_F64: 8, I.DTYPE_BF16_F32: 4, I.DTYPE_TF32_F32: 4, I.DTYPE_E4M3_F32: 4, I.DTYPE_F16_F32: 4}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons (one `nvidia-smi -lms` process) while the
    timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, period_ms: int = 20):
        self.cmd = ["nvidia-smi", "-i", str(index), "--query-gpu=" + self.QUERY,
                    "--format=csv,noheader,nounits", "-lms", str(period_ms)]
        self.proc = None
        self.rows = []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(self.cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            time.sleep(0.15)                      # let the first samples arrive before the load starts
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is None:
            return
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
                sm.append(float(r[0]))
                mx = max(mx, float(r[1]))
                power.append(float(r[2]))
                for name, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        # "under load": samples drawing more than half of the largest power seen
        load = [c for c, w in zip(sm, power) if power and w >= 0.5 * max(power)]
        return {"sm_mhz": float(np.median(load)) if load else None, "sm_max_mhz": mx or None,
                "reasons": sorted(reasons), "samples": len(sm), "samples_under_load": len(load),
                "power_w_max": max(power) if power else None}


def cpu_reference_sample(wl: I.Workload, A: np.ndarray, target_macs: float = 2.0e11):
    """Times the CPU reference, as it stands, on a bounded sample of the workload.

    The sample is the first R rows of the lower triangle (R chosen so that the work is
    about `target_macs` multiply-adds); throughput is scaled to the metric's unit by the
    flops of the sampled part, 2 * M per entry.
    """
    from oracle import syrk as O
    N, M = wl.N, wl.M
    R = int(min(N, max(64, np.sqrt(2.0 * target_macs / M))))
    sub = np.ascontiguousarray(A[:R])
    t0 = time.perf_counter()
    O.syrk_lower(sub, None, wl.alpha, 0.0, wl.dtype)
    dt = time.perf_counter() - t0
    flops = R * (R + 1) * M
    return {"value": flops / dt * 1e-12, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
            "sample": "first %d of %d rows of the lower triangle (%.3g flops, %.1f s)" % (R, N, flops, dt)}


def run_reference(args, wl: I.Workload, rank: int):
    """--impl reference: the CPU oracle on host cores, rank 0 only."""
    if rank != 0:
        return
    A = wl.make_A()
    target = 6.0e9
    for _ in range(args.warmup):
        cpu_reference_sample(wl, A, target_macs=target / 8)
    vals, t0 = [], time.perf_counter()
    for _ in range(args.steps):
        vals.append(cpu_reference_sample(wl, A, target_macs=target))
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    last = vals[-1]
    value = float(np.mean([v["value"] for v in vals]))
    base = dict(last)
    base["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "N": wl.N, "M": wl.M, "alpha": wl.alpha, "beta": wl.beta,
                   "note": "CPU oracle (plain triple loop) on a bounded sample per step"},
        "cpu_baseline": base,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/.  Valid only for the kernel source it was taken on.
NCU_TRAFFIC = {
    # workload: (bytes per launch, sha256 of the kernel source at capture time)
    "c2_f64_4096x4096": (550_938_112, "5ff99b8d23c3c4eedbfdffd679b1b3bb77d03743e9c42059eea89c7430b6c642"),
    "c3_bf16_16384x4096": (1_938_945_792, "4821ed7dd649bee40152f9f9c7cae9ba3a0f61e5860377e22447fa74776ae46e"),
    "c4_bf16_2048x262144": (2_929_146_880, "4821ed7dd649bee40152f9f9c7cae9ba3a0f61e5860377e22447fa74776ae46e"),
}


def max_over_ranks(value: float, dist, device) -> float:
    """Slowest rank's time (every rank gets it); the identity without a process group."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(flops_per_replica: int, world: int, seconds: float) -> float:
    """Replicas only: every rank does the same work, the job lasts as long as its slowest rank."""
    return world * flops_per_replica / seconds * 1e-12


def kernel_source_hash(dtype: int) -> str:
    import hashlib
    name = "syrk_f64.cu" if dtype == I.DTYPE_F64 else "syrk_bf16.cu"
    with open(os.path.join(ROOT, "paper_2202_10217_b200", "csrc", name), "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()


def run_ours(args, wl: I.Workload, rank: int, world: int, local_rank: int):
    import torch
    from paper_2202_10217_b200 import binding as B

    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    N, M, dtype = wl.N, wl.M, wl.dtype
    if args.batch > 0:
        run_batched(args, wl)
        return
    if args.syr2k:
        run_syr2k(args, wl)
        return
    A_host = wl.make_A()
    cdt = I.c_storage_dtype(dtype)
    if dtype in (I.DTYPE_F64, I.DTYPE_TF32_F32, I.DTYPE_E4M3_F32):
        A_pinned = torch.from_numpy(A_host).pin_memory()
        dA = A_pinned.cuda()
    else:
        A_pinned = torch.from_numpy(A_host.view(np.int16)).pin_memory()
        dA = A_pinned.cuda().view(torch.bfloat16)
    C_pinned = torch.zeros((N, N), dtype=torch.float64 if dtype == I.DTYPE_F64 else torch.float32).pin_memory()
    dC = torch.zeros((N, N), dtype=C_pinned.dtype, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")     # > L2 (126 MB)

    if args.schedule != "tbs":                            # comparison schedules (kernel-only runs)
        B.syrk_set_schedule({"square": B.SCHEDULE_SQUARE, "pair": B.SCHEDULE_PAIR_SQUARE, "auto": B.SCHEDULE_AUTO}[args.schedule])
    B.syrk_plan_prepare(N, M, dtype)
    stats = B.syrk_get_schedule_stats(N, M, dtype)
    n_warm = args.warmup if args.kernel_only else max(args.warmup, 3)
    if args.gram:                                          # same operand stored M x N: C = A^T A
        dA = dA.t().contiguous()
        device_call = lambda: B.syrk_lower_tn(N, M, dA, N, dC, N, wl.alpha, wl.beta, dtype)
    else:
        device_call = lambda: B.syrk_lower(N, M, dA, M, dC, N, wl.alpha, wl.beta, dtype)
    for _ in range(n_warm):
        device_call()
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0

    ev0 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ev1 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    with ClockSampler(local_rank) as clocks:
        for i in range(args.steps):
            flush.zero_()                                  # evict A and C from L2 (not timed)
            ev0[i].record()
            device_call()
            ev1[i].record()
        barrier()
    assert B.syrk_last_status() == 0
    times = [a.elapsed_time(b) for a, b in zip(ev0, ev1)]
    total_ms = float(sum(times))
    total_ms = max_over_ranks(total_ms, dist, "cuda")
    ms_per_step = total_ms / args.steps
    value = whole_job_tflops(wl.flops, world, ms_per_step * 1e-3)

    if args.kernel_only:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
                              "steps": args.steps, "ms_per_step": ms_per_step, "kernel_only": True,
                              "config": {"workload": wl.name, "N": N, "M": M, "schedule": args.schedule,
                                         "operand": "M x N (Gram form)" if args.gram else "N x M"}}))
        return

    # end to end: host buffers through the C ABI, copies inside the timed region
    e2e_steps = max(1, min(args.steps, 3))
    B.syrk_lower_host(N, M, A_pinned, M, C_pinned, N, wl.alpha, wl.beta, dtype)      # warm-up (allocates staging)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        B.syrk_lower_host(N, M, A_pinned, M, C_pinned, N, wl.alpha, wl.beta, dtype)
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    e2e_s = max_over_ranks(e2e_s, dist, "cuda")
    e2e = {"value": whole_job_tflops(wl.flops, world, e2e_s), "unit": UNIT,
           "h2d_bytes_per_step": N * M * ELEM_A[dtype] + (N * N * ELEM_C[dtype] if wl.beta != 0 else 0),
           "d2h_bytes_per_step": N * (N + 1) // 2 * ELEM_C[dtype]}

    if rank != 0:
        return
    peaks, peak_kind = measured_peaks()
    kernel_ms = float(np.mean(times))
    achieved = wl.flops / (kernel_ms * 1e-3) * 1e-12
    if dtype == I.DTYPE_F64:
        peak = B.syrk_probe_f64_mma_peak(20000)
        peak_note = ("FP64 tensor-core (DMMA) rate measured in this run by the library's register-only "
                     "mma.sync probe; MEASURED_PEAKS.json has no FP64 figure (bf16 %s %.1f x 40/2250 = %.1f)"
                     % (peak_kind, peaks["bf16_tflops"], peaks["bf16_tflops"] * 40.0 / 2250.0))
    elif dtype == I.DTYPE_E4M3_F32:
        # no measured FP8 figure: the measured bf16 burst peak times the nominal ratio 4.5 / 2.25 PFLOP/s
        peak = float(peaks["bf16_tflops"]) * 2.0
        peak_note = "cuBLAS bf16 burst, MEASURED_PEAKS.json (%s), x nominal fp8/bf16 ratio 2" % peak_kind
    elif dtype == I.DTYPE_TF32_F32:
        # no measured TF32 figure: the measured bf16 burst peak times the nominal ratio 1.1 / 2.25 PFLOP/s
        peak = float(peaks["bf16_tflops"]) * 1.1 / 2.25
        peak_note = "cuBLAS bf16 burst, MEASURED_PEAKS.json (%s), x nominal tf32/bf16 ratio 1.1/2.25" % peak_kind
    else:
        peak = float(peaks["bf16_tflops"])
        peak_note = "cuBLAS bf16 burst, MEASURED_PEAKS.json (%s); sustained %.1f" % (
            peak_kind, peaks.get("bf16_tflops_sustained", float("nan")))
    traffic = None
    if wl.name in NCU_TRAFFIC and NCU_TRAFFIC[wl.name][1] == kernel_source_hash(dtype):
        traffic = NCU_TRAFFIC[wl.name][0]
    launches_per_step = 1 if dtype == I.DTYPE_F64 else (2 if stats["split_k"] > 1 else 1)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": DTYPE_NAME[dtype], "data": "synthetic",
        "config": {"workload": wl.name, "N": N, "M": M, "alpha": wl.alpha, "beta": wl.beta,
                   "schedule": "tbs", "tile": stats["tile"], "k": stats["k"], "items": stats["items"],
                   "tri_items": stats["tri_items"], "parallelism": "replicas only" if world > 1 else "1 gpu",
                   "l2": "256 MiB buffer written between timed steps (L2 flush)"},
        "clocks": clocks.summary(),
        "e2e": e2e,
        "gpu_launches": args.steps * launches_per_step,
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": UNIT,
                     "frac": achieved / peak, "traffic": traffic, "peak_source": peak_note,
                     "algorithmic_flops_per_launch": wl.flops,
                     "model_a_bytes_per_launch": stats["a_loads"] * ELEM_A[dtype]},
    }
    if world == 1:
        line["cpu_baseline"] = cpu_reference_sample(wl, A_host)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_sweep(args, rank: int, world: int, local_rank: int):
    """Config 5: C_n <- C_n - A_n A_n^T on the trailing n x n view of one 32768^2 FP64 matrix,
    n = 32768, 32256, ..., 512 (64 calls, M = 512, ldc = 32768).  One step = the whole sweep."""
    import torch
    from paper_2202_10217_b200 import binding as B

    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    n_max, step, M = 32768, 512, I.SWEEP_K
    sizes = I.sweep_sizes(n_max, step)
    flops = sum(n * (n + 1) * M for n in sizes)
    # A_n = the trailing n rows of one seeded n_max x 512 panel (same shapes, pitches and value
    # distribution as a fresh panel per step); C = n_max * I + G G^T / 512 prepared with torch.
    A_pinned = torch.from_numpy(I.sweep_panel(n_max, n_max)).pin_memory()
    dA = A_pinned.cuda()
    G = torch.from_numpy(I.sweep_factor(n_max)).cuda()
    C = torch.matmul(G, G.T) / float(M)
    C.diagonal().add_(float(n_max))
    del G
    diag_host = torch.empty(n_max, dtype=torch.float64).pin_memory()
    for n in sizes:
        B.syrk_plan_prepare(n, M, I.DTYPE_F64)

    def sweep(src):
        for n in sizes:
            off = n_max - n
            B.syrk_lower(n, M, src.data_ptr() + off * M * 8, M, C.data_ptr() + (off * n_max + off) * 8, n_max,
                         -1.0, 1.0, I.DTYPE_F64)

    steps = max(1, min(args.steps, 10))
    for _ in range(1 if args.kernel_only else 3):
        sweep(dA)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    ev0 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ev1 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    barrier()
    with ClockSampler(local_rank) as clocks:
        for i in range(steps):
            ev0[i].record()
            sweep(dA)
            ev1[i].record()
        barrier()
    assert B.syrk_last_status() == 0
    times = [a.elapsed_time(b) for a, b in zip(ev0, ev1)]
    ms_per_step = max_over_ranks(float(sum(times)), dist, "cuda") / steps
    value = whole_job_tflops(flops, world, ms_per_step * 1e-3)
    if args.kernel_only:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
                              "ms_per_step": ms_per_step, "kernel_only": True,
                              "config": {"workload": "c5_f64_sweep_32768..512_x512"}}))
        return
    # end to end: every panel copied from pinned host memory before its call, the diagonal read back
    dA2 = torch.empty_like(dA)
    barrier()
    t0 = time.perf_counter()
    for n in sizes:
        off = n_max - n
        dA2[off:].copy_(A_pinned[off:], non_blocking=True)
        B.syrk_lower(n, M, dA2.data_ptr() + off * M * 8, M, C.data_ptr() + (off * n_max + off) * 8, n_max,
                     -1.0, 1.0, I.DTYPE_F64)
    diag_host.copy_(C.diagonal(), non_blocking=True)
    torch.cuda.synchronize()
    e2e_s = max_over_ranks(time.perf_counter() - t0, dist, "cuda")
    if rank != 0:
        return
    peak = B.syrk_probe_f64_mma_peak(20000)
    achieved = flops / (float(np.mean(times)) * 1e-3) * 1e-12
    small = I.Workload("c5_step_n4096", 4096, M, I.DTYPE_F64, -1.0, 1.0, I.SWEEP_SEED, "normal", std=M ** -0.5)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": 3,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "c5_f64_sweep_32768..512_x512", "calls_per_step": len(sizes), "M": M, "alpha": -1.0,
                   "beta": 1.0, "ldc": n_max, "schedule": "tbs",
                   "l2": "inputs larger than L2 (C view 8.6 GB .. 2 MB, read and written once per call)"},
        "clocks": clocks.summary(),
        "e2e": {"value": whole_job_tflops(flops, world, e2e_s), "unit": UNIT,
                "h2d_bytes_per_step": sum(n * M * 8 for n in sizes), "d2h_bytes_per_step": n_max * 8},
        "gpu_launches": steps * len(sizes),
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": UNIT, "frac": achieved / peak,
                     "traffic": None, "peak_source": "FP64 DMMA rate measured in this run by the library's probe",
                     "algorithmic_flops_per_launch": flops / len(sizes)},
    }
    if world == 1:
        line["cpu_baseline"] = cpu_reference_sample(small, small.make_A())
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


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
    """--kernel-only --syr2k: the rank-2k update alpha (A B^T + B A^T) + beta C of the workload's shape
    (binary64; B drawn like A from the next seed); 2 N (N+1) M flops."""
    import torch
    from paper_2202_10217_b200 import binding as B

    N, M = wl.N, wl.M
    dA = torch.from_numpy(wl.make_A()).cuda()
    dB = torch.from_numpy(I.Workload(wl.name, N, M, wl.dtype, wl.alpha, wl.beta, wl.seed + 1, wl.dist, wl.std).make_A()).cuda()
    dC = torch.zeros((N, N), dtype=torch.float64, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(max(args.warmup, 1)):
        B.syr2k_lower(N, M, dA, M, dB, M, dC, N, wl.alpha, wl.beta)
    torch.cuda.synchronize()
    times = []
    for _ in range(args.steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.syr2k_lower(N, M, dA, M, dB, M, dC, N, wl.alpha, wl.beta)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    assert B.syrk_last_status() == 0
    ms = float(np.mean(times))
    print(json.dumps({"metric": "syr2k_tflops_2N(N+1)M", "value": 2 * wl.flops / (ms * 1e-3) * 1e-12, "unit": UNIT,
                      "n_gpus": 1, "steps": args.steps, "ms_per_step": ms, "kernel_only": True,
                      "config": {"workload": wl.name, "N": N, "M": M, "op": "syr2k"}}))


def run_cholesky(args, rank: int, world: int, local_rank: int):
    """Large Block Cholesky of a seeded 32768^2 FP64 matrix (n*I + G G^T / 512); a step is one
    factorisation (the matrix is restored from a device copy between steps, outside the timing)."""
    import torch
    from paper_2202_10217_b200 import binding as B

    torch.cuda.set_device(local_rank)
    n, M = args.lbc_n, I.SWEEP_K
    G = torch.from_numpy(I.sweep_factor(n)).cuda()
    A0 = torch.matmul(G, G.T) / float(M)
    A0.diagonal().add_(float(n))
    del G
    A = A0.clone()
    flops = n ** 3 / 3.0
    steps = max(1, min(args.steps, 5))
    times = []
    for i in range(steps + 1):                       # first pass is the warm-up (allocates work lists)
        A.copy_(A0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.cholesky_lower(n, A, n, args.block)
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
    rec = (L[idx] * L[jdx]).sum(dim=1)
    err = float((rec - A0[idx, jdx]).abs().max() / A0.abs().max())
    peak = B.syrk_probe_f64_mma_peak(20000)
    print(json.dumps({"metric": "cholesky_tflops_N^3/3", "value": flops / (ms * 1e-3) * 1e-12, "unit": UNIT,
                      "n_gpus": 1, "steps": steps, "ms_per_step": ms, "higher_is_better": True, "dtype": "f64",
                      "data": "synthetic", "config": {"workload": "lbc_f64_%d" % n, "block": args.block or 512},
                      "sampled_relative_residual": err, "gpu_launches": None,
                      "roofline": {"bound": "tensor", "achieved": flops / (ms * 1e-3) * 1e-12, "peak": peak,
                                   "unit": UNIT, "frac": flops / (ms * 1e-3) * 1e-12 / peak, "traffic": None}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c2", choices=sorted(I.CONFIGS) + ["c5", "lbc"])
    ap.add_argument("--lbc-n", type=int, default=32768, help="matrix size of --workload lbc")
    ap.add_argument("--block", type=int, default=0, help="panel width of --workload lbc (0 = library default)")
    ap.add_argument("--shape", default=None,
                    help="N,M,dtype,alpha,beta (dtype f64|bf16|tf32|e4m3|f16): a custom seeded N(0,1) workload")
    ap.add_argument("--kernel-only", action="store_true",
                    help="device-timed kernel steps only (no end-to-end leg, CPU baseline or peak probe); "
                         "for short profiler runs")
    ap.add_argument("--gram", action="store_true",
                    help="with --kernel-only: hand the operand over stored M x N and time syrk_lower_tn (C = A^T A)")
    ap.add_argument("--batch", type=int, default=0,
                    help="with --kernel-only: that many problems of the workload's shape through syrk_lower_batched")
    ap.add_argument("--schedule", default="tbs", choices=["tbs", "square", "pair", "auto"],
                    help="with --kernel-only: the triangle-block schedule (default), the square-block comparison "
                         "schedule, or square blocks on CTA pairs (16-bit types)")
    ap.add_argument("--syr2k", action="store_true",
                    help="with --kernel-only and an f64 workload: time syr2k_lower (rank-2k update) instead")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    args = ap.parse_args()
    if args.schedule != "tbs" and not args.kernel_only:
        ap.error("--schedule needs --kernel-only")
    if args.syr2k and not args.kernel_only:
        ap.error("--syr2k needs --kernel-only")
    if args.batch > 0 and not args.kernel_only:
        ap.error("--batch needs --kernel-only")
    if args.gram and not args.kernel_only:
        ap.error("--gram needs --kernel-only (the host-buffer entry point takes the N x M form)")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.workload == "lbc":
        if rank == 0 and args.impl != "reference":
            run_cholesky(args, rank, world, local_rank)
        return
    if args.workload == "c5" and not args.shape:
        if args.impl == "reference":
            args.workload = "c2"                     # the oracle arm samples a single FP64 call
        else:
            run_sweep(args, rank, world, local_rank)
            return
    wl = I.CONFIGS[args.workload]
    if args.shape:
        n, m, dt, al, be = args.shape.split(",")
        dtype = {"f64": I.DTYPE_F64, "bf16": I.DTYPE_BF16_F32, "tf32": I.DTYPE_TF32_F32, "e4m3": I.DTYPE_E4M3_F32,
                 "f16": I.DTYPE_F16_F32}[dt]
        wl = I.Workload("custom_%s_%sx%s" % (dt, n, m), int(n), int(m), dtype, float(al), float(be), 99, "normal")
    if args.impl == "reference":
        run_reference(args, wl, rank)
        return
    run_ours(args, wl, rank, world, local_rank)


if __name__ == "__main__":
    main()
