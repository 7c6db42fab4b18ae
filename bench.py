#!/usr/bin/env python
"""Benchmark of the bf16 GEMM library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One *step* is one call of the whole hot path -- ``cudallm_gemm_bf16`` on the
headline workload C2 (M = N = K = 4096, bf16 in, fp32 accumulate, bf16 out) --
on seeded synthetic operands that are already resident in HBM.  The line
printed by rank 0 carries the device-timed TFLOP/s (``value``), the same
metric through the host-buffer entry point with the copies inside the timed
region (``e2e``), the roofline fraction of the GEMM kernel against the measured
cuBLAS bf16 burst peak of this pool (``roofline``), the same kernel run back to
back for two seconds against the measured sustained peak (``sustained``, with
the SM clocks seen), the skinny HBM-bound workload C5a in GB/s against the
measured copy bandwidth (``roofline_hbm``), and the CPU oracle timed on the
host cores on a bounded sample (``cpu_baseline``).

With N > 1 every rank multiplies its own row shard of the same size: weak
scaling, no data-path collective.  Under torchrun the ranks are taken from the
environment; a plain ``python bench.py --gpus N`` starts the N ranks itself.

``--impl reference`` times the CPU oracle as it stands (no GPU work).
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
sys.path.insert(0, ROOT)

METRIC = "GEMM TFLOP/s & % of dense-bf16 peak at 4096^3; HBM GB/s & % on skinny M=16"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_BYTES = 126e6
# Where the DRAM traffic of one launch of the dominant kernel is recorded: the committed
# summaries of the ncu captures (dram__bytes_read.sum and dram__bytes_write.sum rows).
NCU_SUMMARY = {"C2": "profiles/umma_gemm_2cta_C2_4096cubed.md", "C5a": "profiles/umma_gemm_n128_C5a_skinny.md"}


def ncu_traffic_bytes(name):
    """dram read + write bytes per launch from the committed ncu summary, or None."""
    import re
    try:
        text = open(os.path.join(ROOT, NCU_SUMMARY[name])).read()
    except (OSError, KeyError):
        return None
    total = 0.0
    for key in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
        m = re.search(re.escape(key) + r"[^|\n]*\|\s*([0-9.]+)\s*MB", text)
        if not m:
            m2 = re.search(r"dram__bytes_read\.sum / write\s*\|\s*([0-9.]+)\s*MB\s*/\s*([0-9.]+)\s*MB", text)
            if not m2:
                return None
            return (float(m2.group(1)) + float(m2.group(2))) * 1e6
        total += float(m.group(1)) * 1e6
    return total


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------ clocks --
class ClockSampler:
    """Polls SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _poll_once(self):
        nv = self.nv
        try:
            mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
            r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                    if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons")
                    else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            self.samples.append(mhz)
            table = {
                "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
                "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
                "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
                "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
            }
            for name, bit in table.items():
                if r & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():       # an NVML query takes a fraction of a millisecond: no pause
            self._poll_once()

    def start(self):
        if self.nv is None:
            return
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "sm_mhz_min": s[0] if s else None, "reasons": sorted(self.reasons), "samples": len(s)}


# ------------------------------------------------------------------ helpers --
def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    return rank, local, world


def time_steps(launch, steps, warmup, barrier, sampler=None):
    """W warm-up steps, then exactly ``steps`` timed steps between two CUDA
    events on the launching stream (nothing else is enqueued in between, so
    consecutive launches follow each other as they would in an application).
    Returns (total seconds, average seconds per step)."""
    import torch
    for i in range(warmup):
        launch(i)
    torch.cuda.synchronize()
    barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if sampler:
        sampler.start()
    e0.record()
    for i in range(steps):
        launch(warmup + i)
    e1.record()
    if sampler:
        sampler._poll_once() if sampler.nv is not None else None
    torch.cuda.synchronize()
    if sampler:
        sampler.stop()
    barrier()
    torch.cuda.synchronize()
    total = e0.elapsed_time(e1) * 1e-3
    return total, total / steps


def launches_per_call(cfg):
    """Kernels of the library per call: the GEMM kernel (split tiles are summed inside it), plus
    one repacking launch if an operand cannot be addressed by TMA."""
    unaligned = (cfg.lda_ % 8 or cfg.ldb_ % 8
                 or (cfg.batch > 1 and (cfg.strideA % 8 or cfg.strideB % 8)))
    return 2 if unaligned else 1


def kernel_name(variant_name):
    """The __global__ function a variant runs."""
    if variant_name == "simt":
        return "simt_gemm_kernel"
    return "umma_gemm_2cta_kernel" if variant_name.startswith("umma2_") else "umma_gemm_kernel"


def sustained_run(launch, flops_per_call, est_s_per_call, seconds, peak_sustained, local, barrier):
    """Back-to-back calls for about `seconds` between two CUDA events, NVML clocks sampled
    throughout (sampling only).  Returns the record for the JSON line."""
    import torch
    n = max(10, int(seconds / max(est_s_per_call, 1e-7)) + 1)
    sampler = ClockSampler(local)
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    e0.record()
    for i in range(n):
        launch(i)
    e1.record()
    torch.cuda.synchronize()
    sampler.stop()
    barrier()
    t = e0.elapsed_time(e1) * 1e-3
    clocks = sampler.summary()
    tfl = flops_per_call * n / t / 1e12
    us = t / n * 1e6
    return {"value": tfl, "unit": "TFLOP/s", "seconds": t, "calls": n, "us_per_call": us,
            "peak": peak_sustained, "frac": tfl / peak_sustained, "frac_of_nominal_2250": tfl / 2250.0,
            "clocks": clocks,
            "us_x_mhz": us * clocks["sm_mhz"] if clocks["sm_mhz"] else None}


def cpu_baseline_sample(cfg, A, Bm, target_s=12.0):
    """The oracle as it stands, timed on the host cores on a bounded number of
    rows of the same workload."""
    import numpy as np
    import oracle
    cores = oracle.num_threads()
    probe_rows = np.arange(min(cfg.M, 4 * cores), dtype=np.int64)
    t0 = time.perf_counter()
    oracle.gemm_rows(A, Bm, probe_rows, cfg.N, cfg.K, cfg.lda_, cfg.ldb_)
    dt = max(time.perf_counter() - t0, 1e-6)
    rate = probe_rows.size / dt
    nrows = int(min(cfg.M, max(cores, rate * target_s)))
    nrows = max(cores, (nrows // cores) * cores)
    rows = np.arange(nrows, dtype=np.int64)
    t0 = time.perf_counter()
    oracle.gemm_rows(A, Bm, rows, cfg.N, cfg.K, cfg.lda_, cfg.ldb_)
    dt = time.perf_counter() - t0
    flops = 2.0 * nrows * cfg.N * cfg.K
    return {"value": flops / dt / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
            "sample": f"rows 0..{nrows - 1} of {cfg.name} ({nrows} x {cfg.N} x {cfg.K}), "
                      f"C_ref and S in fp64, {dt:.2f} s"}


def task_cpu_baselines(workloads):
    """The task oracles as they stand (single-threaded C), timed on the same seeded inputs and
    sizes as the GPU figures beside them (`workloads`: (task, size) pairs); algorithmic GB/s."""
    import numpy as np
    import oracle
    from paper_2506_09092_b200 import inputs as gi
    out = {}
    for task, size in workloads:
        if task == "transpose":
            A = gi.task_array(8, 0, size * size)
            t0 = time.perf_counter(); oracle.transpose_f32(A, size, size); dt = time.perf_counter() - t0
            rec = {"value": 8.0 * size * size / dt / 1e9, "sample": f"{size} x {size} fp32, {dt:.2f} s"}
            del A
        elif task == "sum":
            x = gi.task_array(14, 0, size)
            t0 = time.perf_counter(); oracle.sum_f32(x); dt = time.perf_counter() - t0
            rec = {"value": 4.0 * size / dt / 1e9, "sample": f"n = {size}, {dt:.3f} s"}
        elif task == "dot":
            x = gi.task_array(14, 0, size)
            y = gi.task_array(15, 0, size, "uniform")
            t0 = time.perf_counter(); oracle.dot_f32(x, y); dt = time.perf_counter() - t0
            rec = {"value": 8.0 * size / dt / 1e9, "sample": f"n = {size}, {dt:.3f} s"}
        else:
            batch, m = 16, 4 * size * size
            xs, g, b = gi.layernorm_inputs(4, batch, m)
            t0 = time.perf_counter(); oracle.layernorm_f32(xs, g, b, batch, m); dt = time.perf_counter() - t0
            rec = {"value": (8.0 * batch * m + 8.0 * m) / dt / 1e9,
                   "sample": f"(16, 4, {size}, {size}) fp32, y in fp64, {dt:.2f} s"}
            del xs
        rec.update({"unit": "GB/s", "cores": 1, "kind": "oracle"})
        out[(task, size)] = rec
    return out


# ------------------------------------------------------------ reference arm --
def run_reference(args):
    rank, local, world = dist_env()
    if rank != 0:
        return 0
    import numpy as np
    import oracle
    from paper_2506_09092_b200 import inputs as gi
    cfg = gi.CONFIGS["C2"]
    A, Bm = cfg.make()
    cores = oracle.num_threads()
    rows_per_step = max(cores, 64)
    rng = np.random.default_rng(0)

    def step(i):
        start = (i * rows_per_step) % (cfg.M - rows_per_step + 1)
        rows = np.arange(start, start + rows_per_step, dtype=np.int64)
        oracle.gemm_rows(A, Bm, rows, cfg.N, cfg.K, cfg.lda_, cfg.ldb_)

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(args.warmup + i)
    dt = time.perf_counter() - t0
    flops = 2.0 * rows_per_step * cfg.N * cfg.K * args.steps
    value = flops / dt / 1e12
    sample = (f"each step = {rows_per_step} consecutive rows of {cfg.name} "
              f"({rows_per_step} x {cfg.N} x {cfg.K}), C_ref and S in fp64")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def workload_name(cfg):
    out = "bf16" if cfg.out_dtype == 1 else "fp32"
    return (f"{cfg.name}: GEMM M={cfg.M} N={cfg.N} K={cfg.K} batch={cfg.batch}, bf16 in, "
            f"fp32 accumulate, {out} out, row-major")


# ------------------------------------------------------------------- our arm --
def run_ours(args):
    import numpy as np
    import torch
    from paper_2506_09092_b200 import binding as B
    from paper_2506_09092_b200 import harness as H
    from paper_2506_09092_b200 import inputs as gi
    from paper_2506_09092_b200 import sharding

    rank, local, world = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU fallback")
    B.lib()                                            # fail loudly if the library is not built
    torch.cuda.set_device(local)
    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        barrier = lambda: dist.barrier()
    else:
        barrier = lambda: None
    peaks, peak_src = load_peaks()
    stream = torch.cuda.current_stream().cuda_stream    # raw handle: no per-step Python lookups

    # ------------------------------------------------ headline workload: C2 --
    cfg = gi.CONFIGS["C2"]
    A, Bm = cfg.make()
    prob = H.DeviceProblem(cfg, A, Bm, min_bytes=3.2 * L2_BYTES)
    vname = B.describe_code(B.select_variant(cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_,
                                            cfg.batch, cfg.out_dtype))
    sampler = ClockSampler(local)
    total, kern_avg = time_steps(lambda i: prob.launch(i, stream=stream), args.steps, args.warmup,
                                 barrier, sampler)
    code, detail = B.device_status(stream)
    if code != 0:
        raise RuntimeError(f"device status {code} detail {detail:#x}")
    total_max = sharding.max_over_ranks(total, device="cuda")
    value = sharding.aggregate_throughput(cfg.flops * args.steps, world, total_max) / 1e12
    achieved = cfg.flops / kern_avg / 1e12             # one kernel per step: step time = launch duration
    n_launch = launches_per_call(cfg)

    # ---------------- the same kernel back to back for seconds (clock sag), C2 and C3 --
    sustained = {}
    if not args.no_sustained:
        sustained["C2"] = sustained_run(lambda i: prob.launch(i, stream=stream), cfg.flops, kern_avg,
                                        args.sustained_seconds, peaks["bf16_tflops_sustained"], local, barrier)
        c3 = gi.CONFIGS["C3"]
        c3p = H.DeviceProblem(c3, nsets=1)             # one set is 338 MB > L2
        c3_name = B.describe_code(B.select_variant(c3.M, c3.N, c3.K, c3.lda_, c3.ldb_, c3.ldc_, c3.batch, c3.out_dtype))
        _, c3_avg = time_steps(lambda i: c3p.launch(i, stream=stream), 20, 3, barrier)
        sustained["C3"] = sustained_run(lambda i: c3p.launch(i, stream=stream), c3.flops, c3_avg,
                                        args.sustained_seconds, peaks["bf16_tflops_sustained"], local, barrier)
        sustained["C3"].update({"workload": workload_name(c3), "variant": c3_name,
                                "burst": {"us_per_call": c3_avg * 1e6, "value": c3.flops / c3_avg / 1e12,
                                          "frac_of_burst_peak": c3.flops / c3_avg / 1e12 / peaks["bf16_tflops"]}})
        sustained["C2"].update({"workload": workload_name(cfg), "variant": vname})
        del c3p
        torch.cuda.empty_cache()
        code, detail = B.device_status(stream)
        if code != 0:
            raise RuntimeError(f"device status {code} detail {detail:#x}")

    # -------------------------------------------- e2e: host buffers, copies --
    hA = torch.from_numpy(A.view(np.int16)).pin_memory()
    hB = torch.from_numpy(Bm.view(np.int16)).pin_memory()
    hC = torch.empty(cfg.M * cfg.ldc_, dtype=torch.int16).pin_memory()
    need = B.host_staging_bytes(cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_, cfg.out_dtype)
    stage = torch.empty(need, dtype=torch.uint8, device="cuda")
    e2e_steps = max(3, min(args.steps, 20))

    def e2e_call(i):
        B.gemm_bf16_host(hA, hB, hC, cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_,
                         cfg.out_dtype, stage, need, stream)
    e2e_total, _ = time_steps(e2e_call, e2e_steps, 2, barrier)
    e2e_value = sharding.aggregate_throughput(cfg.flops * e2e_steps, world,
                                              sharding.max_over_ranks(e2e_total, device="cuda")) / 1e12

    # ------------------------------------------- skinny HBM-bound workload --
    sk = gi.CONFIGS["C5a"]
    sA, sB = sk.make()
    skp = H.DeviceProblem(sk, sA, sB, min_bytes=2.2 * L2_BYTES)
    sk_name = B.describe_code(B.select_variant(sk.M, sk.N, sk.K, sk.lda_, sk.ldb_, sk.ldc_, sk.batch,
                                              sk.out_dtype))
    sk_steps = max(args.steps, 20)
    sk_total, sk_avg = time_steps(lambda i: skp.launch(i, stream=stream), sk_steps, args.warmup, barrier)
    sk_gbs = sk.algorithmic_bytes / sk_avg / 1e9

    # ---------- the paper's literal Task 2: fp32 operands, size 2^14 of its ladder ----------
    t2 = gi.task2_ladder(2)                            # A (16384 x 4096) x B (4096 x 2048), fp32
    fa = torch.randn(t2.M, t2.K, device="cuda", generator=torch.Generator("cuda").manual_seed(7))
    fb = torch.randn(t2.K, t2.N, device="cuda", generator=torch.Generator("cuda").manual_seed(8))
    fcs = [torch.empty(t2.M, t2.N, device="cuda") for _ in range(2)]
    f_steps = max(3, min(args.steps, 10))
    f_total, f_avg = time_steps(
        lambda i: B.gemm_f32(fa, fb, fcs[i & 1], t2.M, t2.N, t2.K, t2.K, t2.N, t2.N, -1, stream),
        f_steps, 3, barrier)
    f_tflops = t2.flops / f_avg / 1e12
    tf_steps = max(3, min(args.steps, 20))
    tf_total, tf_avg = time_steps(
        lambda i: B.gemm_tf32(fa, fb, fcs[i & 1], t2.M, t2.N, t2.K, t2.K, t2.N, t2.N, stream),
        tf_steps, 3, barrier)
    tf_tflops = t2.flops / tf_avg / 1e12

    # ---------- the paper's Task 6 at its largest size: N = 512, d_model = 512, h = 16 ----------
    aN, aD, aH = 512, 512, 16
    gq = torch.Generator("cuda").manual_seed(9)
    aq, ak, av = (torch.randn(aN, aD, device="cuda", generator=gq).to(torch.bfloat16) for _ in range(3))
    ao = torch.empty(aN, aD, device="cuda")
    a_steps = max(args.steps, 50)
    a_total, a_avg = time_steps(lambda i: B.mhsa_bf16(aq, ak, av, ao, aN, aD, aH, aD, aD, aD, aD, stream),
                                a_steps, 5, barrier)

    # ---------- the bandwidth-bound float32 tasks (8, 14, 15, 4) at their largest paper size,
    #            plus a 1 GiB stream for the two reductions (the paper's largest is 4 MB) ----------
    hbm_tasks = []
    task_workloads = []
    for task, size, label in (("transpose", gi.TRANSPOSE_SIZES[-1], "Task 8"), ("layernorm", 1024, "Task 4"),
                              ("sum", gi.REDUCTION_SIZES[-1], "Task 14"), ("dot", gi.DOT_SIZES[-1], "Task 15"),
                              ("sum", 1 << 28, "Task 14 beyond the paper's sizes"),
                              ("dot", 1 << 27, "Task 15 beyond the paper's sizes")):
        launch_t, bytes_t, what = H.task_problem(task, size)
        task_workloads.append((task, size))
        t_steps = max(args.steps, 20)
        _, t_avg = time_steps(launch_t, t_steps, 3, barrier)
        hbm_tasks.append({"task": label, "call": f"cudallm_{task}_f32", "input": what, "us_per_call": t_avg * 1e6,
                          "steps": t_steps, "value": bytes_t / t_avg / 1e9, "unit": "GB/s (algorithmic bytes)",
                          "frac_of_measured_hbm": bytes_t / t_avg / 1e9 / peaks["hbm_gbs"]})
        del launch_t
        torch.cuda.empty_cache()

    line = None
    if rank == 0:
        clocks = sampler.summary()
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_max / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {
                "workload": workload_name(cfg), "variant": vname,
                "inputs": "A, B ~ N(0,1) rounded to bf16, numpy default_rng([1,0]) / ([1,1])",
                "l2": f"rotating {prob.nsets} operand/output sets ({prob.nsets * prob.set_bytes / 1e6:.0f} MB)"
                      f" > {L2_BYTES / 1e6:.0f} MB L2",
                "sharding": f"rank r owns rows [{cfg.M}*r, {cfg.M}*(r+1)) of a {sharding.weak_scaling_rows(cfg.M, world)}-row product "
                            "(B replicated), no data-path collective",
            },
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "TFLOP/s",
                    "h2d_bytes_per_step": int(A.nbytes + Bm.nbytes),
                    "d2h_bytes_per_step": int(cfg.M * cfg.N * cfg.out_bytes),
                    "steps": e2e_steps, "call": "cudallm_gemm_bf16_host (pinned host buffers)"},
            "gpu_launches": n_launch * args.steps,
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"],
                         "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                         "traffic": ncu_traffic_bytes("C2"), "traffic_source": NCU_SUMMARY["C2"],
                         "peak_source": f"of {peak_src} (burst: the timed region is milliseconds long)",
                         "kernel": f"{kernel_name(vname)} ({vname})",
                         "frac_of_nominal_2250": achieved / 2250.0},
            # the second half of the metric: the skinny M = 16 product against the copy bandwidth
            "roofline_hbm": {"workload": workload_name(sk), "variant": sk_name, "kernel": f"{kernel_name(sk_name)} ({sk_name})",
                             "bound": "hbm", "achieved": sk_gbs, "value": sk_gbs, "peak": peaks["hbm_gbs"],
                             "unit": "GB/s", "frac": sk_gbs / peaks["hbm_gbs"],
                             "traffic": ncu_traffic_bytes("C5a"), "traffic_source": NCU_SUMMARY["C5a"],
                             "peak_source": f"of {peak_src}", "us_per_call": sk_avg * 1e6, "steps": sk_steps,
                             "frac_of_nominal_8000": sk_gbs / 8000.0},
            "sustained": sustained,
        }
        line["task2_fp32"] = {
            "workload": f"paper Task 2, size 2^14: A ({t2.M} x {t2.K}) x B ({t2.K} x {t2.N}), fp32 in and out, N(0,1)",
            "call": "cudallm_gemm_f32 (three bf16 pieces per operand, six piece products, fp32 accumulate)",
            "value": f_tflops, "unit": "TFLOP/s (2MNK)", "us_per_call": f_avg * 1e6, "steps": f_steps,
            "tensor_rate": {"value": 6 * f_tflops, "unit": "TFLOP/s of bf16 MMA work (6 x 2MNK)",
                            "frac_of_measured_bf16_peak": 6 * f_tflops / peaks["bf16_tflops"]},
            "note": "inputs 436 MB > L2; fp32-grade accuracy (<= 1e-5 * sum|a||b|, observed ~1e-7)",
            "tf32": {"call": "cudallm_gemm_tf32 (operands read in place, tcgen05.mma kind::tf32)",
                     "value": tf_tflops, "unit": "TFLOP/s (2MNK)", "us_per_call": tf_avg * 1e6, "steps": tf_steps,
                     "peak": peaks["bf16_tflops"] * 0.5,
                     "frac": tf_tflops / (peaks["bf16_tflops"] * 0.5),
                     "peak_source": f"half of the bf16 peak {peak_src} (the nominal ratio of the two dense rates)",
                     "note": "<= 2.5e-3 * sum|a||b| (ten fraction bits per operand)"}}
        line["task6_attention"] = {
            "workload": f"paper Task 6, largest size: N={aN}, d_model={aD}, h={aH} (d_k={aD // aH}), bf16 in, fp32 out",
            "call": "cudallm_mhsa_bf16 (one fused kernel, 64 CTAs)", "us_per_call": a_avg * 1e6,
            "steps": a_steps, "value": 4.0 * aN * aN * aD / a_avg / 1e12, "unit": "TFLOP/s (4 N^2 d_model)",
            "note": "2.6 MB of operands and output: L2-resident and launch-latency bound, no roofline claimed"}
        line["hbm_tasks_f32"] = hbm_tasks
        if world == 1:
            line["cpu_baseline"] = cpu_baseline_sample(cfg, A, Bm)
            if not args.no_task_baselines:
                cpu_tasks = task_cpu_baselines(task_workloads)
                for entry, key in zip(hbm_tasks, task_workloads):
                    entry["cpu_baseline"] = cpu_tasks[key]
    if use_dist:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line), flush=True)
    return 0


def self_launch(args):
    """`python bench.py --gpus N` outside torchrun: start the N ranks here, one per GPU."""
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        port = so.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--sustained-seconds", type=float, default=2.2,
                    help="length of the back-to-back runs of C2 and C3 behind the `sustained` record")
    ap.add_argument("--no-sustained", action="store_true", help="skip the seconds-long runs")
    ap.add_argument("--no-task-baselines", action="store_true",
                    help="skip timing the CPU oracles of the float32 tasks")
    args = ap.parse_args()
    if args.steps < 1:
        ap.error("--steps must be >= 1")
    if args.gpus < 1:
        ap.error("--gpus must be >= 1")
    args.warmup = max(args.warmup, 3)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return self_launch(args)
    if "WORLD_SIZE" in os.environ and int(os.environ["WORLD_SIZE"]) != args.gpus:
        ap.error(f"--gpus {args.gpus} but WORLD_SIZE={os.environ['WORLD_SIZE']}")
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
