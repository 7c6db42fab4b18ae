"""Validate / profile / arg-min over kernel variants, shaped like the paper's
Feature Search and Reinforcement loop (Algorithm 1) without the LLM.

Algorithm 1 draws candidates, keeps the set V of those that pass the
Compilation Verifier and the Function Validator, profiles V, and keeps the
fastest.  Here the candidates are the library's precompiled kernel variants
(compilation is checked when the library is built), so one pass is:

    V      <- { k in candidates : function_validator(k) }
    k*     <- argmin_{k in V} performance_profiler(k)
    return (k*, tau*)            # or a failure report when V is empty

Algorithm 1 as printed loops again without advancing the depth when V is
empty; with a fixed candidate list that could never end, so an empty V is
reported as a failure instead.

The reference outputs come from the caller (``expected`` callables): this
module never imports a CPU implementation of the product, it only compares.
Failure classes mirror the paper's three refinement prompts: launch failure,
output mismatch (plus timeout, which the bounded in-kernel waits add).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Callable, Iterable, Sequence

OK = "OK"
UNSUPPORTED = "UNSUPPORTED"
LAUNCH_FAIL = "LAUNCH_FAIL"
MISMATCH = "MISMATCH"
TIMEOUT = "TIMEOUT"


@dataclass
class ValidationReport:
    status: str
    cases: int = 0
    failed_case: str = ""
    detail: str = ""
    max_scaled_err: float = 0.0

    @property
    def ok(self):
        return self.status == OK


@dataclass
class SearchResult:
    best: int | None                      # k_best (None if V is empty)
    best_latency: float                   # tau_best, seconds (inf if none)
    valid: list = field(default_factory=list)          # V
    reports: dict = field(default_factory=dict)        # candidate -> ValidationReport
    latencies: dict = field(default_factory=dict)      # candidate -> seconds


def function_validator(candidate, cases: Iterable, run: Callable, compare: Callable) -> ValidationReport:
    """Run ``candidate`` on every test case and compare with the expected output.

    ``run(candidate, case)`` returns ``(status_code, output)`` where a non-zero
    status is a launch failure, -9 a device timeout and ``None`` output with
    status ``"unsupported"`` means the candidate cannot take the case.
    ``compare(case, output)`` returns ``(ok, max_scaled_err, detail)``.
    """
    n = 0
    worst = 0.0
    for case in cases:
        status, out = run(candidate, case)
        name = getattr(case, "name", str(case))
        if status == "unsupported":
            return ValidationReport(UNSUPPORTED, n, name)
        if status == -9:
            return ValidationReport(TIMEOUT, n, name, "a bounded wait inside the kernel ran out")
        if status != 0:
            return ValidationReport(LAUNCH_FAIL, n, name, f"status {status}")
        ok, err, detail = compare(case, out)
        worst = max(worst, err if math.isfinite(err) else float("inf"))
        n += 1
        if not ok:
            return ValidationReport(MISMATCH, n, name, detail, worst)
    return ValidationReport(OK, n, max_scaled_err=worst)


def search(candidates: Sequence[int], validate: Callable[[int], ValidationReport],
           profile: Callable[[int], float]) -> SearchResult:
    """One round of Algorithm 1 over a fixed candidate list."""
    res = SearchResult(best=None, best_latency=float("inf"))
    for k in candidates:
        rep = validate(k)
        res.reports[k] = rep
        if rep.ok:
            res.valid.append(k)
    for k in res.valid:
        tau = float(profile(k))
        res.latencies[k] = tau
        if tau < res.best_latency:          # strict: ties keep the earlier candidate
            res.best, res.best_latency = k, tau
    return res


# ---------------------------------------------------------------- on the GPU --

def performance_profiler(launch: Callable[[int], None], iters: int = 20, warmup: int = 3,
                         batch_calls: int = 1) -> dict:
    """Time ``launch(i)`` with CUDA events on the current stream.

    ``launch(i)`` enqueues call number ``i`` (callers rotate buffer sets with it
    so that successive calls do not hit in L2).  Each of ``iters`` samples
    brackets ``batch_calls`` back-to-back calls.  Returns min / median seconds
    per call."""
    import torch
    for i in range(warmup):
        launch(i)
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(iters)]
    n = warmup
    for e0, e1 in evs:
        e0.record()
        for _ in range(batch_calls):
            launch(n)
            n += 1
        e1.record()
    torch.cuda.synchronize()
    ts = sorted(e0.elapsed_time(e1) * 1e-3 / batch_calls for e0, e1 in evs)
    return {"min_s": ts[0], "median_s": ts[len(ts) // 2], "samples": len(ts)}


class DeviceProblem:
    """Device-resident operands for one configuration, in ``nsets`` rotating
    copies so that a timed call does not find the previous call's data in L2."""

    def __init__(self, cfg, A_bits=None, B_bits=None, min_bytes: float = 300e6, nsets: int | None = None):
        import numpy as np
        import torch
        from . import inputs as gi
        self.cfg = cfg
        if A_bits is None or B_bits is None:
            A_bits, B_bits = cfg.make()
        esz = cfg.out_bytes
        nC = cfg.batch * cfg.strideC
        set_bytes = A_bits.nbytes + B_bits.nbytes + nC * esz
        if nsets is None:
            nsets = max(1, int(min_bytes // set_bytes) + 1)
        self.nsets = nsets
        self.set_bytes = set_bytes
        a0 = torch.from_numpy(A_bits.view(np.int16)).cuda()
        b0 = torch.from_numpy(B_bits.view(np.int16)).cuda()
        self.sets = []
        for i in range(nsets):
            a = a0 if i == 0 else a0.clone()
            b = b0 if i == 0 else b0.clone()
            c = torch.empty(nC * esz, dtype=torch.uint8, device="cuda")
            self.sets.append((a, b, c))

    def launch(self, i: int, variant: int = -1, stream=None, check: bool = True) -> int:
        import torch
        from . import binding as B
        cfg = self.cfg
        a, b, c = self.sets[i % self.nsets]
        return B.gemm_bf16_variant(variant, a, b, c, cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_,
                                   cfg.strideA, cfg.strideB, cfg.strideC, cfg.batch, cfg.out_dtype,
                                   stream if stream is not None else torch.cuda.current_stream(),
                                   check=check)

    def output(self, i: int = 0):
        """C of set ``i`` as a host numpy array of raw elements [batch, M, ldc-strided]."""
        import numpy as np
        import torch
        cfg = self.cfg
        torch.cuda.synchronize()
        raw = self.sets[i % self.nsets][2].cpu().numpy()
        return raw.view(np.float32 if cfg.out_dtype == 0 else np.uint16)


def _main(argv=None):
    """``python -m paper_2506_09092_b200.harness --config C2``: run one benchmark
    configuration a few times and print its timing (also the command that ncu
    captures are taken from)."""
    import argparse
    import json
    import torch
    from . import binding as B
    from . import inputs as gi

    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="C2", choices=sorted(gi.CONFIGS))
    ap.add_argument("--variant", default="auto")
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--sets", type=int, default=None, help="rotating buffer sets (default: > L2)")
    ap.add_argument("--all-variants", action="store_true", help="time every variant that supports the shape")
    args = ap.parse_args(argv)
    cfg = gi.CONFIGS[args.config]
    names = {B.variant_name(v): v for v in range(B.num_variants())}
    prob = DeviceProblem(cfg, nsets=args.sets)
    if args.all_variants:
        todo = [v for v in range(1, B.num_variants())
                if B.variant_supports(v, cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_, cfg.batch,
                                      cfg.out_dtype) == 1]
    elif args.variant == "auto":
        todo = [B.select_variant(cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_, cfg.batch, cfg.out_dtype)]
    else:
        todo = [names[args.variant]]
    for v in todo:
        t = performance_profiler(lambda i: prob.launch(i, v), iters=args.iters, warmup=args.warmup)
        code, detail = B.device_status(torch.cuda.current_stream())
        print(json.dumps({"config": cfg.name, "variant": B.variant_name(v), "status": code,
                          "us_min": t["min_s"] * 1e6, "us_median": t["median_s"] * 1e6,
                          "tflops": cfg.flops / t["median_s"] / 1e12,
                          "gbs": cfg.algorithmic_bytes / t["median_s"] / 1e9}), flush=True)


if __name__ == "__main__":
    _main()
