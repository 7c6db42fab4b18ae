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
        self._calls = {}
        self.stream_handle = torch.cuda.current_stream().cuda_stream
        for i in range(nsets):
            a = a0 if i == 0 else a0.clone()
            b = b0 if i == 0 else b0.clone()
            c = torch.empty(nC * esz, dtype=torch.uint8, device="cuda")
            self.sets.append((a, b, c))

    def _bound(self, variant: int, stream_handle):
        """Per buffer set, the C call with its arguments already converted (the
        conversion costs more than a small GEMM takes on the device)."""
        import ctypes
        from . import binding as B
        key = (variant, stream_handle)
        calls = self._calls.get(key)
        if calls is None:
            cfg = self.cfg
            fn = B.lib().cudallm_gemm_bf16_variant
            i64 = ctypes.c_int64
            calls = []
            for a, b, c in self.sets:
                args = (ctypes.c_int(variant), ctypes.c_void_p(a.data_ptr()), ctypes.c_void_p(b.data_ptr()),
                        ctypes.c_void_p(c.data_ptr()), i64(cfg.M), i64(cfg.N), i64(cfg.K), i64(cfg.lda_),
                        i64(cfg.ldb_), i64(cfg.ldc_), i64(cfg.strideA), i64(cfg.strideB), i64(cfg.strideC),
                        i64(cfg.batch), ctypes.c_int(cfg.out_dtype), ctypes.c_void_p(stream_handle or None))
                calls.append((fn, args))
            self._calls[key] = calls
        return calls

    def launch(self, i: int, variant: int = -1, stream=None, check: bool = True) -> int:
        from . import binding as B
        if stream is None:
            handle = self.stream_handle          # torch's current stream when the problem was built
        else:
            handle = stream if isinstance(stream, int) else stream.cuda_stream
        fn, args = self._bound(variant, handle)[i % self.nsets]
        st = fn(*args)
        if check and st != 0:
            raise B.CudallmError(st, "cudallm_gemm_bf16_variant")
        return st

    def output(self, i: int = 0):
        """C of set ``i`` as a host numpy array of raw elements [batch, M, ldc-strided]."""
        import numpy as np
        import torch
        cfg = self.cfg
        torch.cuda.synchronize()
        raw = self.sets[i % self.nsets][2].cpu().numpy()
        return raw.view(np.float32 if cfg.out_dtype == 0 else np.uint16)


# ------------------------------------------------- search over the variants --

@dataclass
class ClosedFormCase:
    """A test case whose exact result is known without multiplying matrices:
    A = u p^T and B = q v^T with small integers give C = (p . q) u v^T, every
    partial sum an integer below 2**24 (exact in fp32 in any summation order)."""
    name: str
    M: int
    N: int
    K: int
    out_dtype: int
    seed: int
    lda: int | None = None
    ldb: int | None = None
    ldc: int | None = None


def default_cases(cfg=None):
    """Seeded shapes for the Function Validator: ragged small shapes that touch
    every tile edge, both output types, padded leading dimensions, and (if
    given) the configuration's own shape."""
    cases = [
        ClosedFormCase("edge-129x257x1000-f32", 129, 257, 1000, 0, 1),
        ClosedFormCase("edge-300x127x65-bf16", 300, 127, 65, 1, 2),
        ClosedFormCase("pad-257x129x129-f32", 257, 129, 129, 0, 3, lda=136, ldb=136, ldc=131),
        ClosedFormCase("odd-ld-255x300x515-f32", 255, 300, 515, 0, 4, lda=517, ldb=301, ldc=303),
        ClosedFormCase("deep-16x520x4096-f32", 16, 520, 4096, 0, 5),
        ClosedFormCase("wide-1100x700x200-bf16", 1100, 700, 200, 1, 6),
    ]
    if cfg is not None and cfg.batch == 1:
        cases.append(ClosedFormCase(f"{cfg.name}-shape", cfg.M, cfg.N, cfg.K, cfg.out_dtype, 7,
                                    cfg.lda, cfg.ldb, cfg.ldc))
    return cases


def run_closed_form_case(variant: int, case: ClosedFormCase):
    """(status, (got_bits_or_values, exact)) for ``function_validator``'s ``run``."""
    import numpy as np
    import torch
    from . import binding as B
    from . import inputs as gi
    M, N, K = case.M, case.N, case.K
    lda = K if case.lda is None else case.lda
    ldb = N if case.ldb is None else case.ldb
    ldc = N if case.ldc is None else case.ldc
    if B.variant_supports(variant, M, N, K, lda, ldb, ldc, 1, case.out_dtype) != 1:
        return "unsupported", None
    u, v, p, q = gi.rank1_int_factors(M, N, K, case.seed)
    A = gi.embed(gi.int_to_bf16_bits(np.outer(u, p)), lda)
    Bm = gi.embed(gi.int_to_bf16_bits(np.outer(q, v)), ldb)
    exact = np.outer(u, v).astype(np.float64) * float(np.dot(p, q))
    dA = torch.from_numpy(A.view(np.int16)).cuda()
    dB = torch.from_numpy(Bm.view(np.int16)).cuda()
    dt = torch.float32 if case.out_dtype == 0 else torch.bfloat16
    dC = torch.full((M * ldc,), float("nan"), dtype=dt, device="cuda")
    st = B.gemm_bf16_variant(variant, dA, dB, dC, M, N, K, lda, ldb, ldc, M * lda, K * ldb, M * ldc, 1,
                             case.out_dtype, torch.cuda.current_stream(), check=False)
    if st != 0:
        return st, None
    code, _ = B.device_status(torch.cuda.current_stream())
    if code != 0:
        return code, None
    got = dC.view(M, ldc)[:, :N].to(torch.float64).cpu().numpy()
    pad = dC.view(M, ldc)[:, N:]
    pad_ok = bool(torch.isnan(pad).all().item()) if pad.numel() else True
    return 0, (got, exact, pad_ok)


def compare_closed_form(case: ClosedFormCase, out):
    """Exact comparison: fp32 output must equal the integer result; bf16 output
    must equal it after ONE round-to-nearest-even (checked through the error
    bound |got - exact| <= half a bf16 spacing and got being a bf16 value)."""
    import numpy as np
    got, exact, pad_ok = out
    if not pad_ok:
        return False, float("inf"), "padding columns of C were overwritten"
    if case.out_dtype == 0:
        bad = got != exact
    else:
        # spacing of bf16 at |exact|: 2**(floor(log2|x|) - 7); nearest => |err| <= spacing / 2
        mag = np.maximum(np.abs(exact), 2.0 ** -126)
        half_ulp = 2.0 ** (np.floor(np.log2(mag)) - 8)
        bad = np.abs(got - exact) > half_ulp
    n_bad = int(bad.sum())
    if n_bad:
        i, j = (int(x) for x in np.argwhere(bad)[0])
        return False, float("inf"), f"{n_bad} wrong, first at ({i}, {j}): got {got[i, j]}, want {exact[i, j]}"
    return True, 0.0, ""


def knob_candidates(base: int, tiles_m: int):
    """Variant codes that add the two search knobs to ``base``: raster groups of 1, 2, 4, ... tile
    rows (while a group is smaller than the matrix), and for the tail-splitting variants the
    number of parts."""
    from . import binding as B
    out = []
    g = 1
    while g < max(2, tiles_m) and g <= 64:
        out.append(B.variant_code(base, g, 0))
        g *= 2
    if B.variant_name(base).endswith("_ts"):
        out += [B.variant_code(base, 0, t) for t in (2, 3, 6)]
    return out


def search_config(cfg, candidates=None, iters: int = 10, passes: int = 3, cases=None, knobs: bool = False,
                  top: int = 3) -> SearchResult:
    """Algorithm 1's round over the library's variants for one configuration:
    validate every candidate on seeded closed-form cases, time the valid ones
    (interleaved passes, median), keep the fastest.  With ``knobs`` a second round
    widens the candidate set around the ``top`` fastest variants: the same kernels
    with other raster-group heights and tail-split depths (variant codes), which
    are validated and timed the same way; a code replaces its plain variant only
    if it is more than 1 % faster (timing noise)."""
    import statistics
    from . import binding as B
    if candidates is None:
        candidates = [v for v in range(B.num_variants())
                      if B.variant_supports(v, cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_, cfg.batch,
                                            cfg.out_dtype) == 1 and B.variant_name(v) != "simt"]
    cases = default_cases(cfg) if cases is None else cases

    def run(v, case):
        st, out = run_closed_form_case(v, case)
        # a case the candidate cannot take does not disqualify it for other shapes
        return (0, (None, None, None)) if st == "unsupported" else (st, out)

    def compare(case, out):
        return (True, 0.0, "") if out[0] is None else compare_closed_form(case, out)

    prob = DeviceProblem(cfg)
    samples = {}
    batch = {}

    def time_round(todo):
        # every sample brackets enough back-to-back calls to last about 200 us: a short kernel is
        # then timed as a stream of launches (what a caller's pipeline sees), not as one launch
        # plus its latency
        for v in todo:
            samples[v] = []
            if v not in batch:
                est = performance_profiler(lambda i: prob.launch(i, v), iters=3, warmup=2)["median_s"]
                batch[v] = max(1, min(64, int(math.ceil(200e-6 / max(est, 1e-7)))))
        for _ in range(passes):
            for v in todo:
                t = performance_profiler(lambda i: prob.launch(i, v), iters=iters, warmup=2, batch_calls=batch[v])
                samples[v].append(t["median_s"])
        for v in todo:
            samples[v] = statistics.median(samples[v])

    res = SearchResult(best=None, best_latency=float("inf"))
    for v in candidates:
        res.reports[v] = function_validator(v, cases, run, compare)
        if res.reports[v].ok:
            res.valid.append(v)
    time_round(res.valid)
    if knobs and res.valid:
        leaders = sorted(res.valid, key=lambda v: samples[v])[:top]
        tiles_m = -(-cfg.M // 128)
        extra = [c for v in leaders for c in knob_candidates(v, tiles_m)]
        ok_extra = []
        for c in extra:
            res.reports[c] = function_validator(c, cases, run, compare)
            if res.reports[c].ok:
                ok_extra.append(c)
        time_round(ok_extra + leaders)                  # the leaders again, in the same round
        for c in ok_extra:
            if samples[c] < 0.99 * samples[c & 0xFF]:
                res.valid.append(c)
    timed = search(res.valid, lambda v: res.reports[v], lambda v: samples[v])
    timed.reports = res.reports
    return timed


class TunedTable:
    """Persisted outcome of the search: problem shape -> variant name.  Lookups
    that miss fall back to the library's own choice."""

    def __init__(self, entries=None):
        self.entries = dict(entries or {})

    @staticmethod
    def key(M, N, K, batch, out_dtype):
        return f"{M}x{N}x{K}x{batch}:{'bf16' if out_dtype == 1 else 'f32'}"

    def record(self, cfg, code, latency_s):
        """Enter the winner (a variant id or code) for the configuration's shape."""
        from . import binding as B
        g, t = (code >> 8) & 0xF, (code >> 12) & 0x7
        tma = cfg.lda_ % 8 == 0 and cfg.ldb_ % 8 == 0 and (cfg.batch == 1 or (cfg.strideA % 8 == 0 and cfg.strideB % 8 == 0))
        rec = {"variant": B.variant_name(code), "us": round(latency_s * 1e6, 2), "tma": bool(tma)}
        if g:
            rec["group"] = 1 << (g - 1)
        if t:
            rec["tail"] = t
        self.entries[self.key(cfg.M, cfg.N, cfg.K, cfg.batch, cfg.out_dtype)] = rec

    def lookup(self, M, N, K, batch, out_dtype):
        e = self.entries.get(self.key(M, N, K, batch, out_dtype))
        return None if e is None else e["variant"]

    def variant_id(self, M, N, K, batch, out_dtype, names=None):
        """Variant id for the shape, or -1 (let the library choose)."""
        name = self.lookup(M, N, K, batch, out_dtype)
        if name is None:
            return -1
        if names is None:
            from . import binding as B
            names = {B.variant_name(v): v for v in range(B.num_variants())}
        return names.get(name, -1)

    def save(self, path):
        import json
        with open(path, "w") as f:
            json.dump(self.entries, f, indent=1, sort_keys=True)

    @classmethod
    def load(cls, path):
        import json
        with open(path) as f:
            return cls(json.load(f))

    def install(self) -> int:
        """Enter every record into the library's dispatch tables (``cudallm_dispatch_set_class``: the
        record's shape stands for all shapes that are tiled like it), so that its automatic
        choice uses the searched winners; returns how many were entered (records that name a
        variant this build does not have are skipped)."""
        from . import binding as B
        names = {B.variant_name(v): v for v in range(B.num_variants())}
        n = 0
        for key, rec in self.entries.items():
            shape, dtype = key.split(":")
            M, N, K, batch = (int(x) for x in shape.split("x"))
            v = names.get(rec["variant"])
            if v is None:
                continue
            code = B.variant_code(v, rec.get("group", 0), rec.get("tail", 0))
            B.dispatch_set_class(M, N, K, batch, B.BF16 if dtype == "bf16" else B.F32, rec.get("tma", True), code)
            n += 1
        return n

    @classmethod
    def packaged(cls):
        """The table recorded on a B200 with ``--search --config all --table ...`` and shipped with
        the package (benchmark configurations and the paper's Task 2 sizes)."""
        import os
        return cls.load(os.path.join(os.path.dirname(os.path.abspath(__file__)), "tuned_b200.json"))


def search_grid():
    """Shapes beyond the benchmark configurations that the packaged table covers: M from 16 to
    8192 against eight N x K pairs (bf16 output), plus a few irregular ones."""
    from . import inputs as gi
    shapes = []
    for (N, K) in [(4096, 4096), (11008, 4096), (4096, 11008), (8192, 8192), (18944, 4096), (1024, 8192),
                   (2048, 2048), (6144, 3072)]:
        for M in (16, 128, 256, 512, 1024, 2048, 4096, 8192):
            if M * N * K <= 6e11:
                shapes.append((M, N, K))
    shapes += [(777, 3333, 1111), (1000, 1000, 1000), (5000, 5000, 512), (300, 20000, 256), (20000, 300, 2048)]
    return [gi.GemmConfig(f"G{M}x{N}x{K}", M, N, K, gi.BF16, seed=900 + i) for i, (M, N, K) in enumerate(shapes)]


def _search_one(cfg, iters, table_path, knobs=True, cases=None, passes=3):
    """Validate and time every variant on one configuration; print one JSON line per candidate
    (validation outcome: ok / mismatch / launch error / device timeout) and the winner; record
    the winner in the table file if one is given."""
    import json
    import os
    from . import binding as B

    res = search_config(cfg, iters=iters, knobs=knobs, cases=cases, passes=passes)
    for v, rep in res.reports.items():
        print(json.dumps({"config": cfg.name, "candidate": B.describe_code(v), "validation": rep.status,
                          "detail": rep.detail,
                          "us": None if v not in res.latencies else round(res.latencies[v] * 1e6, 2)}), flush=True)
    best = None if res.best is None else B.describe_code(res.best)
    choice = B.select_variant(cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_, cfg.batch, cfg.out_dtype)
    print(json.dumps({"config": cfg.name, "shape": [cfg.M, cfg.N, cfg.K, cfg.batch], "best": best,
                      "us": None if res.best is None else round(res.best_latency * 1e6, 2),
                      "library_choice": B.describe_code(choice),
                      "library_choice_us": None if choice not in res.latencies else round(res.latencies[choice] * 1e6, 2)}),
          flush=True)
    if table_path and res.best is not None:
        table = TunedTable.load(table_path) if os.path.exists(table_path) else TunedTable()
        table.record(cfg, res.best, res.best_latency)
        table.save(table_path)


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
    ladder = {f"T2-{k + 1}": gi.task2_ladder(k) for k in range(5)}     # the paper's Task 2 sizes
    all_configs = dict(gi.CONFIGS, **ladder)
    ap.add_argument("--config", default="C2", choices=sorted(all_configs) + ["all", "grid"],
                    help="a benchmark configuration, a size of the paper's Task 2 ladder, or (with --search) all of "
                         "those / the grid of other shapes that the packaged table covers")
    ap.add_argument("--no-knobs", action="store_true", help="with --search: plain variants only")
    ap.add_argument("--model-only", action="store_true",
                    help="empty the dispatch tables first, so that the cost model alone chooses")
    ap.add_argument("--variant", default="auto")
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--sets", type=int, default=None, help="rotating buffer sets (default: > L2)")
    ap.add_argument("--all-variants", action="store_true", help="time every variant that supports the shape")
    ap.add_argument("--search", action="store_true",
                    help="validate every variant on closed-form cases, time the valid ones, report the fastest")
    ap.add_argument("--table", default=None, help="with --search: JSON file to record the winner in")
    ap.add_argument("--dispatch", default=None,
                    help="a table file, or 'packaged': enter its records into the library's dispatch table first")
    ap.add_argument("--task", default=None, choices=["transpose", "sum", "dot", "layernorm", "attention", "tf32", "f32"],
                    help="time one of the other tasks (8, 14, 15, 4, 6; tf32 / f32: Task 2 with float32 operands "
                         "through cudallm_gemm_tf32 / cudallm_gemm_f32) instead of a GEMM configuration")
    ap.add_argument("--size", type=int, default=None,
                    help="with --task: N (transpose: N x N; sum, dot: N elements; layernorm: (16, 4, N, N); "
                         "attention: N queries and keys; tf32, f32: A (N x 4096) x B (4096 x 2048))")
    ap.add_argument("--layernorm-kernels", default="auto", choices=["auto", "two", "persistent"],
                    help="with --task layernorm: let the library choose by size, or force the two plain "
                         "kernels / the persistent kernel (cudallm_debug_set)")
    args = ap.parse_args(argv)
    if args.task:
        return _task_main(args)
    if args.model_only:
        B.dispatch_clear()
    if args.dispatch:
        table = TunedTable.packaged() if args.dispatch == "packaged" else TunedTable.load(args.dispatch)
        table.install()
    if args.search:
        if args.config == "grid":
            # the candidates' arithmetic does not depend on the shape: two ragged cases and the shape itself
            for cfg in search_grid():
                cases = default_cases()[:2] + [ClosedFormCase(f"{cfg.name}-shape", cfg.M, cfg.N, cfg.K, cfg.out_dtype, 7)]
                _search_one(cfg, args.iters, args.table, not args.no_knobs, cases=cases, passes=2)
            return
        for name in (sorted(all_configs) if args.config == "all" else [args.config]):
            cfg = all_configs[name]
            cases = None
            if cfg.flops > 2e12:                           # the largest ladder size: skip the shape-sized case
                cases = default_cases()
            _search_one(cfg, args.iters, args.table, not args.no_knobs, cases=cases)
        return
    if args.config in ("all", "grid"):
        ap.error("--config all / grid needs --search")
    cfg = all_configs[args.config]
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
        print(json.dumps({"config": cfg.name, "variant": B.describe_code(v), "status": code,
                          "us_min": t["min_s"] * 1e6, "us_median": t["median_s"] * 1e6,
                          "tflops": cfg.flops / t["median_s"] / 1e12,
                          "gbs": cfg.algorithmic_bytes / t["median_s"] / 1e9}), flush=True)


def task_problem(task: str, size: int, nsets: int | None = None):
    """(launch(i), algorithmic bytes per call, description) for one task on seeded device
    inputs, with enough rotating buffer sets to exceed L2 (at most 8)."""
    import torch
    from . import binding as B
    from . import inputs as gi

    st = torch.cuda.current_stream()
    if task in ("tf32", "f32"):
        # the paper's Task 2 ladder: A (size x 4096) x B (4096 x 2048), float32
        M, K, N = size, 4096, 2048
        bytes_ = 4 * (M * K + K * N + M * N)
        n = nsets or max(2, min(8, (400 << 20) // bytes_ + 1))
        gen = torch.Generator(device="cuda").manual_seed(700)
        A = [torch.randn(M, K, device="cuda", generator=gen) for _ in range(n)]
        Bm = [torch.randn(K, N, device="cuda", generator=gen) for _ in range(n)]
        C = [torch.empty(M, N, device="cuda") for _ in range(n)]
        if task == "tf32":
            return (lambda i: B.gemm_tf32(A[i % n], Bm[i % n], C[i % n], M, N, K, K, N, N, st)), bytes_, \
                f"A ({M} x {K}) x B ({K} x {N}), float32 as TF32"
        return (lambda i: B.gemm_f32(A[i % n], Bm[i % n], C[i % n], M, N, K, K, N, N, -1, st)), bytes_, \
            f"A ({M} x {K}) x B ({K} x {N}), float32 in three bf16 pieces"
    if task == "attention":
        # Task 6: the paper's (N, d_model, h) with this N, else about N columns, 32 per head
        paper = {64: (32, 4), 128: (64, 8), 256: (128, 8), 384: (256, 16), 512: (512, 16)}
        heads = max(1, size // 32)
        dm, h = paper.get(size, (32 * heads, heads))
        bytes_ = 3 * 2 * size * dm + 4 * size * dm
        n = nsets or 8
        rng = [torch.Generator(device="cuda").manual_seed(600 + i) for i in range(n)]
        Q, K, V = ([torch.randn(size, dm, device="cuda", generator=rng[i]).bfloat16() for i in range(n)]
                   for _ in range(3))
        O = [torch.empty(size, dm, device="cuda") for _ in range(n)]
        return (lambda i: B.mhsa_bf16(Q[i % n], K[i % n], V[i % n], O[i % n], size, dm, h, dm, dm, dm, dm, st)), \
            bytes_, f"N = {size}, d_model = {dm}, h = {h}"
    if task == "transpose":
        bytes_ = 8 * size * size
        n = nsets or max(1, min(8, (600 << 20) // bytes_))
        A = [torch.from_numpy(gi.task_array(8, i, size * size)).cuda() for i in range(n)]
        T = [torch.empty(size * size, device="cuda") for _ in range(n)]
        return (lambda i: B.transpose_f32(A[i % n], T[i % n], size, size, size, size, st)), bytes_, f"{size} x {size}"
    if task in ("sum", "dot"):
        per = 4 * size * (2 if task == "dot" else 1)
        n = nsets or max(1, min(8, (600 << 20) // per))
        X = [torch.from_numpy(gi.task_array(14, i, size)).cuda() for i in range(n)]
        r = torch.zeros(1, device="cuda")
        if task == "sum":
            return (lambda i: B.sum_f32(X[i % n], size, r, st)), per, f"n = {size}"
        Y = [torch.from_numpy(gi.task_array(15, i, size, "uniform")).cuda() for i in range(n)]
        return (lambda i: B.dot_f32(X[i % n], Y[i % n], size, r, st)), per, f"n = {size}"
    batch, m = 16, 4 * size * size
    bytes_ = 8 * batch * m + 8 * m
    n = nsets or max(1, min(8, (600 << 20) // bytes_))
    x, gamma, beta = gi.layernorm_inputs(4, batch, m)
    X = [torch.from_numpy(x).cuda() for _ in range(n)]
    Y = [torch.empty(batch * m, device="cuda") for _ in range(n)]
    g, b = torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda()
    return (lambda i: B.layernorm_f32(X[i % n], g, b, Y[i % n], batch, m, 1e-5, st)), bytes_, f"(16, 4, {size}, {size})"


def _task_main(args):
    import json
    import torch
    from . import binding as B

    default = {"transpose": 8192, "sum": 1 << 28, "dot": 1 << 27, "layernorm": 512, "attention": 512,
               "tf32": 1 << 14, "f32": 1 << 14}
    size = args.size or default[args.task]
    if args.task == "layernorm":
        B.debug_set(B.DEBUG_LAYERNORM_PATH, {"auto": 0, "two": 1, "persistent": 2}[args.layernorm_kernels])
    launch, bytes_, what = task_problem(args.task, size, args.sets)
    t = performance_profiler(launch, iters=args.iters, warmup=args.warmup)
    code, detail = B.device_status(torch.cuda.current_stream())
    rec = {"task": args.task, "input": what, "status": code, "us_min": t["min_s"] * 1e6,
           "us_median": t["median_s"] * 1e6, "gbs": bytes_ / t["median_s"] / 1e9}
    if args.task in ("tf32", "f32"):
        rec["tflops"] = 2.0 * size * 4096 * 2048 / t["median_s"] / 1e12
    print(json.dumps(rec), flush=True)


if __name__ == "__main__":
    _main()
