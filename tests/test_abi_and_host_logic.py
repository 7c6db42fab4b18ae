"""CPU-only checks of the C ABI: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching CUDA; plus the
host-side variant table, selection and the search loop."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2506_09092_b200 import binding as B
from paper_2506_09092_b200 import build as libbuild
from paper_2506_09092_b200 import harness as H
from paper_2506_09092_b200 import inputs as gi

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    libbuild.build()


def header_symbols():
    import glob
    syms = set()
    for h in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))):
        text = re.sub(r"/\*.*?\*/", "", open(h).read(), flags=re.S)
        syms |= set(re.findall(r"\b(cudallm_[a-z0-9_]+)\s*\(", text))
    return sorted(syms)


def test_library_exports_every_declared_symbol():
    syms = header_symbols()
    assert len(syms) >= 21
    L = ctypes.CDLL(B.LIB_PATH)
    for s in syms:
        assert hasattr(L, s), s
    assert sorted(B.SIGNATURES) == syms          # the binding covers the same set


def test_version_and_variant_table():
    assert B.version() >= 100
    n = B.num_variants()
    names = [B.variant_name(v) for v in range(n)]
    assert names[0] == "simt" and len(set(names)) == n
    assert B.variant_name(n) is None and B.variant_name(-1) is None
    assert any(nm.startswith("umma_n256") for nm in names)


def test_argument_errors_are_reported_before_any_cuda_call():
    p = 4096            # a non-null, aligned stand-in address; never dereferenced on error
    g = lambda *a, **k: B.gemm_bf16(*a, check=False, **k)
    assert g(None, p, p, 4, 4, 4, 4, 4, 4, 0) == B.ERR_INVALID_POINTER
    assert g(p, None, p, 4, 4, 4, 4, 4, 4, 0) == B.ERR_INVALID_POINTER
    assert g(p, p, None, 4, 4, 4, 4, 4, 4, 0) == B.ERR_INVALID_POINTER
    assert g(p, p, p, -1, 4, 4, 4, 4, 4, 0) == B.ERR_INVALID_DIM
    assert g(p, p, p, 4, 4, 1 << 40, 1 << 40, 4, 4, 0) == B.ERR_INVALID_DIM
    assert g(p, p, p, 4, 4, 4, 3, 4, 4, 0) == B.ERR_INVALID_LD
    assert g(p, p, p, 4, 4, 4, 4, 3, 4, 0) == B.ERR_INVALID_LD
    assert g(p, p, p, 4, 4, 4, 4, 4, 3, 0) == B.ERR_INVALID_LD
    assert g(p, p, p, 4, 4, 4, 4, 4, 4, 2) == B.ERR_INVALID_DTYPE
    assert g(p + 1, p, p, 4, 4, 4, 4, 4, 4, 0) == B.ERR_MISALIGNED
    assert g(p, p, p + 2, 4, 4, 4, 4, 4, 4, 0) == B.ERR_MISALIGNED     # fp32 C needs 4 bytes
    # empty problems succeed without a device, even with null pointers
    assert g(None, None, None, 0, 4, 4, 4, 4, 4, 0) == B.OK
    assert g(None, None, None, 4, 0, 4, 4, 0, 0, 1) == B.OK
    # batched: overlapping items of C are refused
    st = B.gemm_bf16_batched(p, p, p, 4, 4, 4, 4, 4, 4, 16, 16, 15, 2, 0, check=False)
    assert st == B.ERR_INVALID_LD
    assert B.gemm_bf16_batched(p, p, p, 4, 4, 4, 4, 4, 4, 16, 16, 16, 0, 0, check=False) == B.OK
    st = B.gemm_bf16_variant(999, p, p, p, 4, 4, 4, 4, 4, 4, 16, 16, 16, 1, 0, check=False)
    assert st == B.ERR_INVALID_VARIANT
    assert "leading dimension" in B.strerror(B.ERR_INVALID_LD)
    assert B.strerror(12345) == "unknown status"


def test_fp32_entry_point_validates_first():
    p = 4096
    f = lambda *a: B.gemm_f32(*a, check=False)
    assert f(None, p, p, 4, 4, 4, 4, 4, 4) == B.ERR_INVALID_POINTER
    assert f(p, p, p, 4, 4, 4, 3, 4, 4) == B.ERR_INVALID_LD
    assert f(p + 2, p, p, 4, 4, 4, 4, 4, 4) == B.ERR_MISALIGNED
    assert f(p, p, p + 2, 4, 4, 4, 4, 4, 4) == B.ERR_MISALIGNED
    assert f(p, p, p, 4, 4, 4, 4, 4, 4, 0) == B.ERR_INVALID_VARIANT      # simt: bf16 operands only
    assert f(p, p, p, 4, 4, 4, 4, 4, 4, 999) == B.ERR_INVALID_VARIANT
    assert f(p, p, p, 4, 4, 1 << 30, 1 << 30, 4, 4) == B.ERR_INVALID_DIM  # 6 K must stay indexable
    assert f(None, None, None, 0, 4, 4, 4, 4, 4) == B.OK


def test_tf32_entry_point_and_debug_hooks_validate_first():
    p = 4096
    f = lambda *a: B.gemm_tf32(*a, check=False)
    assert f(None, p, p, 4, 4, 4, 4, 4, 4) == B.ERR_INVALID_POINTER
    assert f(p, p, p, 4, 4, 4, 3, 4, 4) == B.ERR_INVALID_LD
    assert f(p, p, p, 4, -4, 4, 4, 4, 4) == B.ERR_INVALID_DIM
    assert f(p + 2, p, p, 4, 4, 4, 4, 4, 4) == B.ERR_MISALIGNED
    assert f(p, p, p + 2, 4, 4, 4, 4, 4, 4) == B.ERR_MISALIGNED
    assert f(None, None, None, 0, 4, 4, 4, 4, 4) == B.OK
    # the hooks are host-side switches: unknown ones and values out of range are refused
    assert B.debug_set(B.DEBUG_LAYERNORM_PATH, 3, check=False) == B.ERR_INVALID_VARIANT
    assert B.debug_set(B.DEBUG_LAYERNORM_PATH, 0, check=False) == B.OK
    assert B.debug_set(99, 0, check=False) == B.ERR_INVALID_VARIANT


def test_attention_entry_point_validates_first():
    p = 4096
    f = lambda *a: B.mhsa_bf16(*a, check=False)
    assert f(p, p, p, p, -1, 32, 4, 32, 32, 32, 32) == B.ERR_INVALID_DIM
    assert f(p, p, p, p, 64, 32, 3, 32, 32, 32, 32) == B.ERR_INVALID_DIM          # h must divide d_model
    assert f(p, p, p, p, 64, 32, 4, 32, 31, 32, 32) == B.ERR_INVALID_LD
    assert f(p, None, p, p, 64, 32, 4, 32, 32, 32, 32) == B.ERR_INVALID_POINTER
    assert f(p, p, p, p + 2, 64, 32, 4, 32, 32, 32, 32) == B.ERR_MISALIGNED
    assert f(p, p, p, p, 1 << 31, 32, 4, 32, 32, 32, 32) == B.ERR_INVALID_DIM      # any sequence length below 2^31 - 1024
    assert f(p, p, p, p, 64, 160, 4, 160, 160, 160, 160) == B.ERR_UNSUPPORTED_SHAPE  # d_k = 40
    assert f(p + 2, p, p, p, 64, 32, 4, 32, 32, 32, 32) == B.ERR_UNSUPPORTED_SHAPE  # Q not 16-byte aligned
    assert f(None, None, None, None, 0, 32, 4, 32, 32, 32, 32) == B.OK


def test_host_entry_point_validates_first():
    p = 4096
    assert B.gemm_bf16_host(None, p, p, 4, 4, 4, 4, 4, 4, 0, p, 1 << 20, check=False) == B.ERR_INVALID_POINTER
    assert B.gemm_bf16_host(p, p, p, 4, 4, 4, 4, 4, 4, 0, None, 0, check=False) == B.ERR_WORKSPACE
    need = B.host_staging_bytes(4, 4, 4, 4, 4, 4, 0)
    assert need == 3 * 256
    assert B.gemm_bf16_host(p, p, p, 4, 4, 4, 4, 4, 4, 0, p, need - 1, check=False) == B.ERR_WORKSPACE


def test_variant_support_rules():
    table = {B.variant_name(v): v for v in range(B.num_variants())}
    # split-K needs at least one 64-deep k-block per split
    assert B.variant_supports(table["umma_n64_sk16"], 128, 128, 64, 64, 128, 128, 1, 0) == 0
    assert B.variant_supports(table["umma2_n256_sk4"], 512, 512, 128, 128, 512, 512, 1, 0) == 0
    assert B.variant_supports(table["umma2_n256_ts"], 512, 512, 128, 128, 512, 512, 1, 0) == 1
    assert B.variant_supports(table["umma_n64_sk16"], 128, 128, 1024, 1024, 128, 128, 1, 0) == 1
    assert B.variant_supports(table["simt"], 1, 1, 0, 0, 1, 1, 1, 0) == 1
    assert B.variant_supports(table["umma_n128"], 1, 1, 0, 0, 1, 1, 1, 0) == 0      # K == 0
    assert B.variant_supports(-3, 1, 1, 1, 1, 1, 1, 1, 0) == B.ERR_INVALID_VARIANT
    assert B.variant_supports(0, 4, 4, 4, 3, 4, 4, 1, 0) == B.ERR_INVALID_LD


def test_selection_and_workspace_queries():
    for cfg in gi.CONFIGS.values():
        v = B.select_variant(cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_, cfg.batch, cfg.out_dtype)
        assert 0 < (v & 0xFF) < B.num_variants() and B.variant_name(v) is not None      # an id or a code
        assert B.variant_supports(v, cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_, cfg.batch,
                                  cfg.out_dtype) == 1
        ws = B.workspace_bytes(cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_, cfg.batch, cfg.out_dtype)
        assert ws >= 256 and ws % 256 == 0
    c2 = gi.CONFIGS["C2"]
    # the large square problem goes to 256-wide tiles (CTA pairs), never to plain split-K
    name = B.variant_name(B.select_variant(c2.M, c2.N, c2.K, c2.K, c2.N, c2.N, 1, 1))
    assert "n256" in name and "_sk" not in name
    assert B.select_variant(4, 4, 0, 0, 4, 4, 1, 0) == 0          # K == 0 runs on the simt kernel


# ------------------------------------------------------------ search loop ----

class _Case:
    def __init__(self, name):
        self.name = name


def test_search_keeps_fastest_valid_candidate():
    lat = {0: 5.0, 1: 1.0, 2: 2.0, 3: 0.5}
    broken = {1: H.MISMATCH, 3: H.LAUNCH_FAIL}

    def validate(k):
        return H.ValidationReport(broken.get(k, H.OK))

    res = H.search([0, 1, 2, 3], validate, lambda k: lat[k])
    assert res.valid == [0, 2] and res.best == 2 and res.best_latency == 2.0
    assert res.reports[1].status == H.MISMATCH and 3 not in res.latencies


def test_search_with_no_valid_candidate_reports_failure_and_terminates():
    res = H.search([0, 1], lambda k: H.ValidationReport(H.MISMATCH), lambda k: 1.0)
    assert res.best is None and res.best_latency == float("inf") and res.valid == []


def test_search_tie_keeps_earlier_candidate():
    res = H.search([4, 2], lambda k: H.ValidationReport(H.OK), lambda k: 1.0)
    assert res.best == 4


def test_function_validator_failure_classes():
    cases = [_Case("a"), _Case("b"), _Case("c")]
    good = lambda k, c: (0, 1.0)
    cmp_ok = lambda c, out: (True, 1e-6, "")
    assert H.function_validator(0, cases, good, cmp_ok).status == H.OK
    rep = H.function_validator(0, cases, lambda k, c: (-8, None) if c.name == "b" else (0, 1.0), cmp_ok)
    assert rep.status == H.LAUNCH_FAIL and rep.failed_case == "b" and rep.cases == 1
    rep = H.function_validator(0, cases, lambda k, c: (-9, None), cmp_ok)
    assert rep.status == H.TIMEOUT
    rep = H.function_validator(0, cases, lambda k, c: ("unsupported", None), cmp_ok)
    assert rep.status == H.UNSUPPORTED
    rep = H.function_validator(0, cases, good, lambda c, out: (c.name != "c", 0.5, "edge column stale"))
    assert rep.status == H.MISMATCH and rep.failed_case == "c" and rep.detail == "edge column stale"


def test_tuned_table_roundtrip(tmp_path):
    names = {B.variant_name(v): v for v in range(B.num_variants())}
    t = H.TunedTable()
    t.record(gi.CONFIGS["C2"], B.variant_code(names["umma2_n256_ts"], 4, 3), 98.7e-6)
    t.record(gi.CONFIGS["C4"], names["umma_n128"], 14.4e-6)
    t.record(gi.CONFIGS["C5b"], names["umma2_n256"], 70e-6)
    path = tmp_path / "tuned.json"
    t.save(path)
    u = H.TunedTable.load(path)
    assert u.entries[H.TunedTable.key(4096, 4096, 4096, 1, 1)] == {"variant": "umma2_n256_ts", "us": 98.7, "tma": True,
                                                                  "group": 4, "tail": 3}
    assert u.entries[H.TunedTable.key(3001, 1999, 5003, 1, 0)]["tma"] is False     # odd pitches
    assert u.lookup(4096, 4096, 4096, 1, 1) == "umma2_n256_ts"
    assert u.lookup(4096, 4096, 4096, 1, 0) is None            # other output type: not tuned
    assert u.variant_id(128, 128, 64, 512, 0, names) == names["umma_n128"]
    assert u.variant_id(1, 2, 3, 1, 0, names) == -1            # miss: the library chooses
    u.entries[H.TunedTable.key(5, 5, 5, 1, 0)] = {"variant": "no_such_kernel", "us": 1.0}
    assert u.variant_id(5, 5, 5, 1, 0, names) == -1


def test_closed_form_comparison_rules():
    case = H.ClosedFormCase("t", 2, 2, 4, 0, 0)
    exact = np.array([[3.0, -8.0], [0.0, 257.0]])
    assert H.compare_closed_form(case, (exact.copy(), exact, True))[0]
    off = exact.copy(); off[1, 1] += 1
    ok, _, detail = H.compare_closed_form(case, (off, exact, True))
    assert not ok and "(1, 1)" in detail
    assert not H.compare_closed_form(case, (exact.copy(), exact, False))[0]     # padding clobbered
    bf = H.ClosedFormCase("t", 2, 2, 4, 1, 0)
    rounded = exact.copy(); rounded[1, 1] = 256.0               # 257 -> 256 (tie to even)
    assert H.compare_closed_form(bf, (rounded, exact, True))[0]
    trunc = exact.copy(); trunc[1, 1] = 254.0                   # more than half a spacing away
    assert not H.compare_closed_form(bf, (trunc, exact, True))[0]


def test_packaged_tuned_table_names_existing_variants():
    """The dispatch table recorded by the search on a B200 covers the benchmark configurations
    and names only variants the library has and that support the shape."""
    table = H.TunedTable.packaged()
    names = {B.variant_name(v): v for v in range(B.num_variants())}
    for cfg in gi.CONFIGS.values():
        name = table.lookup(cfg.M, cfg.N, cfg.K, cfg.batch, cfg.out_dtype)
        assert name in names, (cfg.name, name)
        assert B.variant_supports(names[name], cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_, cfg.batch,
                                  cfg.out_dtype) == 1
        assert table.variant_id(cfg.M, cfg.N, cfg.K, cfg.batch, cfg.out_dtype) == names[name]
    assert table.lookup(7, 7, 7, 1, 0) is None and table.variant_id(7, 7, 7, 1, 0) == -1


def test_dispatch_table_overrides_the_cost_model_for_its_shapes():
    """An entry of the dispatch table is what the automatic choice returns for that shape
    (and only that shape); an entry whose variant cannot run the shape is ignored; removing
    or clearing restores the cost model's answer.  Host logic only: no GPU needed."""
    names = {B.variant_name(v): v for v in range(B.num_variants())}
    shape = (4096, 4096, 4096)
    args = shape + (4096, 4096, 4096, 1, B.BF16)           # M, N, K, lda, ldb, ldc, batch, dtype
    assert B.dispatch_clear() >= 0
    try:
        model = B.select_variant(*args)
        other = names["umma_n128"] if model != names["umma_n128"] else names["umma_n256"]
        assert B.dispatch_get(*shape, 1, B.BF16) == -1
        B.dispatch_set(*shape, 1, B.BF16, other)
        assert B.dispatch_get(*shape, 1, B.BF16) == other
        assert B.select_variant(*args) == other
        f32_model = B.select_variant(*shape, 4096, 4096, 4096, 1, B.F32)
        B.dispatch_set(*shape, 1, B.BF16, other)                 # (again: replaces)
        assert B.select_variant(*shape, 4096, 4096, 4096, 1, B.F32) == f32_model      # another key: the model
        B.dispatch_set(*shape, 1, B.BF16, -1)
        assert B.select_variant(*args) == model
        # a variant that cannot run the shape (16 K-parts of a single k-block) is not used
        small = (256, 256, 64)
        small_model = B.select_variant(*small, 64, 256, 256, 1, B.F32)
        B.dispatch_set(*small, 1, B.F32, names["umma_n64_sk16"])
        assert B.variant_supports(names["umma_n64_sk16"], *small, 64, 256, 256, 1, B.F32) == 0
        assert B.select_variant(*small, 64, 256, 256, 1, B.F32) == small_model
        assert B.dispatch_clear() == 1
        # argument errors
        assert B.dispatch_set(-1, 1, 1, 1, B.F32, 1, check=False) == B.ERR_INVALID_DIM
        assert B.dispatch_set(1, 1, 1, 1, 7, 1, check=False) == B.ERR_INVALID_DTYPE
        assert B.dispatch_set(1, 1, 1, 1, B.F32, B.num_variants(), check=False) == B.ERR_INVALID_VARIANT
        assert B.dispatch_set(1, 1, 1, 1, B.F32, -2, check=False) == B.ERR_INVALID_VARIANT
    finally:
        B.dispatch_clear()
        B.dispatch_load_packaged()


def test_variant_codes_carry_the_search_knobs():
    names = {B.variant_name(v): v for v in range(B.num_variants())}
    ts, plain = names["umma2_n256_ts"], names["umma_n128"]
    assert B.variant_code(ts) == ts and B.describe_code(ts) == "umma2_n256_ts"
    code = B.variant_code(ts, 8, 3)
    assert code != ts and code & 0xFF == ts and B.variant_name(code) == "umma2_n256_ts"
    assert B.describe_code(code) == "umma2_n256_ts+g8+t3"
    assert B.variant_supports(code, 4096, 4096, 4096, 4096, 4096, 4096, 1, B.BF16) == 1
    assert B.variant_code(plain, 0, 3, check=False) == B.ERR_INVALID_VARIANT      # not a tail-splitting variant
    assert B.variant_code(plain, 3, 0, check=False) == B.ERR_INVALID_VARIANT      # not a power of two
    assert B.variant_code(ts, 0, 8, check=False) == B.ERR_INVALID_VARIANT
    assert B.variant_code(99, 0, 0, check=False) == B.ERR_INVALID_VARIANT
    assert B.variant_name(1 << 20) is None
    p = 4096
    assert B.gemm_bf16_variant(1 << 20, p, p, p, 4, 4, 4, 4, 4, 4, 16, 16, 16, 1, 0, check=False) == B.ERR_INVALID_VARIANT
    # the two arrangements of the shared-memory ring are separate candidates
    for n in ("umma_n128_k1", "umma_n256_k2", "umma2_n256_k1", "umma2_n256_k1_ts"):
        assert n in names


def test_class_entries_cover_every_shape_that_is_tiled_alike():
    """A class entry recorded for one shape is used for every shape with the same tile and
    k-block counts (and only those); the exact-shape table wins over it; shapes whose operands
    TMA cannot address form classes of their own."""
    names = {B.variant_name(v): v for v in range(B.num_variants())}
    try:
        B.dispatch_clear()
        model = B.select_variant(4000, 4090, 4050, 4056, 4096, 4096, 1, B.BF16)
        code = B.variant_code(names["umma_n128_ts"] if model != names["umma_n128_ts"] else names["umma_n256_ts"], 2, 3)
        B.dispatch_set_class(4096, 4096, 4096, 1, B.BF16, True, code)
        assert B.dispatch_get_class(3969, 4033, 4090, 1, B.BF16, True) == code       # same ceilings
        assert B.select_variant(4096, 4096, 4096, 4096, 4096, 4096, 1, B.BF16) == code
        assert B.select_variant(4000, 4090, 4050, 4056, 4096, 4096, 1, B.BF16) == code
        assert B.select_variant(4000, 4090, 4050, 4051, 4096, 4096, 1, B.BF16) != code    # lda odd: another class
        assert B.select_variant(4096, 4096, 4097, 4104, 4096, 4096, 1, B.BF16) != code    # one more k-block
        assert B.select_variant(4096, 4096, 4096, 4096, 4096, 4096, 1, B.F32) != code     # other output type
        exact = names["umma2_n256"]
        B.dispatch_set(4000, 4090, 4050, 1, B.BF16, exact)
        assert B.select_variant(4000, 4090, 4050, 4056, 4096, 4096, 1, B.BF16) == exact
        assert B.select_variant(4096, 4096, 4096, 4096, 4096, 4096, 1, B.BF16) == code
        # short-A buckets are classes of their own
        B.dispatch_set_class(16, 4096, 4096, 1, B.F32, True, names["umma_n128_sk2"])
        assert B.dispatch_get_class(9, 4096, 4096, 1, B.F32, True) == names["umma_n128_sk2"]
        assert B.dispatch_get_class(17, 4096, 4096, 1, B.F32, True) == -1
        assert B.dispatch_set_class(16, 4096, 4096, 1, B.F32, True, -1) == B.OK
        assert B.dispatch_get_class(9, 4096, 4096, 1, B.F32, True) == -1
        assert B.dispatch_clear() == 2
    finally:
        B.dispatch_clear()
        B.dispatch_load_packaged()


def test_library_starts_with_the_packaged_winners():
    """The packaged table is compiled into the library and entered at first use; clearing
    removes it, cudallm_dispatch_load_packaged brings it back."""
    table = H.TunedTable.packaged()
    names = {B.variant_name(v): v for v in range(B.num_variants())}
    try:
        B.dispatch_clear()
        assert B.dispatch_load_packaged() == len(table.entries)
        for key, rec in table.entries.items():
            shape, dtype = key.split(":")
            M, N, K, batch = (int(x) for x in shape.split("x"))
            dt = B.BF16 if dtype == "bf16" else B.F32
            code = B.variant_code(names[rec["variant"]], rec.get("group", 0), rec.get("tail", 0))
            assert B.dispatch_get_class(M, N, K, batch, dt, rec.get("tma", True)) == code, key
        B.dispatch_clear()
        assert table.install() == len(table.entries)                     # the same through the Python table
        for key, rec in table.entries.items():
            shape, dtype = key.split(":")
            M, N, K, batch = (int(x) for x in shape.split("x"))
            dt = B.BF16 if dtype == "bf16" else B.F32
            assert B.variant_name(B.dispatch_get_class(M, N, K, batch, dt, rec.get("tma", True))) == rec["variant"]
    finally:
        B.dispatch_clear()
        B.dispatch_load_packaged()
