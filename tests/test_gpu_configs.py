"""The benchmark configurations at full size, in the launch configuration the
benchmark times (automatic variant choice, device-resident operands).

Every configuration, C2 and C3 included, is compared with the oracle on every
element (the oracle needs a few seconds for C2 and some tens of seconds for C3
on the host cores), and against the integer rank-1 closed form, which holds at
any size.  The largest scaled error each comparison observed is appended to a
JSON-lines file beside the tests' other output, so that the margin under each
tolerance can be read off."""
import numpy as np
import pytest
import torch

import oracle
import gpu_util as G
from paper_2506_09092_b200 import binding as B
from paper_2506_09092_b200 import inputs as gi

pytestmark = pytest.mark.gpu


def _run(cfg, A, Bm, variant=B.VARIANT_AUTO):
    vals, raw, guards = G.run_config(cfg, variant, (A, Bm))
    assert guards
    return vals, raw


@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C4", "C5a", "C5b"])
def test_config_every_element(name):
    """Every element of every benchmark configuration against the oracle; the product is run
    twice and must come out bit for bit the same (fixed summation order, also where tiles
    are split along K)."""
    cfg = gi.CONFIGS[name]
    A, Bm = cfg.make()
    vals, raw = _run(cfg, A, Bm)
    _, raw2 = _run(cfg, A, Bm)
    assert np.array_equal(raw, raw2), f"{name}: two runs differ"
    del raw2
    if cfg.batch > 1:
        Cref, S = oracle.gemm_batched(A, Bm, cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_,
                                      cfg.strideA, cfg.strideB, cfg.batch)
        r = oracle.check(vals, Cref, S, G.tol_for(cfg.out_dtype))
    else:
        Cref, S = oracle.gemm(A, Bm, cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_)
        r = oracle.check(vals[0], Cref, S, G.tol_for(cfg.out_dtype))
    G.log_observed_error("gemm_bf16", name, r.max_scaled_err, G.tol_for(cfg.out_dtype),
                         "max |C - C_ref| / sum|a||b|", variant=B.variant_name(
                             B.select_variant(cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_, cfg.batch, cfg.out_dtype)))
    assert r.ok, (name, r)
    assert np.isfinite(vals).all()


@pytest.mark.parametrize("name", ["C2", "C3", "C5a", "C5b"])
def test_config_size_integer_closed_form(name):
    """A = u p^T, B = q v^T with small integers: C = (p.q) u v^T exactly, at the
    configuration's full size and strides, every element."""
    cfg = gi.CONFIGS[name]
    u, v_, p, q = gi.rank1_int_factors(cfg.M, cfg.N, cfg.K, seed=cfg.seed + 50)
    A = gi.embed(gi.int_to_bf16_bits(np.outer(u, p)), cfg.lda_)
    Bm = gi.embed(gi.int_to_bf16_bits(np.outer(q, v_)), cfg.ldb_)
    exact = np.outer(u, v_).astype(np.float64) * float(np.dot(p, q))
    vals, raw = _run(cfg, A, Bm)
    if cfg.out_dtype == gi.F32:
        assert np.array_equal(vals[0], exact)
    else:
        want = oracle.f64_to_bf16_bits(exact)
        assert ((raw[0] == want) | ((exact == 0) & (vals[0] == 0))).all()


@pytest.mark.parametrize("name,variants", [
    ("C2", ["umma2_n256", "umma_n256_ts"]),
    ("C5a", ["umma_n128_sk2", "umma_n64_sk4"]),
    ("C5b", ["umma2_n256_sk2", "umma_n128_ts"]),
])
def test_config_size_runs_are_bitwise_repeatable(name, variants):
    """Split-K and tail-split variants at full size: two runs, identical bits."""
    cfg = gi.CONFIGS[name]
    A, Bm = cfg.make()
    table = {B.variant_name(v): v for v in range(B.num_variants())}
    for vn in variants:
        _, raw = _run(cfg, A, Bm, table[vn])
        _, raw2 = _run(cfg, A, Bm, table[vn])
        assert np.array_equal(raw, raw2), (name, vn)


def test_paper_task2_ladder_first_two_sizes():
    """The paper's own Task 2 shapes (A size x 4096, B 4096 x 2048), the two
    smallest sizes, sampled rows."""
    for step in (0, 1):
        cfg = gi.task2_ladder(step)
        A, Bm = cfg.make()
        vals, _ = _run(cfg, A, Bm)
        rows = np.random.default_rng(step).choice(cfg.M, size=64, replace=False)
        Cref, S = oracle.gemm_rows(A, Bm, rows, cfg.N, cfg.K, cfg.lda_, cfg.ldb_)
        assert oracle.check(vals[0][rows], Cref, S, G.tol_for(cfg.out_dtype)).ok


@pytest.mark.parametrize("name,variants", [
    ("C2", ["umma2_n256", "umma2_n256_ts", "umma_n256_ts"]),
    ("C5b", ["umma2_n256_ts", "umma_n256_ts", "umma_n128", "umma2_n256_sk2"]),
    ("C5a", ["umma_n128", "umma_n256_sk2", "umma_n64_sk4"]),
])
def test_config_size_closed_form_on_named_variants(name, variants):
    """The tile-splitting variants at full size: tail tiles cut along N, tiles cut
    along K with in-kernel fix-up, CTA pairs.  Integer closed form, every element."""
    cfg = gi.CONFIGS[name]
    table = {B.variant_name(v): v for v in range(B.num_variants())}
    u, v_, p, q = gi.rank1_int_factors(cfg.M, cfg.N, cfg.K, seed=cfg.seed + 70)
    A = gi.embed(gi.int_to_bf16_bits(np.outer(u, p)), cfg.lda_)
    Bm = gi.embed(gi.int_to_bf16_bits(np.outer(q, v_)), cfg.ldb_)
    exact = np.outer(u, v_).astype(np.float64) * float(np.dot(p, q))
    for vn in variants:
        vals, raw = _run(cfg, A, Bm, table[vn])
        if cfg.out_dtype == gi.F32:
            assert np.array_equal(vals[0], exact), vn
        else:
            want = oracle.f64_to_bf16_bits(exact)
            assert ((raw[0] == want) | ((exact == 0) & (vals[0] == 0))).all(), vn


def test_search_finds_a_valid_fastest_variant_and_rejects_a_broken_one():
    """One round of the paper's Algorithm 1 over the library's variants on the
    small configuration: every tcgen05 variant validates, the winner is the
    fastest of them, and a candidate whose output is wrong is filtered out."""
    from paper_2506_09092_b200 import harness as H
    cfg = gi.CONFIGS["C1"]
    names = {B.variant_name(v): v for v in range(B.num_variants())}
    cands = [names[n] for n in ("umma_n64", "umma_n128", "umma_n256_sk2", "umma2_n256", "umma_n128_ts")]
    res = H.search_config(cfg, candidates=cands, iters=5, passes=2)
    assert sorted(res.valid) == sorted(cands), {B.variant_name(v): r.status for v, r in res.reports.items()}
    assert res.best in cands and res.best_latency == min(res.latencies.values())
    # the validator itself: a wrong element, or clobbered padding, is a MISMATCH
    case = H.default_cases()[2]
    st, out = H.run_closed_form_case(names["umma_n128"], case)
    assert st == 0 and H.compare_closed_form(case, out)[0]
    got, exact, pad_ok = out
    broken = got.copy(); broken[-1, -1] += 1.0                       # last row / column of an edge tile
    rep = H.function_validator(0, [case], lambda v, c: (0, (broken, exact, pad_ok)), H.compare_closed_form)
    assert rep.status == H.MISMATCH


@pytest.mark.parametrize("task,size", [("transpose", 256), ("sum", 1 << 12), ("dot", 1 << 12), ("layernorm", 64),
                                       ("attention", 64), ("attention", 200)])
def test_harness_task_commands_run(task, size, capsys):
    """The command line that the task profiles cite (`--task ... --size ...`) runs, reports a
    clean device status and a positive time."""
    import json
    from paper_2506_09092_b200 import harness as H
    H._main(["--task", task, "--size", str(size), "--iters", "2", "--warmup", "1"])
    line = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    assert line["task"] == task and line["status"] == 0 and line["us_median"] > 0
