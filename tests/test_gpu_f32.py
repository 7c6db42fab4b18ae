"""The fp32-operand entry point (the paper's Task 2 as stated: "multiplies two
matrices of 32-bit floating point numbers") against the fp64 oracle on float32
operands.

Tolerance: every element within 1e-5 * sum_k |a_ik||b_kj|.  The three-piece
split drops products of relative size <= 2^-26; fp32 accumulation of the
leading products behaves as in the bf16 path (observed 1e-7 .. 2e-6).  A lost
first-order piece product would show up at ~2^-9 / sqrt(K), above the
tolerance; the second-order ones (a2*b2, a1*b3, a3*b1) are pinned separately by
integer cases that are exact only if every one of the six products is there.
"""
import numpy as np
import pytest
import torch

import oracle
import gpu_util as G
from paper_2506_09092_b200 import binding as B
from paper_2506_09092_b200 import inputs as gi

pytestmark = pytest.mark.gpu
TOL = oracle.TOL_F32_IN
VARIANTS = ["auto", "umma_n64", "umma_n128", "umma_n256", "umma2_n256", "umma_n128_sk2",
            "umma2_n256_sk2", "umma2_n256_ts", "umma_n256_ts"]


def _names():
    return {B.variant_name(v): v for v in range(B.num_variants())}


def run_f32(Af, Bf, M, N, K, pad=0, variant=-1, lead=0, expect=B.OK):
    """Af, Bf: dense float32 operands.  Returns C (M x N float64) with NaN-filled
    padding and guard elements checked."""
    lda, ldb, ldc = K + pad, N + pad, N + pad
    A = np.full(lead + max(M * lda, 1), np.nan, dtype=np.float32)
    Bm = np.full(lead + max(K * ldb, 1), np.nan, dtype=np.float32)
    if M and K:
        A[lead:lead + M * lda].reshape(M, lda)[:, :K] = Af
    if K and N:
        Bm[lead:lead + K * ldb].reshape(K, ldb)[:, :N] = Bf
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(Bm).cuda()
    guard = 32
    dC = torch.full((guard + lead + M * ldc + guard,), float("nan"), dtype=torch.float32, device="cuda")
    st = B.gemm_f32(dA.data_ptr() + 4 * lead, dB.data_ptr() + 4 * lead, dC.data_ptr() + 4 * (guard + lead),
                    M, N, K, lda, ldb, ldc, variant, torch.cuda.current_stream(), check=False)
    assert st == expect, B.strerror(st)
    assert B.device_status(torch.cuda.current_stream()) == (B.OK, 0)
    host = dC.cpu().numpy()
    assert np.isnan(host[:guard + lead]).all() and np.isnan(host[guard + lead + M * ldc:]).all()
    body = host[guard + lead: guard + lead + M * ldc].reshape(M, ldc) if M and ldc else np.zeros((M, 0))
    if pad and M:
        assert np.isnan(body[:-1, N:]).all()              # padding columns untouched
    return body[:, :N].astype(np.float64)


def check(got, Af, Bf, M, N, K):
    Cref, S = oracle.gemm_f32(Af, Bf, M, N, K)
    r = oracle.check(got, Cref, S, TOL)
    G.log_observed_error("gemm_f32", f"{M}x{N}x{K}", r.max_scaled_err, TOL, "max |C - C_ref| / sum|a||b|")
    assert r.ok, r
    return r.max_scaled_err


@pytest.mark.parametrize("vn", VARIANTS)
def test_random_shapes_against_oracle(vn):
    names = _names()
    v = -1 if vn == "auto" else names[vn]
    rng = np.random.default_rng(11)
    for (M, N, K, pad) in [(37, 53, 29, 0), (129, 257, 1000, 3), (256, 256, 256, 0), (300, 127, 65, 1),
                           (17, 300, 129, 8), (1, 1, 1, 0), (255, 129, 640, 0)]:
        if v >= 0 and B.variant_supports(v, M, N, 6 * ((K + 63) // 64) * 64, 6 * K + 400, N, N, 1, 0) != 1:
            continue
        Af = rng.standard_normal((M, K)).astype(np.float32)
        Bf = rng.uniform(-1, 1, (K, N)).astype(np.float32)
        check(run_f32(Af, Bf, M, N, K, pad, v), Af, Bf, M, N, K)
        if pad:
            check(run_f32(Af, Bf, M, N, K, pad, v, lead=1), Af, Bf, M, N, K)   # bases only 4-byte aligned


def test_wide_dynamic_range():
    rng = np.random.default_rng(12)
    M, N, K = 200, 300, 777
    Af = (rng.standard_normal((M, K)) * np.exp(rng.uniform(-8, 8, (M, K)))).astype(np.float32)
    Bf = (rng.standard_normal((K, N)) * np.exp(rng.uniform(-8, 8, (K, N)))).astype(np.float32)
    assert check(run_f32(Af, Bf, M, N, K), Af, Bf, M, N, K) < TOL


def test_every_piece_product_is_present_integer_exact():
    """Outer products (K = 1) of integers whose product stays below 2^24: exact
    only if a1*b1, a1*b2, a2*b1, a2*b2 (12-bit x 12-bit), a3*b1 (20-bit x 4-bit)
    and a1*b3 (4-bit x 20-bit) all arrive."""
    rng = np.random.default_rng(13)
    names = _names()
    cases = [(rng.integers(1, 1 << 12, 150), rng.integers(1, 1 << 12, 200)),
             (rng.integers(1 << 16, 1 << 20, 150) | 1, rng.integers(1, 16, 200)),
             (rng.integers(1, 16, 150), rng.integers(1 << 16, 1 << 20, 200) | 1)]
    for a, b in cases:
        a = a * rng.choice([-1, 1], a.size); b = b * rng.choice([-1, 1], b.size)
        exact = np.outer(a, b).astype(np.float64)
        assert np.abs(exact).max() < (1 << 24)
        for vn in ("auto", "umma_n128", "umma2_n256"):
            got = run_f32(a.astype(np.float32)[:, None], b.astype(np.float32)[None, :], a.size, b.size, 1,
                          variant=-1 if vn == "auto" else names[vn])
            assert np.array_equal(got, exact), vn
    # and a longer integer closed form (entries up to 60: two pieces each)
    M, N, K = 300, 200, 1000
    u, v_, p, q = gi.rank1_int_factors(M, N, K, seed=5, umax=20, pmax=3)
    Af, Bf = np.outer(u, p).astype(np.float32), np.outer(q, v_).astype(np.float32)
    want = np.outer(u, v_).astype(np.float64) * float(np.dot(p, q))
    for vn in ("auto", "umma_n128_sk2", "umma2_n256_ts"):
        assert np.array_equal(run_f32(Af, Bf, M, N, K, variant=-1 if vn == "auto" else names[vn]), want), vn


def test_identity_and_bitwise_repeatability():
    rng = np.random.default_rng(14)
    n, N = 192, 260
    X = rng.standard_normal((n, N)).astype(np.float32)
    got = run_f32(np.eye(n, dtype=np.float32), X, n, N, n)
    assert np.array_equal(got, X.astype(np.float64))          # 1 * (x0 + x1 + x2) is exact
    A = rng.standard_normal((n, 500)).astype(np.float32); Bm = rng.standard_normal((500, N)).astype(np.float32)
    c0 = run_f32(A, Bm, n, N, 500); c1 = run_f32(A, Bm, n, N, 500)
    assert np.array_equal(c0, c1)


def test_degenerate_and_errors():
    Af = np.ones((4, 4), dtype=np.float32)
    got = run_f32(Af[:, :0], Af[:0, :], 4, 4, 0)               # K = 0: zeros
    assert got.shape == (4, 4) and not got.any()
    run_f32(Af[:0], Af, 0, 4, 4)
    run_f32(Af, Af[:, :0], 4, 0, 4)
    p = torch.zeros(64, dtype=torch.float32, device="cuda")
    f = lambda *a: B.gemm_f32(*a, check=False)
    assert f(p.data_ptr() + 2, p, p, 4, 4, 4, 4, 4, 4) == B.ERR_MISALIGNED
    assert f(p, p, p, 4, 4, 4, 3, 4, 4) == B.ERR_INVALID_LD
    assert f(p, p, p, 4, 4, 4, 4, 4, 4, 0) == B.ERR_INVALID_VARIANT        # the simt variant is bf16 only
    assert f(None, p, p, 4, 4, 4, 4, 4, 4) == B.ERR_INVALID_POINTER


def test_paper_task2_ladder_fp32_sampled_rows():
    """The paper's own Task 2 shapes, float32, sizes 2^10 and 2^12 rows."""
    for step in (0, 1):
        cfg = gi.task2_ladder(step)
        rng = np.random.default_rng([cfg.seed, 3])
        Af = rng.standard_normal((cfg.M, cfg.K), dtype=np.float32)
        Bf = rng.standard_normal((cfg.K, cfg.N), dtype=np.float32)
        got = run_f32(Af, Bf, cfg.M, cfg.N, cfg.K)
        rows = np.sort(rng.choice(cfg.M, size=48, replace=False))
        Cref, S = oracle.gemm_f32_rows(Af, Bf, rows, cfg.N, cfg.K)
        assert oracle.check(got[rows], Cref, S, TOL).ok
        assert np.isfinite(got).all()
