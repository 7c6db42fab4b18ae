"""The fp32-operand entry points (the element type the paper's Task 2 gives for
both factors and the product) against the fp64 oracle on float32 operands.

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


# ---------------------------------------------------------------- TF32 -----
# cudallm_gemm_tf32: the tensor cores read the float32 operands as TF32 (ten fraction bits).
# Tolerance 2.5e-3 * S (2^-9 per product of two truncated operands + float32 accumulation);
# operands with at most 11 significant bits are multiplied exactly, which pins the operand
# layout (every k-block, every 32-column box of B, both edges) bit for bit.

def run_tf32(Af, Bf, M, N, K, pad_ab=0, pad_c=0, lead=0):
    lda, ldb, ldc = K + pad_ab, N + pad_ab, N + pad_c
    A = np.full(lead + max(M * lda, 1), np.nan, dtype=np.float32)
    Bm = np.full(lead + max(K * ldb, 1), np.nan, dtype=np.float32)
    A[lead:lead + M * lda].reshape(M, lda)[:, :K] = Af
    Bm[lead:lead + K * ldb].reshape(K, ldb)[:, :N] = Bf
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(Bm).cuda()
    guard = 32
    dC = torch.full((guard + M * ldc + guard,), float("nan"), dtype=torch.float32, device="cuda")
    B.gemm_tf32(dA.data_ptr() + 4 * lead, dB.data_ptr() + 4 * lead, dC.data_ptr() + 4 * guard,
                M, N, K, lda, ldb, ldc, torch.cuda.current_stream())
    assert B.device_status(torch.cuda.current_stream()) == (B.OK, 0)
    host = dC.cpu().numpy()
    assert np.isnan(host[:guard]).all() and np.isnan(host[guard + M * ldc:]).all()
    body = host[guard: guard + M * ldc].reshape(M, ldc)
    if pad_c:
        assert np.isnan(body[:-1, N:]).all()
    return body[:, :N].astype(np.float64)


# lone CTAs up to M = 128, CTA pairs above; (100, 300, 77), (257, 513, 129) and (129, 31, 33) have
# pitches that are not multiples of 4 and take the three-piece path
TF32_SHAPES = [(128, 256, 32), (128, 256, 64), (1, 1, 1), (100, 300, 77), (257, 513, 129), (300, 260, 1000),
               (1024, 2048, 4096), (129, 31, 33), (512, 1000, 2048), (64, 512, 256), (128, 1000, 516),
               (129, 260, 36), (384, 256, 32), (256, 256, 8), (1000, 4, 4)]


@pytest.mark.parametrize("M,N,K", TF32_SHAPES)
def test_tf32_integer_operands_are_exact(M, N, K):
    """Integers of magnitude < 16 (and, on a few entries, up to 2047: eleven significant
    bits) have exact TF32 forms and exact float32 sums here, so the result must equal the
    oracle's bit for bit: a misplaced k-block, box or swizzle row would not."""
    rng = np.random.default_rng(5000 + M + N + K)
    Af = rng.integers(-15, 16, (M, K)).astype(np.float32)
    Bf = rng.integers(-15, 16, (K, N)).astype(np.float32)
    Af[rng.integers(0, M), rng.integers(0, K)] = 2047.0
    Bf[rng.integers(0, K), rng.integers(0, N)] = -1025.0
    Cref, _ = oracle.gemm_f32(Af, Bf, M, N, K)
    assert np.abs(Cref).max() < 2 ** 24
    pad = 4 if (M + N) % 2 else 0
    assert np.array_equal(run_tf32(Af, Bf, M, N, K, pad_ab=pad, pad_c=pad + 1 if pad else 0), Cref)


@pytest.mark.parametrize("M,N,K", TF32_SHAPES + [(2048, 2048, 8192)])
def test_tf32_against_oracle(M, N, K):
    rng = np.random.default_rng(5100 + M + N + K)
    Af = rng.standard_normal((M, K)).astype(np.float32)
    Bf = rng.uniform(-1, 1, (K, N)).astype(np.float32)
    got = run_tf32(Af, Bf, M, N, K)
    Cref, S = oracle.gemm_f32(Af, Bf, M, N, K)
    r = oracle.check(got, Cref, S, oracle.TOL_TF32)
    G.log_observed_error("gemm_tf32", f"{M}x{N}x{K}", r.max_scaled_err, oracle.TOL_TF32, "max |C - C_ref| / sum|a||b|")
    assert r.ok, r
    # and where the operands can be read in place it IS a reduced-precision product: some element is
    # further off than the three-piece path allows
    if K >= 64 and K % 4 == 0 and N % 4 == 0:
        assert r.max_scaled_err > oracle.TOL_F32_IN


def test_tf32_unaligned_operands_take_the_three_piece_path_and_errors():
    """Pitches that are not multiples of 4 elements (or bases off 16 bytes) cannot be read in
    place by TMA: the call is then served by cudallm_gemm_f32, to ITS tolerance."""
    rng = np.random.default_rng(5200)
    M, N, K = 130, 270, 333
    Af = rng.standard_normal((M, K)).astype(np.float32)
    Bf = rng.standard_normal((K, N)).astype(np.float32)
    Cref, S = oracle.gemm_f32(Af, Bf, M, N, K)
    for pad, lead in ((1, 0), (0, 1), (3, 1)):
        assert oracle.check(run_tf32(Af, Bf, M, N, K, pad_ab=pad, lead=lead), Cref, S, TOL).ok
    got = run_tf32(Af[:, :0], Bf[:0, :], M, N, 0)           # the empty sum
    assert np.array_equal(got, np.zeros((M, N)))
    s = torch.cuda.current_stream()
    x = torch.zeros(64, device="cuda")
    assert B.gemm_tf32(x, x, x, 4, 4, -1, 4, 4, 4, s, check=False) == B.ERR_INVALID_DIM
    assert B.gemm_tf32(x, x, x, 4, 4, 4, 3, 4, 4, s, check=False) == B.ERR_INVALID_LD
    assert B.gemm_tf32(x.data_ptr() + 2, x, x, 4, 4, 4, 4, 4, 4, s, check=False) == B.ERR_MISALIGNED
    assert B.gemm_tf32(x, x, x, 0, 4, 4, 4, 4, 4, s, check=False) == B.OK


@pytest.mark.parametrize("step", [2, 3, 4])
def test_tf32_paper_task2_ladder_closed_form(step):
    """The paper's Task 2 shapes A (size x 4096) x B (4096 x 2048), size = 2^14, 2^16 and 2^18 (4 GiB of A), as
    float32 through the TF32 kernel (CTA pairs, the last wave split along K): rank-one integer
    operands with at most 8 significant bits, every element exact."""
    cfg = gi.task2_ladder(step)
    u, v_, p, q = gi.rank1_int_factors(cfg.M, cfg.N, cfg.K, seed=60 + step)
    dA = torch.outer(torch.from_numpy(u.astype(np.float32)).cuda(), torch.from_numpy(p.astype(np.float32)).cuda())
    dB = torch.outer(torch.from_numpy(q.astype(np.float32)).cuda(), torch.from_numpy(v_.astype(np.float32)).cuda())
    dC = torch.full((cfg.M * cfg.N,), float("nan"), dtype=torch.float32, device="cuda")
    B.gemm_tf32(dA, dB, dC, cfg.M, cfg.N, cfg.K, cfg.K, cfg.N, cfg.N, torch.cuda.current_stream())
    assert B.device_status(torch.cuda.current_stream()) == (B.OK, 0)
    scale = float(np.dot(p, q))
    want = torch.outer(torch.from_numpy(u.astype(np.float32)).cuda(),
                       torch.from_numpy(v_.astype(np.float32)).cuda()) * scale      # exact in fp32
    assert torch.equal(dC.view(cfg.M, cfg.N), want)


def test_tf32_random_shapes():
    rng = np.random.default_rng(5300)
    for it in range(40):
        M = int(np.exp(rng.uniform(0, np.log(700)))); N = 4 * int(np.exp(rng.uniform(0, np.log(200))))
        K = 4 * int(np.exp(rng.uniform(0, np.log(400))))
        Af = rng.standard_normal((M, K)).astype(np.float32)
        Bf = rng.uniform(-1, 1, (K, N)).astype(np.float32)
        got = run_tf32(Af, Bf, M, N, K, pad_ab=4 * int(rng.integers(0, 3)), pad_c=int(rng.integers(0, 4)))
        Cref, S = oracle.gemm_f32(Af, Bf, M, N, K)
        r = oracle.check(got, Cref, S, oracle.TOL_TF32)
        assert r.ok, (M, N, K, r)
