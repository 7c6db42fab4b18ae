"""Parity of the CUDA library against the CPU oracle, through the C ABI.

Floating-point bar (from the target statement): every element within
1e-3 * sum_k |a_ik||b_kj| (fp32 output) or 1e-2 * the same (bf16 output) of
the fp64 oracle.  Integer-valued closed-form cases must be bit-exact.
"""
import numpy as np
import pytest
import torch

import oracle
import gpu_util as G
from paper_2506_09092_b200 import binding as B
from paper_2506_09092_b200 import inputs as gi

pytestmark = pytest.mark.gpu

DIMS = [1, 15, 16, 17, 127, 128, 129, 255, 256, 257, 300]
KS = [1, 15, 16, 17, 63, 64, 65, 129, 1000]


def bits(x):
    return gi.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def variant_ids(*names):
    table = {B.variant_name(v): v for v in range(B.num_variants())}
    return [table[n] for n in names if n in table]


def check_case(A, Bm, M, N, K, out_dtype, variant, lda=None, ldb=None, ldc=None, ref=None, **kw):
    lda = K if lda is None else lda
    ldb = N if ldb is None else ldb
    ldc = N if ldc is None else ldc
    vals, raw, guards = G.run_gemm(A, Bm, M, N, K, lda, ldb, ldc, out_dtype, variant=variant, **kw)
    Cref, S = ref if ref is not None else oracle.gemm(A, Bm, M, N, K, lda, ldb)
    r = oracle.check(vals[0], Cref, S, G.tol_for(out_dtype))
    assert guards, f"guard band or padding overwritten ({B.variant_name(variant)})"
    assert r.ok, (f"{B.variant_name(variant)} M={M} N={N} K={K} out={out_dtype}: {r.n_bad} bad, "
                  f"max scaled err {r.max_scaled_err:.3e} at {r.argmax}")
    return vals, raw


# ----------------------------------------------------- validation shape set --

@pytest.mark.parametrize("M", DIMS)
def test_shape_grid(M):
    """Every (N, K) of the grid, both output types, on the automatic choice, the CUDA-core
    kernel and every listed tcgen05 variant that supports the shape (one per tile width and
    ring arrangement, lone CTAs and pairs, two CTAs per SM, split-K and tail-split ones)."""
    rng = np.random.default_rng(1000 + M)
    names = ["simt", "umma_n64", "umma_n128", "umma_n256", "umma_n64_sk2", "umma_n256_sk4",
             "umma2_n256", "umma2_n256_sk2", "umma_n256_ts", "umma2_n256_ts", "umma_n64_x2", "umma_n128_x2",
             "umma_n128_k1", "umma_n256_k2_ts", "umma2_n256_k1", "umma2_n256_k1_ts"]
    ids = variant_ids(*names)
    for N in DIMS:
        for K in KS:
            A = bits(rng.standard_normal((M, K)))
            Bm = bits(rng.uniform(-1, 1, (K, N)))
            ref = oracle.gemm(A, Bm, M, N, K)
            for out_dtype in (gi.F32, gi.BF16):
                for v in [B.VARIANT_AUTO] + [v for v in ids if B.variant_supports(v, M, N, K, K, N, N, 1, out_dtype) == 1]:
                    check_case(A.ravel(), Bm.ravel(), M, N, K, out_dtype, v, ref=ref)


@pytest.mark.parametrize("pad", [1, 3, 8])
@pytest.mark.parametrize("out_dtype", [gi.F32, gi.BF16])
def test_padded_leading_dimensions_and_offset_bases(pad, out_dtype):
    rng = np.random.default_rng(77 + pad)
    for (M, N, K) in [(129, 257, 65), (300, 127, 1000), (17, 300, 129), (256, 256, 64)]:
        A = bits(rng.standard_normal((M, K)))
        Bm = bits(rng.standard_normal((K, N)))
        ref = oracle.gemm(A, Bm, M, N, K)
        lda, ldb, ldc = K + pad, N + pad, N + pad
        Ap, Bp = gi.embed(A, lda), gi.embed(Bm, ldb)       # NaN padding: reading it poisons C
        ids = variant_ids("simt", "umma_n128", "umma_n256_sk2", "umma2_n256", "umma2_n256_ts", "umma_n256_k2",
                          "umma2_n256_k1_ts")
        # the same kernels with the search's knobs set: raster groups of one or two tile rows,
        # the ragged last wave cut into up to two or six parts
        ts = variant_ids("umma2_n256_ts", "umma_n128_ts")
        codes = [B.variant_code(ts[0], 1, 2), B.variant_code(ts[1], 2, 6), B.variant_code(ids[1], 1, 0)]
        for v in [B.VARIANT_AUTO] + ids + codes:
            if v >= 0 and B.variant_supports(v, M, N, K, lda, ldb, ldc, 1, out_dtype) != 1:
                continue
            check_case(Ap, Bp, M, N, K, out_dtype, v, lda, ldb, ldc, ref=ref)
            # base pointers offset by one element (2-byte aligned only)
            check_case(Ap, Bp, M, N, K, out_dtype, v, lda, ldb, ldc, ref=ref,
                       lead_a=1, lead_b=1, lead_c=1)


def test_random_shapes():
    rng = np.random.default_rng(1234)
    for it in range(200):
        M = int(np.exp(rng.uniform(0, np.log(600))))
        N = int(np.exp(rng.uniform(0, np.log(600))))
        K = int(np.exp(rng.uniform(0, np.log(1100))))
        out_dtype = int(rng.integers(0, 2))
        A = bits(rng.standard_normal((M, K)))
        Bm = bits(rng.standard_normal((K, N)))
        ref = oracle.gemm(A, Bm, M, N, K)
        vs = G.supported_variants(M, N, K, K, N, N, 1, out_dtype)
        v = vs[int(rng.integers(0, len(vs)))] if it % 2 else B.VARIANT_AUTO
        check_case(A.ravel(), Bm.ravel(), M, N, K, out_dtype, v, ref=ref)


@pytest.mark.parametrize("batch", [1, 3, 512])
@pytest.mark.parametrize("out_dtype", [gi.F32, gi.BF16])
def test_batched(batch, out_dtype):
    rng = np.random.default_rng(batch)
    for (M, N, K, pad) in [(128, 128, 64, 0), (50, 70, 33, 0), (128, 128, 64, 8), (33, 65, 100, 3)]:
        if batch == 512 and (M, N, K) == (33, 65, 100):
            continue
        lda, ldb, ldc = K + pad, N + pad, N + pad
        sA, sB, sC = M * lda + pad, K * ldb + pad, M * ldc + 2 * pad
        cfgA = gi.random_operand(batch * 7 + M, 0, M, K, lda, batch=batch, stride=sA)
        cfgB = gi.random_operand(batch * 7 + M, 1, K, N, ldb, batch=batch, stride=sB)
        Cref, S = oracle.gemm_batched(cfgA, cfgB, M, N, K, lda, ldb, sA, sB, batch)
        for v in [B.VARIANT_AUTO] + variant_ids("simt", "umma_n64", "umma_n128", "umma_n128_sk2", "umma2_n256",
                                                "umma2_n256_sk2", "umma_n128_ts", "umma2_n256_ts", "umma_n64_x2",
                                                "umma_n128_x2"):
            if v >= 0 and B.variant_supports(v, M, N, K, lda, ldb, ldc, batch, out_dtype) != 1:
                continue
            vals, raw, guards = G.run_gemm(cfgA, cfgB, M, N, K, lda, ldb, ldc, out_dtype, batch,
                                           sA, sB, sC, variant=v)
            r = oracle.check(vals, Cref, S, G.tol_for(out_dtype))
            assert guards and r.ok, (B.variant_name(v), M, N, K, batch, r)


@pytest.mark.parametrize("out_dtype", [gi.F32, gi.BF16])
def test_aligned_c_with_ragged_edges(out_dtype):
    """C aligned for 16-byte row stores (the epilogue's TMA path) while N and M
    end inside a 32 x 32 store box: N a multiple of the 16-byte granule or not,
    N just past a box boundary, M ragged, batch items with padded strides.
    The padding columns, the rows below M and the guard bands must stay intact."""
    rng = np.random.default_rng(4242)
    g = 4 if out_dtype == gi.F32 else 8                    # elements per 16 bytes
    cases = [(300, 127, 200, 128, 1), (300, 124, 64, 128, 1), (45, 33, 64, 40, 1), (129, 258, 130, 264, 1),
             (256, 257, 64, 272, 1), (70, 100, 96, 104, 3), (128, 120, 64, 128, 5), (31, 8, 16, 8, 2)]
    for (M, N, K, ldc, batch) in cases:
        assert ldc % g == 0
        sA, sB, sC = M * K, K * N, M * ldc + 3 * g
        A = gi.random_operand(M + N, 0, M, K, K, batch=batch, stride=sA)
        Bm = gi.random_operand(M + N, 1, K, N, N, batch=batch, stride=sB)
        Cref, S = oracle.gemm_batched(A, Bm, M, N, K, K, N, sA, sB, batch)
        names = ("umma_n64", "umma_n128", "umma_n256", "umma_n64_sk2", "umma2_n256", "umma2_n256_sk2", "umma2_n256_ts",
                 "umma_n64_x2", "umma_n128_x2")
        for v in [B.VARIANT_AUTO] + variant_ids(*names):
            if v >= 0 and B.variant_supports(v, M, N, K, K, N, ldc, batch, out_dtype) != 1:
                continue
            vals, raw, guards = G.run_gemm(A, Bm, M, N, K, K, N, ldc, out_dtype, batch, sA, sB, sC, variant=v)
            r = oracle.check(vals, Cref, S, G.tol_for(out_dtype))
            assert guards, f"padding or guard band overwritten ({B.variant_name(v)}, {(M, N, K, ldc, batch)})"
            assert r.ok, (B.variant_name(v), M, N, K, ldc, batch, r)


# ------------------------------------------------ integer closed forms: exact --

def all_umma_and_auto(M, N, K, out_dtype, batch=1):
    return [B.VARIANT_AUTO] + G.supported_variants(M, N, K, K, N, N, batch, out_dtype)


@pytest.mark.parametrize("out_dtype", [gi.F32, gi.BF16])
def test_identity_and_permutation_exact(out_dtype):
    rng = np.random.default_rng(5)
    n, N = 256, 320
    X = bits(rng.standard_normal((n, N)))
    P, pi = gi.permutation_bits(n, seed=3)
    for v in all_umma_and_auto(n, N, n, out_dtype):
        vals, raw, g = G.run_gemm(gi.identity_bits(n, n).ravel(), X.ravel(), n, N, n, n, N, N, out_dtype, variant=v)
        assert g and np.array_equal(vals[0], oracle.bf16_bits_to_f64(X)), B.variant_name(v)
        if out_dtype == gi.BF16:
            assert np.array_equal(raw[0], X)        # same bits back
        vals, raw, g = G.run_gemm(P.ravel(), X.ravel(), n, N, n, n, N, N, out_dtype, variant=v)
        assert g and np.array_equal(vals[0], oracle.bf16_bits_to_f64(X)[pi]), B.variant_name(v)
    Y = bits(rng.standard_normal((N, n)))
    for v in all_umma_and_auto(N, n, n, out_dtype):
        vals, raw, g = G.run_gemm(Y.ravel(), P.ravel(), N, n, n, n, n, n, out_dtype, variant=v)
        expect = np.empty((N, n)); expect[:, pi] = oracle.bf16_bits_to_f64(Y)
        assert g and np.array_equal(vals[0], expect), B.variant_name(v)


@pytest.mark.parametrize("M,N,K", [(257, 129, 1000), (16, 300, 8192), (300, 520, 200)])
def test_rank1_integer_closed_form_fp32_exact(M, N, K):
    A, Bm, u, v_, p, q = gi.rank1_int_operands(M, N, K, seed=M + K)
    expect = np.outer(u, v_).astype(np.float64) * float(np.dot(p, q))
    for v in all_umma_and_auto(M, N, K, gi.F32):
        vals, raw, g = G.run_gemm(A.ravel(), Bm.ravel(), M, N, K, K, N, N, gi.F32, variant=v)
        assert g and np.array_equal(vals[0], expect), B.variant_name(v)


def test_rank1_integer_closed_form_bf16_rounds_to_nearest_even():
    M, N, K = 200, 260, 520
    A, Bm, u, v_, p, q = gi.rank1_int_operands(M, N, K, seed=9)
    exact = np.outer(u, v_).astype(np.float64) * float(np.dot(p, q))
    expect_bits = oracle.f64_to_bf16_bits(exact)
    for v in all_umma_and_auto(M, N, K, gi.BF16):
        vals, raw, g = G.run_gemm(A.ravel(), Bm.ravel(), M, N, K, K, N, N, gi.BF16, variant=v)
        same = (raw[0] == expect_bits) | ((exact == 0) & (vals[0] == 0))
        assert g and same.all(), B.variant_name(v)


def test_bf16_ties_round_to_even():
    # C[i][j] = 256 + (i % 128) + j lies in [256, 512) where bf16 has spacing 2:
    # every odd value is an exact tie.  All operand entries are exact in bf16.
    M, N, K = 130, 70, 64
    Am = np.zeros((M, K)); Bmat = np.zeros((K, N))
    Am[:, 0] = 1.0; Bmat[0, :] = 256.0
    Am[:, 1] = np.arange(M) % 128; Bmat[1, :] = 1.0
    Am[:, 2] = 1.0; Bmat[2, :] = np.arange(N)
    exact = 256.0 + (np.arange(M) % 128)[:, None] + np.arange(N)[None, :]
    expect_bits = oracle.f64_to_bf16_bits(exact)
    assert oracle.bf16_bits_to_f64(oracle.f64_to_bf16_bits(np.array([257.0, 259.0]))).tolist() == [256.0, 260.0]
    for v in all_umma_and_auto(M, N, K, gi.BF16):
        vals, raw, g = G.run_gemm(bits(Am).ravel(), bits(Bmat).ravel(), M, N, K, K, N, N, gi.BF16, variant=v)
        assert g and np.array_equal(raw[0], expect_bits), B.variant_name(v)


@pytest.mark.parametrize("K", [1, 63, 64, 65, 4096])
def test_ones_checkerboard_and_k_marker(K):
    M, N = 140, 270
    ones_a, ones_b = bits(np.ones((M, K))), bits(np.ones((K, N)))
    alt = (-1.0) ** np.arange(K)
    Aa = bits(np.tile(alt, (M, 1)))
    for v in all_umma_and_auto(M, N, K, gi.F32):
        vals, _, g = G.run_gemm(ones_a.ravel(), ones_b.ravel(), M, N, K, K, N, N, gi.F32, variant=v)
        assert g and np.all(vals[0] == K), B.variant_name(v)
        vals, _, g = G.run_gemm(Aa.ravel(), ones_b.ravel(), M, N, K, K, N, N, gi.F32, variant=v)
        assert g and np.all(vals[0] == K % 2), B.variant_name(v)
    for k0 in sorted({0, min(15, K - 1), min(16, K - 1), min(63, K - 1), min(64, K - 1), K - 1}):
        Bk = np.zeros((K, N)); Bk[k0] = 1.0
        for v in [B.VARIANT_AUTO] + variant_ids("umma_n64", "umma_n256", "umma_n128_sk2"):
            if v >= 0 and B.variant_supports(v, M, N, K, K, N, N, 1, gi.F32) != 1:
                continue
            vals, _, g = G.run_gemm(ones_a.ravel(), bits(Bk).ravel(), M, N, K, K, N, N, gi.F32, variant=v)
            assert g and np.all(vals[0] == 1.0), (B.variant_name(v), k0)


def test_row_col_index_map_exact():
    M, N, K = 700, 1100, 70
    Am = np.zeros((M, K)); Am[:, 0] = np.arange(M) % 256
    Bmat = np.zeros((K, N)); Bmat[0] = np.arange(N) % 256
    expect = np.outer(np.arange(M) % 256, np.arange(N) % 256).astype(np.float64)
    for v in all_umma_and_auto(M, N, K, gi.F32):
        vals, _, g = G.run_gemm(bits(Am).ravel(), bits(Bmat).ravel(), M, N, K, K, N, N, gi.F32, variant=v)
        assert g and np.array_equal(vals[0], expect), B.variant_name(v)


def test_power_of_two_scaling_bitwise_and_run_to_run_identical():
    rng = np.random.default_rng(21)
    M, N, K = 260, 390, 777
    A = bits(rng.standard_normal((M, K))); Bm = bits(rng.standard_normal((K, N)))
    for out_dtype in (gi.F32, gi.BF16):
        for v in [B.VARIANT_AUTO] + variant_ids("umma_n128", "umma_n256_sk4", "umma_n64_sk8", "umma2_n256_sk4",
                                                "umma2_n256_ts", "umma2_n256_k1_ts", "umma_n128_k1"):
            _, raw0, _ = G.run_gemm(A.ravel(), Bm.ravel(), M, N, K, K, N, N, out_dtype, variant=v)
            _, raw1, _ = G.run_gemm(A.ravel(), Bm.ravel(), M, N, K, K, N, N, out_dtype, variant=v)
            assert np.array_equal(raw0, raw1)                       # deterministic
            A2 = bits(gi.bf16_bits_to_f32(A) * np.float32(16.0))
            vals2, _, _ = G.run_gemm(A2.ravel(), Bm.ravel(), M, N, K, K, N, N, out_dtype, variant=v)
            vals0 = (raw0.view(np.float32).astype(np.float64) if out_dtype == gi.F32
                     else oracle.bf16_bits_to_f64(raw0))
            assert np.array_equal(vals2, vals0 * 16.0)


# ------------------------------------------------------------- degenerate ----

def test_degenerate_sizes_and_k_zero():
    A = bits(np.ones((4, 4))).ravel(); Bm = bits(np.ones((4, 4))).ravel()
    for out_dtype in (gi.F32, gi.BF16):
        vals, _, g = G.run_gemm(A, Bm, 3, 4, 0, 4, 4, 4, out_dtype)      # K = 0 -> zeros
        assert g and vals.shape == (1, 3, 4) and not vals.any()
        vals, _, g = G.run_gemm(A, Bm, 0, 4, 4, 4, 4, 4, out_dtype)
        assert g
        vals, _, g = G.run_gemm(A, Bm, 4, 0, 4, 4, 4, 4, out_dtype)
        assert g
        vals, _, g = G.run_gemm(A, Bm, 4, 4, 4, 4, 4, 4, out_dtype, batch=0)
        assert g


def test_forced_variant_on_unsupported_shape_is_refused():
    v = variant_ids("umma_n64_sk16")[0]
    A = bits(np.ones((8, 64))).ravel(); Bm = bits(np.ones((64, 8))).ravel()
    G.run_gemm(A, Bm, 8, 8, 64, 64, 8, 8, gi.F32, variant=v, expect_status=B.ERR_UNSUPPORTED_SHAPE)


def test_host_buffer_entry_point():
    rng = np.random.default_rng(31)
    for (M, N, K, out_dtype, pad) in [(300, 200, 129, gi.F32, 0), (128, 256, 64, gi.BF16, 8)]:
        lda, ldb, ldc = K + pad, N + pad, N + pad
        A = bits(rng.standard_normal((M, K))); Bm = bits(rng.standard_normal((K, N)))
        Ap, Bp = gi.embed(A, lda, pad_bits=0), gi.embed(Bm, ldb, pad_bits=0)
        hA = torch.from_numpy(Ap.view(np.int16)).pin_memory()
        hB = torch.from_numpy(Bp.view(np.int16)).pin_memory()
        esz = 4 if out_dtype == gi.F32 else 2
        hC = torch.full((M * ldc,), -1, dtype=torch.int32 if esz == 4 else torch.int16).pin_memory()
        need = B.host_staging_bytes(M, N, K, lda, ldb, ldc, out_dtype)
        dev = torch.empty(need, dtype=torch.uint8, device="cuda")
        B.gemm_bf16_host(hA, hB, hC, M, N, K, lda, ldb, ldc, out_dtype, dev, need,
                         torch.cuda.current_stream())
        raw = hC.numpy().reshape(M, ldc)
        got = (raw[:, :N].view(np.float32).astype(np.float64) if esz == 4
               else oracle.bf16_bits_to_f64(raw[:, :N].view(np.uint16)))
        Cref, S = oracle.gemm(A, Bm, M, N, K)
        assert oracle.check(got, Cref, S, G.tol_for(out_dtype)).ok
        if pad:
            assert np.all(raw[:, N:] == -1)           # host padding untouched


@pytest.mark.parametrize("out_dtype", [gi.F32, gi.BF16])
def test_short_wide_products(out_dtype):
    """One or two tile rows and 100 to 280 tile columns (more tiles than the
    grid has CTAs, a thin last round), N a multiple of 16 or not, C with
    padding columns, B's pitch aligned for TMA or not."""
    cases = [(16, 16384, 128, 16384), (16, 16381, 96, 16384), (40, 7104, 64, 7104), (16, 11840, 70, 11848),
             (130, 17760, 64, 17760), (16, 35520, 64, 35520)]
    for (M, N, K, ldc) in cases:
        A = gi.random_operand(M + N, 0, M, K, K)
        Bm = gi.random_operand(M + N, 1, K, N, N)
        Cref, S = oracle.gemm_batched(A, Bm, M, N, K, K, N, M * K, K * N, 1)
        for v in [B.VARIANT_AUTO] + variant_ids("umma_n128", "umma_n256_ts", "umma2_n256_ts", "umma_n64_x2"):
            if v >= 0 and B.variant_supports(v, M, N, K, K, N, ldc, 1, out_dtype) != 1:
                continue
            vals, raw, guards = G.run_gemm(A, Bm, M, N, K, K, N, ldc, out_dtype, 1, M * K, K * N, M * ldc, variant=v)
            r = oracle.check(vals, Cref, S, G.tol_for(out_dtype))
            assert guards, f"padding or guard band overwritten ({B.variant_name(v)}, {(M, N, K, ldc)})"
            assert r.ok, (B.variant_name(v), M, N, K, ldc, r)


@pytest.mark.parametrize("out_dtype", [gi.F32, gi.BF16])
def test_short_a_boundaries(out_dtype):
    """The 128-column kernel has instantiations for M <= 16 and M <= 64 whose
    stages hold fewer rows of A and whose rings are deeper (10 and 8 k-blocks):
    M on both sides of each boundary, K short and long enough to wrap the ring
    several times, plain, split-K and tail-split variants."""
    rng = np.random.default_rng(77)
    for M in (8, 16, 17, 33, 63, 64, 65):
        for (N, K) in ((300, 64), (300, 200), (520, 1000), (129, 2500)):
            A = bits(rng.standard_normal((M, K)))
            Bm = bits(rng.uniform(-1, 1, (K, N)))
            ref = oracle.gemm(A, Bm, M, N, K)
            for v in variant_ids("umma_n128", "umma_n128_sk2", "umma_n128_ts", "umma_n128_sk4"):
                if B.variant_supports(v, M, N, K, K, N, N, 1, out_dtype) != 1:
                    continue
                check_case(A.ravel(), Bm.ravel(), M, N, K, out_dtype, v, ref=ref)


@pytest.mark.parametrize("out_dtype", [gi.F32, gi.BF16])
def test_large_unaligned_operands(out_dtype):
    """Larger products whose operands TMA cannot address (repacked by the warp-per-row-piece
    copy kernel): either operand or both unaligned (odd pitch, or a base two bytes off a
    16-byte boundary), row lengths that end inside a 512-element piece or right after one,
    lone-CTA, CTA-pair, split-K and tail-split kernels."""
    rng = np.random.default_rng(606 + out_dtype)
    cases = [(700, 900, 3000, 1, 3, 0, 0),        # (M, N, K, pad_a, pad_b, lead_a, lead_b)
             (1300, 1000, 2100, 3, 0, 0, 0),      # only A unaligned
             (520, 2100, 1800, 0, 5, 0, 0),       # only B unaligned
             (640, 1024, 2560, 0, 0, 1, 1),       # pitches fine, bases 2 bytes off
             (300, 513, 1025, 1, 1, 1, 0),        # one element past a 512-element piece
             (200, 1536, 512, 3, 3, 0, 1)]        # rows end exactly on a piece boundary
    names = ("umma_n64", "umma_n128_ts", "umma_n256_k2", "umma2_n256", "umma2_n256_ts", "umma2_n256_sk2",
             "umma_n128_sk4")
    for (M, N, K, pa, pb, la, lb) in cases:
        A = bits(rng.standard_normal((M, K))); Bm = bits(rng.standard_normal((K, N)))
        ref = oracle.gemm(A, Bm, M, N, K)
        lda, ldb = K + pa, N + pb
        Ap, Bp = gi.embed(A, lda), gi.embed(Bm, ldb)           # NaN padding
        for v in [B.VARIANT_AUTO] + variant_ids(*names):
            if v >= 0 and B.variant_supports(v, M, N, K, lda, ldb, N, 1, out_dtype) != 1:
                continue
            check_case(Ap, Bp, M, N, K, out_dtype, v, lda, ldb, N, ref=ref, lead_a=la, lead_b=lb)
