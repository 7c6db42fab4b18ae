"""Pins for the oracle of the paper's Tasks 8, 14, 15 and 4 (matrix transpose,
reduction, dot product, LayerNorm on float32 arrays): closed forms, literals,
library special cases and invariants that a dropped term, a wrong index, a
transposed operand or an accumulation in the wrong precision would break.
None of these tests touches the GPU."""
import math

import numpy as np
import pytest

import oracle


# ------------------------------------------------------------ Task 8 -----

@pytest.mark.parametrize("rows,cols,lda,ldat", [(3, 5, 5, 3), (5, 3, 7, 9), (64, 33, 40, 64), (1, 17, 17, 1),
                                                (17, 1, 1, 20)])
def test_transpose_index_map_closed_form(rows, cols, lda, ldat):
    """A[i][j] = i * cols + j  =>  AT[j][i] = i * cols + j, padding untouched."""
    A = np.full(rows * lda, -1.0, dtype=np.float32)
    for i in range(rows):
        A[i * lda: i * lda + cols] = np.arange(i * cols, (i + 1) * cols, dtype=np.float32)
    out = oracle.transpose_f32(A, rows, cols, lda, ldat, fill=777.0)
    assert out.size == (cols - 1) * ldat + rows
    for j in range(cols):
        for i in range(rows):
            assert out[j * ldat + i] == i * cols + j
        for i in range(rows, ldat):
            if j * ldat + i < out.size:
                assert out[j * ldat + i] == 777.0        # padding keeps its old contents


def test_transpose_is_an_involution_on_raw_bits_and_matches_the_library():
    rng = np.random.default_rng(8)
    bits = rng.integers(0, 2 ** 32, size=(37, 53), dtype=np.uint32)   # NaN payloads, denormals, everything
    A = bits.view(np.float32)
    T = oracle.transpose_f32(A, 37, 53).reshape(53, 37)
    assert np.array_equal(T.view(np.uint32), bits.T)                   # numpy's transpose, bit for bit
    back = oracle.transpose_f32(T, 53, 37).reshape(37, 53)
    assert np.array_equal(back.view(np.uint32), bits)


def test_transpose_of_a_symmetric_matrix_and_degenerate_sizes():
    rng = np.random.default_rng(9)
    X = rng.standard_normal((20, 20)).astype(np.float32)
    S = X + X.T
    assert np.array_equal(oracle.transpose_f32(S, 20, 20).reshape(20, 20), S)
    assert oracle.transpose_f32(np.zeros(0, np.float32), 0, 5).size == 0
    assert oracle.transpose_f32(np.zeros(0, np.float32), 5, 0).size == 0
    with pytest.raises(ValueError):
        oracle.transpose_f32(np.zeros(6, np.float32), 2, 3, lda=2)


# ----------------------------------------------------------- Task 14 -----

def test_sum_literals_and_integer_closed_forms():
    assert oracle.sum_f32(np.array([1.0, 2.0, 3.5], np.float32)) == (6.5, 6.5)
    assert oracle.sum_f32(np.array([], np.float32)) == (0.0, 0.0)
    n = 100000                                             # Gauss: exact in double, far beyond 2^24
    s, a = oracle.sum_f32(np.arange(1, n + 1, dtype=np.float32))
    assert s == n * (n + 1) / 2 == a
    alt = np.where(np.arange(1001) % 2 == 0, 1.0, -1.0).astype(np.float32)
    assert oracle.sum_f32(alt) == (1.0, 1001.0)


def test_sum_accumulates_in_double():
    # 1e8 is a float32; in float32 arithmetic 1e8 + 1 == 1e8, so a float32 accumulator returns 0
    assert oracle.sum_f32(np.array([1e8, 1.0, -1e8], np.float32))[0] == 1.0
    # 2^24 + 1 + 1 + ... : a float32 accumulator would stay at 2^24
    x = np.ones(1001, np.float32)
    x[0] = 2.0 ** 24
    assert oracle.sum_f32(x)[0] == 2.0 ** 24 + 1000


def test_sum_against_an_exactly_rounded_library_sum_and_invariances():
    rng = np.random.default_rng(14)
    for n in (1, 7, 1000, 2 ** 18):
        x = (rng.standard_normal(n) * np.exp(rng.uniform(-5, 5, n))).astype(np.float32)
        s, a = oracle.sum_f32(x)
        exact = math.fsum(float(v) for v in x)             # correctly rounded sum of the same values
        assert a == pytest.approx(math.fsum(abs(float(v)) for v in x), rel=1e-13)
        assert abs(s - exact) <= n * 2.0 ** -53 * a
        # a permutation changes the rounding order only
        s2, a2 = oracle.sum_f32(x[rng.permutation(n)])
        assert abs(s2 - s) <= 2 * n * 2.0 ** -53 * a
        # scaling by a power of two is exact
        s3, a3 = oracle.sum_f32(x * np.float32(8.0))
        assert s3 == 8.0 * s and a3 == 8.0 * a
        # sum |x| is the sum of the absolute values
        assert oracle.sum_f32(np.abs(x)) == (a, a)


# ----------------------------------------------------------- Task 15 -----

def test_dot_literals_and_integer_closed_forms():
    a = np.array([1.0, 2.0, 3.0], np.float32)
    b = np.array([4.0, -5.0, 6.0], np.float32)
    assert oracle.dot_f32(a, b) == (12.0, 32.0)
    n = 2000                                               # sum of squares: n (n + 1) (2n + 1) / 6
    v = np.arange(1, n + 1, dtype=np.float32)
    assert oracle.dot_f32(v, v)[0] == n * (n + 1) * (2 * n + 1) / 6
    # a unit vector selects one element; orthogonal vectors give zero
    e = np.zeros(n, np.float32)
    e[1234] = 1.0
    assert oracle.dot_f32(v, e) == (1235.0, 1235.0)
    assert oracle.dot_f32(np.array([1.0, 1.0], np.float32), np.array([1.0, -1.0], np.float32)) == (0.0, 2.0)
    assert oracle.dot_f32(np.array([], np.float32), np.array([], np.float32)) == (0.0, 0.0)
    with pytest.raises(ValueError):
        oracle.dot_f32(np.zeros(3, np.float32), np.zeros(4, np.float32))


def test_dot_products_are_exact_in_double():
    # (2^12 + 1)^2 = 2^24 + 2^13 + 1 is not a float32: a float32 product would lose the final 1
    x = np.array([2.0 ** 12 + 1.0], np.float32)
    assert oracle.dot_f32(x, x)[0] == 2.0 ** 24 + 2.0 ** 13 + 1.0
    # and the sum is a double sum: 2^24 * 1 + 1 * 1 + (-2^24) * 1 = 1
    a = np.array([2.0 ** 24, 1.0, -(2.0 ** 24)], np.float32)
    assert oracle.dot_f32(a, np.ones(3, np.float32))[0] == 1.0


def test_dot_against_an_exactly_rounded_library_sum_and_symmetry():
    rng = np.random.default_rng(15)
    for n in (1, 9, 4096, 2 ** 20):
        a = rng.standard_normal(n).astype(np.float32)
        b = rng.uniform(-1, 1, n).astype(np.float32)
        s, t = oracle.dot_f32(a, b)
        prods = a.astype(np.float64) * b.astype(np.float64)          # exact
        assert abs(s - math.fsum(prods)) <= n * 2.0 ** -53 * t
        assert oracle.dot_f32(b, a) == (s, t)                        # same products, same order
        assert oracle.dot_f32(np.abs(a), np.abs(b))[0] == t
        assert oracle.dot_f32(a, np.ones(n, np.float32))[0] == oracle.sum_f32(a)[0]


# ------------------------------------------------------------ Task 4 -----

EPS = 1e-5


def test_layernorm_two_valued_and_biased_variance_closed_forms():
    # x = (0, 2): mean 1, biased variance 1 (the unbiased estimate would be 2)
    y, mean, rstd = oracle.layernorm_f32(np.array([0.0, 2.0], np.float32), None, None, 1, 2, EPS)
    assert mean[0] == 1.0 and rstd[0] == 1.0 / math.sqrt(1.0 + EPS)
    assert y[0, 0] == -rstd[0] and y[0, 1] == rstd[0]
    # +-1 alternating: mean 0, variance 1
    m = 64
    x = np.where(np.arange(m) % 2 == 0, -1.0, 1.0).astype(np.float32)
    y, mean, rstd = oracle.layernorm_f32(x, None, None, 1, m, EPS)
    assert mean[0] == 0.0
    assert np.allclose(y[0], x.astype(np.float64) / math.sqrt(1.0 + EPS), rtol=1e-14, atol=0)


def test_layernorm_arithmetic_progression_closed_form():
    m = 4 * 16 * 16
    x = np.arange(m, dtype=np.float32)
    y, mean, rstd = oracle.layernorm_f32(x, None, None, 1, m, EPS)
    var = (m * m - 1) / 12.0                               # variance of 0 .. m-1
    assert mean[0] == (m - 1) / 2.0
    assert rstd[0] == pytest.approx(1.0 / math.sqrt(var + EPS), rel=1e-14)
    k = 777
    assert y[0, k] == pytest.approx((k - (m - 1) / 2.0) / math.sqrt(var + EPS), rel=1e-13)


def test_layernorm_affine_is_per_position_and_samples_are_independent():
    rng = np.random.default_rng(4)
    batch, m = 3, 96
    x = rng.standard_normal((batch, m)).astype(np.float32)
    x[1] = x[1] * 5 + 3                                    # a different mean and spread per sample
    gamma = np.arange(1, m + 1, dtype=np.float32)          # position-dependent: a wrong index shows
    beta = -np.arange(m, dtype=np.float32)
    y, mean, rstd = oracle.layernorm_f32(x, gamma, beta, batch, m, EPS)
    plain, _, _ = oracle.layernorm_f32(x, None, None, batch, m, EPS)
    assert np.allclose(y, plain * gamma + beta, rtol=1e-14, atol=1e-12)
    for s in range(batch):                                 # each sample alone gives the same row
        ys, ms, rs = oracle.layernorm_f32(x[s], gamma, beta, 1, m, EPS)
        assert np.array_equal(ys[0], y[s]) and ms[0] == mean[s] and rs[0] == rstd[s]
    # normalised rows: mean 0, variance var / (var + eps)
    var = x.astype(np.float64).var(axis=1)
    assert np.allclose(plain.mean(axis=1), 0.0, atol=1e-14)
    assert np.allclose(plain.var(axis=1), var / (var + EPS), rtol=1e-12)


def test_layernorm_against_an_fp64_library_computation_and_invariances():
    rng = np.random.default_rng(44)
    batch, m = 4, 4 * 8 * 8
    x = (rng.standard_normal((batch, m)) * 3 + 10).astype(np.float32)
    gamma = rng.uniform(0.5, 1.5, m).astype(np.float32)
    beta = rng.standard_normal(m).astype(np.float32)
    y, mean, rstd = oracle.layernorm_f32(x, gamma, beta, batch, m, EPS)
    x64 = x.astype(np.float64)
    ref = (x64 - x64.mean(axis=1, keepdims=True)) / np.sqrt(x64.var(axis=1, keepdims=True) + EPS) * gamma + beta
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)
    assert np.allclose(mean, x64.mean(axis=1), rtol=1e-14)
    # a shift of the input (exact here: integers added to multiples of 2^-10) leaves y unchanged
    xi = np.round(x * 1024) / 1024
    y0, _, _ = oracle.layernorm_f32(xi.astype(np.float32), gamma, beta, batch, m, EPS)
    y1, _, _ = oracle.layernorm_f32((xi + 64).astype(np.float32), gamma, beta, batch, m, EPS)
    assert np.allclose(y0, y1, rtol=0, atol=1e-10)
    # with eps = 0 a positive scaling of the input leaves y unchanged
    y2, _, _ = oracle.layernorm_f32(x, gamma, beta, batch, m, 0.0)
    y3, _, _ = oracle.layernorm_f32(x * np.float32(4.0), gamma, beta, batch, m, 0.0)
    assert np.allclose(y2, y3, rtol=1e-12, atol=1e-12)


def test_layernorm_constant_sample_returns_beta():
    m = 32
    beta = np.linspace(-1, 1, m).astype(np.float32)
    y, mean, rstd = oracle.layernorm_f32(np.full(m, 7.25, np.float32), np.full(m, 3.0, np.float32), beta, 1, m, EPS)
    assert mean[0] == 7.25 and rstd[0] == 1.0 / math.sqrt(EPS)
    assert np.array_equal(y[0], beta.astype(np.float64))
