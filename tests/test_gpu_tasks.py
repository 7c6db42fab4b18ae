"""Parity of the float32 task kernels (Tasks 8, 14, 15, 4: matrix transpose,
reduction, dot product, LayerNorm) against the CPU oracle, through the C ABI.

Bars
----
* transpose: bit-exact (data movement), padding and guard bands untouched;
* sum / dot: the kernels accumulate in double and round once, so
  |gpu - ref| <= 2^-24 |ref| + 2 n 2^-53 * sum|terms|  (the second term covers
  the different summation orders of the two double accumulations);
* LayerNorm: |gpu - ref| <= 2^-20 * (|z| + 1) |gamma| + 2^-22 |beta|, z = (x - mean) rstd.
  The kernels take the moments in float32 about a pilot value near the data
  (7 + 3 roundings of 2^-24 per 32-byte piece, relative to the deviations, so the
  mean is good to ~2^-21.5 of the spread and 1/sqrt(var + eps) to ~2^-22
  relative) and form the output in float32 from a two-float mean (four roundings
  of 2^-24); the bound leaves a factor of two.
"""
import numpy as np
import pytest
import torch

import oracle
import gpu_util as G
from paper_2506_09092_b200 import binding as B
from paper_2506_09092_b200 import inputs as gi

pytestmark = pytest.mark.gpu

SENT = np.float32(-12345.678)


def dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def status_ok():
    code, detail = B.device_status(torch.cuda.current_stream())
    assert code == B.OK, (code, hex(detail))


# ------------------------------------------------------------ Task 8 -----

def run_transpose(A, rows, cols, lda, ldat, lead_in=0, lead_out=0):
    guard = 64
    dA = torch.empty(A.size + lead_in, dtype=torch.float32, device="cuda")
    dA[lead_in:] = dev(A)
    n_out = (cols - 1) * ldat + rows if rows and cols else 0
    dT = torch.full((guard + lead_out + n_out + guard,), float(SENT), dtype=torch.float32, device="cuda")
    B.transpose_f32(dA.data_ptr() + 4 * lead_in, dT.data_ptr() + 4 * (guard + lead_out), rows, cols, lda, ldat,
                    torch.cuda.current_stream())
    status_ok()
    out = dT.cpu().numpy()
    body = out[guard + lead_out: guard + lead_out + n_out]
    assert np.all(out[:guard + lead_out] == SENT) and np.all(out[guard + lead_out + n_out:] == SENT), "guard band"
    return body


@pytest.mark.parametrize("rows,cols,pad_in,pad_out,lead", [
    (64, 64, 0, 0, 0), (256, 128, 0, 0, 0), (100, 36, 0, 0, 0), (36, 100, 4, 8, 0), (1024, 1024, 0, 0, 0),
    (4, 4, 0, 0, 0), (68, 2052, 12, 4, 0), (1000, 24, 0, 0, 0),                 # TMA path, ragged patches
    (37, 53, 0, 0, 0), (129, 257, 3, 1, 0), (64, 64, 0, 0, 1), (1, 1000, 0, 0, 0), (1000, 1, 5, 0, 3),
    (130, 66, 0, 0, 2)])                                                          # plain path
def test_transpose_bit_exact(rows, cols, pad_in, pad_out, lead):
    rng = np.random.default_rng(rows * 131 + cols)
    lda, ldat = cols + pad_in, rows + pad_out
    bits = rng.integers(0, 2 ** 32, size=(rows - 1) * lda + cols, dtype=np.uint32)   # any bit pattern
    A = bits.view(np.float32)
    ref = oracle.transpose_f32(A, rows, cols, lda, ldat, fill=float(SENT))
    got = run_transpose(A, rows, cols, lda, ldat, lead, lead)
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))


def test_transpose_index_map_and_involution_at_a_paper_size():
    n = gi.TRANSPOSE_SIZES[2]                                # 4096: 64 MB, several waves of patches
    A = np.arange(n * n, dtype=np.float32)                   # exact below 2^24 = n * n
    got = run_transpose(A, n, n, n, n).reshape(n, n)
    i = np.arange(n)
    for j in (0, 1, 63, 64, 1000, n - 1):                    # AT[j][i] = i * n + j
        assert np.array_equal(got[j], (i * n + j).astype(np.float32))
    back = run_transpose(got.reshape(-1), n, n, n, n)
    assert np.array_equal(back, A)


def test_transpose_degenerate_and_errors():
    s = torch.cuda.current_stream()
    x = torch.zeros(64, device="cuda")
    assert B.transpose_f32(x, x, 0, 5, 5, 0, s, check=False) == B.OK
    assert B.transpose_f32(x, x, 5, 0, 0, 5, s, check=False) == B.OK
    assert B.transpose_f32(x, x, -1, 5, 5, 5, s, check=False) == B.ERR_INVALID_DIM
    assert B.transpose_f32(x, x, 4, 8, 7, 4, s, check=False) == B.ERR_INVALID_LD
    assert B.transpose_f32(x, x, 4, 8, 8, 3, s, check=False) == B.ERR_INVALID_LD
    assert B.transpose_f32(None, x, 4, 8, 8, 4, s, check=False) == B.ERR_INVALID_POINTER
    assert B.transpose_f32(x.data_ptr() + 2, x, 4, 8, 8, 4, s, check=False) == B.ERR_MISALIGNED


# ----------------------------------------------------- Tasks 14 and 15 -----

def sum_bound(ref, sum_abs, n):
    return 2.0 ** -24 * abs(ref) + 2 * max(n, 1) * 2.0 ** -53 * sum_abs


def gpu_sum(x, lead=0):
    d = torch.empty(x.size + lead, dtype=torch.float32, device="cuda")
    d[lead:] = dev(x)
    r = torch.full((3,), float(SENT), dtype=torch.float32, device="cuda")
    B.sum_f32(d.data_ptr() + 4 * lead, x.size, r.data_ptr() + 4, torch.cuda.current_stream())
    out = r.cpu().numpy()
    assert out[0] == SENT and out[2] == SENT
    return float(out[1])


def gpu_dot(a, b, lead_a=0, lead_b=0):
    da = torch.empty(a.size + lead_a, dtype=torch.float32, device="cuda")
    da[lead_a:] = dev(a)
    db = torch.empty(b.size + lead_b, dtype=torch.float32, device="cuda")
    db[lead_b:] = dev(b)
    r = torch.full((3,), float(SENT), dtype=torch.float32, device="cuda")
    B.dot_f32(da.data_ptr() + 4 * lead_a, db.data_ptr() + 4 * lead_b, a.size, r.data_ptr() + 4,
              torch.cuda.current_stream())
    out = r.cpu().numpy()
    assert out[0] == SENT and out[2] == SENT
    return float(out[1])


@pytest.mark.parametrize("n", [0, 1, 3, 4, 5, 1023, 8192, 8193, 100003] + gi.REDUCTION_SIZES + [(1 << 24) + 77])
def test_sum_against_oracle(n):
    for lead in (0, 1, 3):
        x = gi.task_array(14, n % 1000, n, std=3.0, mean=0.25)
        ref, sabs = oracle.sum_f32(x)
        got = gpu_sum(x, lead)
        assert abs(got - ref) <= sum_bound(ref, sabs, n), (n, lead, got, ref)


def test_sum_integer_closed_forms_and_double_accumulation():
    n = 4000                                                   # Gauss sum, below 2^24: exact in fp32 too
    assert gpu_sum(np.arange(1, n + 1, dtype=np.float32)) == n * (n + 1) / 2
    # cancellation that a float32 accumulator loses
    x = np.ones(100001, np.float32)
    x[0], x[-1] = 2.0 ** 24, -(2.0 ** 24)
    assert gpu_sum(x) == 99999.0
    # run-to-run identical bits
    y = gi.task_array(15, 7, 1 << 20)
    assert gpu_sum(y) == gpu_sum(y)


@pytest.mark.parametrize("n", [0, 1, 2, 5, 4097, 65537] + gi.DOT_SIZES + [(1 << 23) + 5])
def test_dot_against_oracle(n):
    a = gi.task_array(15, 0, n)
    b = gi.task_array(15, 1, n, "uniform")
    ref, t = oracle.dot_f32(a, b)
    for (la, lb) in ((0, 0), (1, 1), (0, 2), (3, 1)):          # equal and unequal misalignment
        got = gpu_dot(a, b, la, lb)
        assert abs(got - ref) <= sum_bound(ref, t, n), (n, la, lb, got, ref)


def test_dot_integer_closed_forms_and_exact_products():
    n = 300                                                    # sum of squares n (n + 1) (2 n + 1) / 6 < 2^24
    v = np.arange(1, n + 1, dtype=np.float32)
    assert gpu_dot(v, v) == n * (n + 1) * (2 * n + 1) / 6
    e = np.zeros(5000, np.float32)
    e[4321] = 1.0
    w = np.arange(5000, dtype=np.float32)
    assert gpu_dot(w, e) == 4321.0
    # (2^12 + 1)^2 - 2^24 - 2^13 = 1 needs the exact product and a double sum
    a = np.array([2.0 ** 12 + 1, 2.0 ** 12, 2.0 ** 7], np.float32)
    b = np.array([2.0 ** 12 + 1, -(2.0 ** 12), -(2.0 ** 6)], np.float32)
    assert gpu_dot(a, b) == 1.0


def test_reduce_errors():
    s = torch.cuda.current_stream()
    x = torch.zeros(16, device="cuda")
    assert B.sum_f32(x, -1, x, s, check=False) == B.ERR_INVALID_DIM
    assert B.sum_f32(None, 4, x, s, check=False) == B.ERR_INVALID_POINTER
    assert B.sum_f32(x, 4, None, s, check=False) == B.ERR_INVALID_POINTER
    assert B.sum_f32(x.data_ptr() + 1, 4, x, s, check=False) == B.ERR_MISALIGNED
    assert B.dot_f32(x, None, 4, x, s, check=False) == B.ERR_INVALID_POINTER


# ------------------------------------------------------------ Task 4 -----

def run_layernorm(x, gamma, beta, batch, m, eps=1e-5, lead=0, in_place=False):
    guard = 64
    dx = torch.empty(x.size + lead, dtype=torch.float32, device="cuda")
    dx[lead:] = dev(x)
    dg = None if gamma is None else dev(gamma)
    db = None if beta is None else dev(beta)
    dy = torch.full((guard + lead + batch * m + guard,), float(SENT), dtype=torch.float32, device="cuda")
    xptr = dx.data_ptr() + 4 * lead
    yptr = xptr if in_place else dy.data_ptr() + 4 * (guard + lead)
    B.layernorm_f32(xptr, dg, db, yptr, batch, m, eps, torch.cuda.current_stream())
    status_ok()
    if in_place:
        return dx[lead:].cpu().numpy().astype(np.float64).reshape(batch, m)
    out = dy.cpu().numpy()
    assert np.all(out[:guard + lead] == SENT) and np.all(out[guard + lead + batch * m:] == SENT), "guard band"
    return out[guard + lead: guard + lead + batch * m].astype(np.float64).reshape(batch, m)


def check_layernorm(got, x, gamma, beta, batch, m, eps=1e-5):
    ref, mean, rstd = oracle.layernorm_f32(x, gamma, beta, batch, m, eps)
    g = np.ones(m) if gamma is None else gamma.astype(np.float64)
    b = np.zeros(m) if beta is None else beta.astype(np.float64)
    z = np.abs(x.astype(np.float64).reshape(batch, m) - mean[:, None]) * rstd[:, None]
    bound = 2.0 ** -20 * (z + 1.0) * np.abs(g) + 2.0 ** -22 * np.abs(b)
    err = np.abs(got - ref)
    assert np.all(np.isfinite(got))
    G.log_observed_error("layernorm_f32", f"batch={batch} m={m}", float((err / np.maximum(bound, 1e-300)).max()), 1.0,
                         "max |y - y_ref| / (2^-20 (|z| + 1)|gamma| + 2^-22 |beta|)")
    assert np.all(err <= bound), (float((err / np.maximum(bound, 1e-300)).max()), np.unravel_index(np.argmax(err - bound), err.shape))


@pytest.mark.parametrize("batch,m", [(1, 4), (3, 7), (16, 4 * 64 * 64), (16, 4 * 128 * 128), (5, 4096 * 3 + 4),
                                     (2, 1 << 20), (200, 1000), (7, 100003), (16, 4 * 256 * 256), (5, 1 << 21),
                                     (40, 200000), (33, 100024), (1, 8)])
def test_layernorm_against_oracle(batch, m):
    x, gamma, beta = gi.layernorm_inputs(4, batch, m)
    check_layernorm(run_layernorm(x, gamma, beta, batch, m), x, gamma, beta, batch, m)


@pytest.fixture
def layernorm_path():
    """Forces cudallm_layernorm_f32 onto one of its two kernels for the test's duration."""
    def force(path):
        B.debug_set(B.DEBUG_LAYERNORM_PATH, path)
    yield force
    B.debug_set(B.DEBUG_LAYERNORM_PATH, 0)


# Sizes that exercise the persistent kernel's rings and hand-over slots: one CTA; a few CTAs with
# a ragged last slice; 148 slices of 1, 2 (ragged), 3 and 7 chunks of 16 KB with more samples
# than the rings hold; one sample with slices of 10 chunks; more samples than one launch has
# room for in the exchange area (148 CTAs: 147 samples); many samples of one short chunk.
@pytest.mark.parametrize("batch,m", [(1, 8), (3, 8000), (16, 4 * 64 * 64), (9, 148 * 4096),
                                     (6, 148 * 4096 * 2 - 4096 * 5 + 24), (5, 148 * 4096 * 3),
                                     (3, 148 * 4096 * 7 - 40), (1, 148 * 4096 * 10 - 8), (7, 100000),
                                     (150, 148 * 1024), (45, 148 * 1024 + 8)])
def test_layernorm_one_pass_kernel_against_oracle(layernorm_path, batch, m):
    x, gamma, beta = gi.layernorm_inputs(14, batch, m)
    layernorm_path(2)
    got = run_layernorm(x, gamma, beta, batch, m)
    check_layernorm(got, x, gamma, beta, batch, m)
    assert np.array_equal(got, run_layernorm(x, gamma, beta, batch, m))          # repeatable bit for bit
    layernorm_path(1)
    check_layernorm(run_layernorm(x, gamma, beta, batch, m), x, gamma, beta, batch, m)


def test_layernorm_random_sizes_on_both_paths(layernorm_path):
    rng = np.random.default_rng(4400)
    for it in range(24):
        batch = int(rng.integers(1, 12)); m = 8 * int(np.exp(rng.uniform(0, np.log(60000))))
        x, gamma, beta = gi.layernorm_inputs(4400 + it, batch, m)
        layernorm_path(int(rng.choice([1, 2])))
        check_layernorm(run_layernorm(x, gamma, beta, batch, m), x, gamma, beta, batch, m)


def test_layernorm_one_pass_kernel_variants_of_the_call(layernorm_path):
    layernorm_path(2)
    batch, m = 6, 148 * 1024 + 64
    x, gamma, beta = gi.layernorm_inputs(45, batch, m)
    check_layernorm(run_layernorm(x, None, None, batch, m), x, None, None, batch, m)
    check_layernorm(run_layernorm(x, gamma, None, batch, m), x, gamma, None, batch, m)
    check_layernorm(run_layernorm(x, gamma, beta, batch, m, in_place=True), x, gamma, beta, batch, m)
    check_layernorm(run_layernorm(x, gamma, beta, batch, m, eps=0.5), x, gamma, beta, batch, m, eps=0.5)
    # closed forms: a constant sample returns beta exactly; a large common offset does not cancel
    m = 148 * 2048
    beta = np.linspace(-1, 1, m).astype(np.float32)
    gamma = np.full(m, 3.0, np.float32)
    got = run_layernorm(np.full(2 * m, 7.25, np.float32), gamma, beta, 2, m)
    assert np.array_equal(got[0], beta.astype(np.float64)) and np.array_equal(got[1], got[0])
    sign = np.where(np.arange(m) % 2 == 0, -1.0, 1.0).astype(np.float32)
    y = (np.float32(4096.0) + sign * np.float32(2.0 ** -6)).astype(np.float32)
    got = run_layernorm(y, None, None, 1, m)
    ref, _, _ = oracle.layernorm_f32(y, None, None, 1, m)
    assert np.allclose(got, ref, rtol=2e-7, atol=0)


def test_layernorm_one_pass_kernel_wait_limit(layernorm_path):
    """The CTAs of the persistent kernel wait for one another's moments; with the entries tagged
    with a value nobody waits for, every such wait runs out after the (shortened) limit, the
    kernel returns, the status word says so, and the next call is unaffected."""
    layernorm_path(2)
    batch, m = 4, 1 << 20
    x, gamma, beta = gi.layernorm_inputs(46, batch, m)
    s = torch.cuda.current_stream()
    dx, dg, db = dev(x), dev(gamma), dev(beta)
    dy = torch.zeros(batch * m, dtype=torch.float32, device="cuda")
    assert B.device_status(s) == (B.OK, 0)
    try:
        B.debug_set(B.DEBUG_WAIT_LIMIT_NS, 1_000_000)
        B.debug_set(B.DEBUG_MISS_NEXT_SPLIT_FLAGS, 1)
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        B.layernorm_f32(dx, dg, db, dy, batch, m, 1e-5, s)
        t1.record()
        code, detail = B.device_status(s)
        assert code == B.ERR_DEVICE_TIMEOUT and detail >> 8 == 5 and detail & 0xF0 == 0x10, (code, hex(detail))
        assert 0.9 <= t0.elapsed_time(t1) < 500.0
        assert B.device_status(s) == (B.OK, 0)
    finally:
        B.debug_set(B.DEBUG_WAIT_LIMIT_NS, 0)
        B.debug_set(B.DEBUG_MISS_NEXT_SPLIT_FLAGS, 0)
    check_layernorm(run_layernorm(x, gamma, beta, batch, m), x, gamma, beta, batch, m)


def test_layernorm_without_affine_misaligned_and_in_place():
    batch, m = 6, 5000
    x, gamma, beta = gi.layernorm_inputs(44, batch, m)
    check_layernorm(run_layernorm(x, None, None, batch, m), x, None, None, batch, m)
    check_layernorm(run_layernorm(x, gamma, None, batch, m, lead=1), x, gamma, None, batch, m)
    check_layernorm(run_layernorm(x, gamma, beta, batch, m, in_place=True), x, gamma, beta, batch, m)
    check_layernorm(run_layernorm(x, gamma, beta, batch, m, eps=0.5), x, gamma, beta, batch, m, eps=0.5)


def test_layernorm_closed_forms():
    # a constant sample returns beta exactly; +-1 gives +-1/sqrt(1 + eps) * gamma + beta
    m = 4096
    beta = np.linspace(-1, 1, m).astype(np.float32)
    gamma = np.full(m, 3.0, np.float32)
    got = run_layernorm(np.full(m, 7.25, np.float32), gamma, beta, 1, m)
    assert np.array_equal(got[0], beta.astype(np.float64))
    x = np.where(np.arange(m) % 2 == 0, -1.0, 1.0).astype(np.float32)
    got = run_layernorm(x, None, None, 1, m)
    want = np.float32(1.0 / np.sqrt(1.0 + 1e-5))
    assert np.array_equal(got[0], x.astype(np.float64) * float(want))
    # a large common offset: the variance must not cancel (mean 4096, spread 2^-6)
    y = (np.float32(4096.0) + x * np.float32(2.0 ** -6)).astype(np.float32)
    got = run_layernorm(y, None, None, 1, m)
    ref, _, _ = oracle.layernorm_f32(y, None, None, 1, m)
    assert np.allclose(got, ref, rtol=2e-7, atol=0)


def test_layernorm_errors():
    s = torch.cuda.current_stream()
    x = torch.zeros(64, device="cuda")
    assert B.layernorm_f32(x, None, None, x, 0, 8, 1e-5, s, check=False) == B.OK
    assert B.layernorm_f32(x, None, None, x, 2, -1, 1e-5, s, check=False) == B.ERR_INVALID_DIM
    assert B.layernorm_f32(x, None, None, x, 2, 8, -1.0, s, check=False) == B.ERR_INVALID_DIM
    assert B.layernorm_f32(None, None, None, x, 2, 8, 1e-5, s, check=False) == B.ERR_INVALID_POINTER
    assert B.layernorm_f32(x, None, None, x.data_ptr() + 2, 2, 8, 1e-5, s, check=False) == B.ERR_MISALIGNED
