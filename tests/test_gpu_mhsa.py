"""Fused multi-head self-attention (the paper's Task 6) against the fp64 oracle.

Tolerance: |O_gpu - O_ref| <= 1e-2 * T with T[i][c] = sum_j p_ij |V[j][c]|: the
GPU rounds each probability to bf16 (relative 2^-9 = 2e-3) before the second
product and accumulates in fp32; scores and exponentials are fp32.
"""
import numpy as np
import pytest
import torch

import oracle
import gpu_util as G
from paper_2506_09092_b200 import binding as B
from paper_2506_09092_b200 import inputs as gi

pytestmark = pytest.mark.gpu

PAPER_SIZES = [(64, 32, 4), (128, 64, 8), (256, 128, 8), (384, 256, 16), (512, 512, 16)]


def bits(x):
    return gi.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def run(Q, K, V, N, dm, h, pad=0, expect=B.OK):
    ldq, ldk, ldv, ldo = dm + 8 * pad, dm + 16 * pad, dm + 8 * pad, dm + 3 * pad
    dQ, dK, dV = (torch.from_numpy(gi.embed(x, ld).view(np.int16)).cuda()
                  for x, ld in ((Q, ldq), (K, ldk), (V, ldv)))
    guard = 16
    dO = torch.full((guard + N * ldo + guard,), float("nan"), dtype=torch.float32, device="cuda")
    st = B.mhsa_bf16(dQ, dK, dV, dO.data_ptr() + 4 * guard, N, dm, h, ldq, ldk, ldv, ldo,
                     torch.cuda.current_stream(), check=False)
    assert st == expect, B.strerror(st)
    assert B.device_status(torch.cuda.current_stream()) == (B.OK, 0)
    host = dO.cpu().numpy()
    assert np.isnan(host[:guard]).all() and np.isnan(host[guard + N * ldo:]).all()
    body = host[guard:guard + N * ldo].reshape(N, ldo)
    if pad:
        assert np.isnan(body[:-1, dm:]).all()
    return body[:, :dm].astype(np.float64)


@pytest.mark.parametrize("N,dm,h", PAPER_SIZES)
def test_paper_sizes(N, dm, h):
    rng = np.random.default_rng([N, dm])
    Q, K, V = (bits(rng.standard_normal((N, dm))) for _ in range(3))
    got = run(Q, K, V, N, dm, h)
    ref, T = oracle.mhsa(Q, K, V, N, dm, h)
    r = oracle.check(got, ref, T, oracle.TOL_MHSA)
    G.log_observed_error("mhsa_bf16", f"N={N} d_model={dm} h={h}", r.max_scaled_err, oracle.TOL_MHSA,
                         "max |O - O_ref| / sum_j p_ij |v_jc|")
    assert r.ok, r
    # sharper score distributions too (larger queries)
    Q2 = bits(3.0 * rng.standard_normal((N, dm)))
    ref2, T2 = oracle.mhsa(Q2, K, V, N, dm, h)
    assert oracle.check(run(Q2, K, V, N, dm, h), ref2, T2, oracle.TOL_MHSA).ok


@pytest.mark.parametrize("N,dm,h,pad", [(37, 48, 3, 0), (100, 64, 8, 1), (300, 96, 4, 1), (1, 8, 1, 0),
                                         (129, 32, 1, 0), (511, 256, 8, 0), (33, 128, 4, 1)])
def test_ragged_sizes_and_padded_strides(N, dm, h, pad):
    rng = np.random.default_rng(N * 7 + dm)
    Q, K, V = (bits(rng.standard_normal((N, dm))) for _ in range(3))
    ref, T = oracle.mhsa(Q, K, V, N, dm, h)
    r = oracle.check(run(Q, K, V, N, dm, h, pad), ref, T, oracle.TOL_MHSA)
    assert r.ok, r


@pytest.mark.parametrize("N,dm,h,pad", [(513, 32, 4, 0), (640, 64, 2, 0), (1000, 64, 8, 1), (1024, 128, 4, 0),
                                         (2049, 64, 2, 0), (4100, 96, 3, 1)])
def test_sequences_longer_than_one_block_of_keys(N, dm, h, pad):
    """More than 512 keys: blocks of 512 with a running maximum (the last block ragged, down to
    one key).  The second data set has its large scores late in the sequence, so that the
    accumulators of the earlier blocks are scaled down by many orders of magnitude."""
    rng = np.random.default_rng(N * 3 + dm)
    Q, K, V = (bits(rng.standard_normal((N, dm))) for _ in range(3))
    ref, T = oracle.mhsa(Q, K, V, N, dm, h)
    r = oracle.check(run(Q, K, V, N, dm, h, pad), ref, T, oracle.TOL_MHSA)
    G.log_observed_error("mhsa_bf16", f"N={N} d_model={dm} h={h}", r.max_scaled_err, oracle.TOL_MHSA,
                         "max |O - O_ref| / sum_j p_ij |v_jc|")
    assert r.ok, r
    K2 = oracle.bf16_bits_to_f64(K).copy()
    K2[N - 40:] *= 6.0                                        # the dominant keys come last
    K2 = bits(K2)
    Q2 = bits(2.0 * rng.standard_normal((N, dm)))
    ref2, T2 = oracle.mhsa(Q2, K2, V, N, dm, h)
    assert oracle.check(run(Q2, K2, V, N, dm, h, pad), ref2, T2, oracle.TOL_MHSA).ok


def test_random_lengths_and_head_shapes():
    rng = np.random.default_rng(77)
    for it in range(30):
        h = int(rng.choice([1, 2, 3, 4, 8])); dk = int(rng.choice([8, 16, 24, 32])); dm = h * dk
        N = int(np.exp(rng.uniform(0, np.log(1800))))
        Q, K, V = (bits(rng.standard_normal((N, dm))) for _ in range(3))
        ref, T = oracle.mhsa(Q, K, V, N, dm, h)
        r = oracle.check(run(Q, K, V, N, dm, h, int(rng.integers(0, 2))), ref, T, oracle.TOL_MHSA)
        assert r.ok, (N, dm, h, r)


def test_closed_forms_over_several_blocks():
    rng = np.random.default_rng(3)
    N, dm, h = 1500, 64, 2
    V = bits(rng.standard_normal((N, dm))); K = bits(rng.standard_normal((N, dm)))
    # zero queries: uniform attention over all 1500 keys, every row is the column mean of V
    got = run(bits(np.zeros((N, dm))), K, V, N, dm, h)
    mean = oracle.bf16_bits_to_f64(V).mean(axis=0)
    assert np.allclose(got, np.tile(mean, (N, 1)), rtol=0, atol=2e-6)
    # one-hot selection across blocks: query i attends to key (i * 97 + 600) mod N only
    n, dm2 = 1100, 32
    target = (np.arange(n) * 97 + 600) % n
    code = lambda idx: np.stack([np.where((idx >> b) & 1, 1.0, -1.0) for b in range(11)], axis=1)
    Ks = np.zeros((n, dm2)); Qs = np.zeros((n, dm2))
    Ks[:, :11] = 16.0 * code(np.arange(n)); Qs[:, :11] = 16.0 * code(target)   # Q.K = 256 * (11 - 2 * Hamming distance)
    Vs = bits(rng.standard_normal((n, dm2)))
    got = run(bits(Qs), bits(Ks), Vs, n, dm2, 1)
    v = oracle.bf16_bits_to_f64(Vs)
    assert np.array_equal(got, v[target])                    # the next best key has e^-90 of the weight


def test_closed_forms():
    rng = np.random.default_rng(2)
    N, dm, h = 200, 64, 4
    V = bits(rng.standard_normal((N, dm))); K = bits(rng.standard_normal((N, dm)))
    # zero queries: uniform attention, every row is the column mean of V
    got = run(bits(np.zeros((N, dm))), K, V, N, dm, h)
    mean = oracle.bf16_bits_to_f64(V).mean(axis=0)
    assert np.allclose(got, np.tile(mean, (N, 1)), rtol=0, atol=2e-6)
    # one-hot selection: each query attends to exactly one key (other weights underflow to 0)
    n, dm2, h2 = 16, 32, 2
    pi = rng.permutation(n)
    Qs = np.zeros((n, dm2)); Ks = np.zeros((n, dm2))
    for i in range(n):
        Ks[i, i] = 16.0; Qs[i, i] = 32.0                       # head 0: identity
        Ks[i, 16 + i] = 16.0; Qs[i, 16 + pi[i]] = 32.0         # head 1: permutation
    Vs = bits(rng.standard_normal((n, dm2)))
    got = run(bits(Qs), bits(Ks), Vs, n, dm2, h2)
    v = oracle.bf16_bits_to_f64(Vs)
    assert np.array_equal(got[:, :16], v[:, :16]) and np.array_equal(got[:, 16:], v[pi][:, 16:])


def test_limits_and_errors():
    p = torch.zeros(4096, dtype=torch.int16, device="cuda")
    o = torch.zeros(4096, dtype=torch.float32, device="cuda")
    f = lambda *a: B.mhsa_bf16(*a, check=False)
    assert f(p, p, p, o, 64, 256, 4, 256, 256, 256, 256) == B.ERR_UNSUPPORTED_SHAPE  # d_k = 64
    assert f(p, p, p, o, 64, 24, 2, 24, 24, 24, 24) == B.ERR_UNSUPPORTED_SHAPE       # d_k = 12
    assert f(p, p, p, o, 64, 32, 4, 36, 32, 32, 32) == B.ERR_UNSUPPORTED_SHAPE       # ldq not a multiple of 8
    assert f(p, p, p, o, 64, 32, 3, 32, 32, 32, 32) == B.ERR_INVALID_DIM             # h does not divide d_model
    assert f(p, p, p, o, 64, 32, 4, 31, 32, 32, 32) == B.ERR_INVALID_LD
    assert f(None, p, p, o, 64, 32, 4, 32, 32, 32, 32) == B.ERR_INVALID_POINTER
    assert f(p, p, p, o, 0, 32, 4, 32, 32, 32, 32) == B.OK
