"""The split-K entry point for callers that may not allocate device memory.

Such callers exist: a serving process that handed the whole GPU to its own
memory pool at start-up, or a plug-in that is only allowed to touch the tensors
it is given, cannot let a library call cudaMalloc behind their back (it may
fail, and it may stall the device).  ``cudallm_gemm_bf16_splitk_noalloc`` keeps
its split-K scratch in an array that is part of the library's device image
instead.  This file checks, through the C ABI, that it computes the same
product as the ordinary entry point and as the CPU oracle, twice in a row on
different problems (the second call finds the first call's leftovers in the
shared scratch), that further calls leave the amount of free device memory
unchanged, and that it accepts the largest problem its fixed scratch holds and
refuses the next larger one.

Named ``test_zz_*`` so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_09092_b200 import binding as B
from paper_2506_09092_b200 import inputs as gi

pytestmark = pytest.mark.gpu


def _bits(x):
    return gi.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _to_f64(t, out_dtype):
    host = t.cpu().numpy()
    return host.astype(np.float64) if out_dtype == gi.F32 else oracle.bf16_bits_to_f64(host.view(np.uint16))


def _both_ways(M, N, K, out_dtype, split_k, seed):
    rng = np.random.default_rng(seed)
    A = _bits(rng.standard_normal((M, K)))
    Bm = _bits(rng.standard_normal((K, N)))
    dA = torch.from_numpy(A.view(np.int16)).cuda()
    dB = torch.from_numpy(Bm.view(np.int16)).cuda()
    dt = torch.float32 if out_dtype == gi.F32 else torch.int16
    c_old = torch.zeros((M, N), dtype=dt, device="cuda")
    c_new = torch.full((M, N), 7, dtype=dt, device="cuda")        # old contents must not matter
    stream = torch.cuda.current_stream()
    B.gemm_bf16(dA, dB, c_old, M, N, K, K, N, N, out_dtype, stream)
    B.gemm_bf16_splitk_noalloc(dA, dB, c_new, M, N, K, K, N, N, out_dtype, split_k, stream)
    torch.cuda.synchronize()
    C_ref, S = oracle.gemm(A, Bm, M, N, K)
    tol = oracle.TOL_F32_OUT if out_dtype == gi.F32 else oracle.TOL_BF16_OUT
    old, new = _to_f64(c_old, out_dtype), _to_f64(c_new, out_dtype)
    assert np.isfinite(new).all()
    # against the ordinary entry point ...
    assert np.all(np.abs(new - old) <= tol * S), float(np.max(np.abs(new - old) / np.maximum(S, 1e-300)))
    # ... and, so that an error both share cannot pass, against the oracle
    r = oracle.check(new, C_ref, S, tol)
    assert r.ok, r


def test_two_calls_in_a_row_match_the_ordinary_entry_point():
    # first call: larger scratch footprint; second: smaller problem, other split and
    # output type, which must not see what the first left behind
    _both_ways(300, 520, 2048, gi.F32, 8, seed=1)
    _both_ways(130, 264, 1000, gi.BF16, 2, seed=2)
    _both_ways(16, 3968, 4096, gi.F32, 4, seed=3)        # 62 tiles x 4 slots: near the limit


def _noalloc_only(M, N, K, out_dtype, split_k, seed):
    """One call of the no-allocation entry point alone, checked against the oracle."""
    rng = np.random.default_rng(seed)
    A = _bits(rng.standard_normal((M, K)))
    Bm = _bits(rng.standard_normal((K, N)))
    dA = torch.from_numpy(A.view(np.int16)).cuda()
    dB = torch.from_numpy(Bm.view(np.int16)).cuda()
    c = torch.full((M, N), 7, dtype=torch.float32 if out_dtype == gi.F32 else torch.int16, device="cuda")
    return (A, Bm, dA, dB, c), lambda: B.gemm_bf16_splitk_noalloc(dA, dB, c, M, N, K, K, N, N, out_dtype, split_k,
                                                                   torch.cuda.current_stream())


def test_further_calls_leave_free_device_memory_unchanged():
    """What the entry point exists for.  After one warm-up call (the driver may load kernels on
    a first launch) further calls, on another shape too, neither take nor return device memory."""
    (A, Bm, dA, dB, c), call = _noalloc_only(260, 336, 1504, gi.F32, 4, seed=5)
    (A2, B2, dA2, dB2, c2), call2 = _noalloc_only(100, 1000, 640, gi.BF16, 2, seed=6)
    call()
    call2()
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        call()
        call2()
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    C_ref, S = oracle.gemm(A, Bm, 260, 336, 1504)
    assert oracle.check(_to_f64(c, gi.F32), C_ref, S, oracle.TOL_F32_OUT).ok
    C_ref, S = oracle.gemm(A2, B2, 100, 1000, 640)
    assert oracle.check(_to_f64(c2, gi.BF16), C_ref, S, oracle.TOL_BF16_OUT).ok


def test_largest_problem_the_scratch_holds_and_the_next_larger_one():
    """P = ceil(M/128) * ceil(N/64) * split_k slots: 254 fit behind the header, 255 and more do not."""
    (A, Bm, dA, dB, c), call = _noalloc_only(128, 8128, 256, gi.F32, 2, seed=7)      # 1 x 127 x 2 = 254
    call()
    torch.cuda.synchronize()
    C_ref, S = oracle.gemm(A, Bm, 128, 8128, 256)
    assert oracle.check(_to_f64(c, gi.F32), C_ref, S, oracle.TOL_F32_OUT).ok
    p = torch.zeros(8, dtype=torch.int16, device="cuda")                          # never dereferenced
    f = lambda *a: B.gemm_bf16_splitk_noalloc(*a, check=False)
    assert f(p, p, p, 128, 8192, 256, 256, 8192, 8192, gi.F32, 2) == B.ERR_TOO_LARGE   # 128 x 2 = 256
    assert f(p, p, p, 129, 8128, 256, 256, 8128, 8128, gi.F32, 2) == B.ERR_TOO_LARGE   # 2 x 127 x 2 = 508


def test_limits_are_reported_not_exceeded():
    p = torch.zeros(1024, dtype=torch.int16, device="cuda")
    f = lambda *a: B.gemm_bf16_splitk_noalloc(*a, check=False)
    # 16 x 4096 x 1024 x 4 B = 256 MiB of partial sums: beyond the 8 MiB scratch
    assert f(p, p, p, 4096, 1024, 4096, 4096, 1024, 1024, gi.F32, 16) == B.ERR_TOO_LARGE
    assert "scratch" in B.strerror(B.ERR_TOO_LARGE)
    assert f(p, p, p, 64, 64, 64, 64, 64, 64, gi.F32, 2) == B.ERR_UNSUPPORTED_SHAPE   # one k-block only
    assert f(p, p, p, 64, 64, 512, 515, 64, 64, gi.F32, 2) == B.ERR_UNSUPPORTED_SHAPE  # lda not TMA-able
    assert f(p, p, p, 64, 64, 512, 512, 64, 64, gi.F32, 3) == B.ERR_INVALID_VARIANT
    assert f(None, p, p, 64, 64, 512, 512, 64, 64, gi.F32, 2) == B.ERR_INVALID_POINTER
