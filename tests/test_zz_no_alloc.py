"""The split-K entry point for callers that may not allocate device memory.

Such callers exist: a serving process that handed the whole GPU to its own
memory pool at start-up, or a plug-in that is only allowed to touch the tensors
it is given, cannot let a library call cudaMalloc behind their back (it may
fail, and it may stall the device).  ``cudallm_gemm_bf16_splitk_noalloc`` keeps
its split-K scratch in an array that is part of the library's device image
instead.  This file checks, through the C ABI, that it computes the same
product as the ordinary entry point, twice in a row on different problems (the
second call finds the first call's leftovers in the shared scratch), and that
it refuses problems beyond its fixed scratch.

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
    _, S = oracle.gemm(A, Bm, M, N, K)
    tol = oracle.TOL_F32_OUT if out_dtype == gi.F32 else oracle.TOL_BF16_OUT
    old, new = _to_f64(c_old, out_dtype), _to_f64(c_new, out_dtype)
    assert np.isfinite(new).all()
    assert np.all(np.abs(new - old) <= tol * S), float(np.max(np.abs(new - old) / np.maximum(S, 1e-300)))


def test_two_calls_in_a_row_match_the_ordinary_entry_point():
    # first call: larger scratch footprint; second: smaller problem, other split and
    # output type, which must not see what the first left behind
    _both_ways(300, 520, 2048, gi.F32, 8, seed=1)
    _both_ways(130, 264, 1000, gi.BF16, 2, seed=2)
    _both_ways(16, 3968, 4096, gi.F32, 4, seed=3)        # 62 tiles x 4 slots: near the limit


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
