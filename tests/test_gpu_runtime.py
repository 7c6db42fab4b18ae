"""Runtime behaviour of the library on the GPU beyond single products: the
caller-provided workspace, calls on two streams, the status word, and the
paper's own Task 2 shapes at larger sizes."""
import numpy as np
import pytest
import torch

import oracle
import gpu_util as G
from paper_2506_09092_b200 import binding as B
from paper_2506_09092_b200 import inputs as gi

pytestmark = pytest.mark.gpu


def bits(x):
    return gi.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _names():
    return {B.variant_name(v): v for v in range(B.num_variants())}


def test_device_status_is_clean_after_normal_calls():
    A = bits(np.ones((64, 64))).ravel()
    G.run_gemm(A, A, 64, 64, 64, 64, 64, 64, gi.F32)
    assert B.device_status(torch.cuda.current_stream()) == (B.OK, 0)


def test_caller_provided_workspace():
    """Split-K and repacking take their scratch from a workspace the caller set;
    one that is too small is refused before anything runs."""
    names = _names()
    rng = np.random.default_rng(3)
    M, N, K = 200, 300, 1030
    lda, ldb, ldc = K + 1, N + 3, N                        # A and B need repacking
    A = bits(rng.standard_normal((M, K))); Bm = bits(rng.standard_normal((K, N)))
    Ap, Bp = gi.embed(A, lda), gi.embed(Bm, ldb)
    Cref, S = oracle.gemm(A, Bm, M, N, K)
    need = B.workspace_bytes(M, N, K, lda, ldb, ldc, 1, gi.F32)
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")          # zero-filled once, as required
    try:
        B.set_workspace(ws, need)
        for vn in ("umma_n128_sk4", "umma2_n256_sk2", "umma_n64"):
            vals, _, g = G.run_gemm(Ap, Bp, M, N, K, lda, ldb, ldc, gi.F32, variant=names[vn])
            assert g and oracle.check(vals[0], Cref, S, G.tol_for(gi.F32)).ok, vn
        small = torch.zeros(1 << 21, dtype=torch.uint8, device="cuda")   # header fits, the rest does not
        B.set_workspace(small, small.numel())
        dA = G.to_device_bits(gi.embed(bits(np.ones((600, 1030))), 1031))
        dB = G.to_device_bits(gi.embed(bits(np.ones((1030, 3000))), 3003))
        dC = torch.zeros(600 * 3000, dtype=torch.float32, device="cuda")
        st = B.gemm_bf16_variant(names["umma_n128_sk4"], dA, dB, dC, 600, 3000, 1030, 1031, 3003, 3000,
                                 0, 0, 0, 1, gi.F32, torch.cuda.current_stream(), check=False)
        assert st == B.ERR_WORKSPACE
        assert B.set_workspace(ws, 100, check=False) == B.ERR_WORKSPACE          # smaller than the header
        assert B.set_workspace(ws.data_ptr() + 8, need - 8, check=False) == B.ERR_WORKSPACE   # misaligned
    finally:
        B.set_workspace(None, 0)
    vals, _, g = G.run_gemm(Ap, Bp, M, N, K, lda, ldb, ldc, gi.F32, variant=names["umma_n128_sk4"])
    assert g and oracle.check(vals[0], Cref, S, G.tol_for(gi.F32)).ok          # internal workspace again


def test_two_streams_without_workspace_use():
    """Aligned, unsplit products need no workspace and may overlap on two streams."""
    names = _names()
    rng = np.random.default_rng(8)
    shapes = [(512, 768, 1024), (384, 1024, 640)]
    ops = []
    for (M, N, K) in shapes:
        A = bits(rng.standard_normal((M, K))); Bm = bits(rng.standard_normal((K, N)))
        ops.append((A, Bm, G.to_device_bits(A.ravel()), G.to_device_bits(Bm.ravel()),
                    torch.zeros(M * N, dtype=torch.float32, device="cuda")))
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for rep in range(10):
        for (M, N, K), (A, Bm, dA, dB, dC), st in zip(shapes, ops, streams):
            B.gemm_bf16_variant(names["umma_n128"], dA, dB, dC, M, N, K, K, N, N, 0, 0, 0, 1, gi.F32, st)
    torch.cuda.synchronize()
    for (M, N, K), (A, Bm, dA, dB, dC) in zip(shapes, ops):
        Cref, S = oracle.gemm(A, Bm, M, N, K)
        got = dC.cpu().numpy().reshape(M, N).astype(np.float64)
        assert oracle.check(got, Cref, S, G.tol_for(gi.F32)).ok
    assert B.device_status(torch.cuda.current_stream()) == (B.OK, 0)


@pytest.mark.parametrize("step", [2, 3])
def test_paper_task2_ladder_larger_sizes_closed_form(step):
    """The paper's Task 2 shapes A (size x 4096) x B (4096 x 2048) for size = 2^14
    and 2^16 rows, integer closed form on every element (fp32 output)."""
    cfg = gi.task2_ladder(step)
    u, v_, p, q = gi.rank1_int_factors(cfg.M, cfg.N, cfg.K, seed=40 + step)
    A = gi.int_to_bf16_bits(np.outer(u, p)).ravel()
    Bm = gi.int_to_bf16_bits(np.outer(q, v_)).ravel()
    dA = G.to_device_bits(A); dB = G.to_device_bits(Bm)
    del A
    dC = torch.full((cfg.M * cfg.N,), float("nan"), dtype=torch.float32, device="cuda")
    B.gemm_bf16(dA, dB, dC, cfg.M, cfg.N, cfg.K, cfg.K, cfg.N, cfg.N, gi.F32, torch.cuda.current_stream())
    assert B.device_status(torch.cuda.current_stream()) == (B.OK, 0)
    scale = float(np.dot(p, q))
    want = torch.outer(torch.from_numpy(u.astype(np.float32)).cuda(),
                       torch.from_numpy(v_.astype(np.float32)).cuda()) * scale      # exact in fp32
    assert torch.equal(dC.view(cfg.M, cfg.N), want)


def test_automatic_choice_follows_the_dispatch_table():
    """With an entry in the dispatch table the plain entry point runs that variant
    (here split-K kernels the cost model would not pick for the shape) and the
    result still agrees with the oracle; other shapes are untouched."""
    names = _names()
    rng = np.random.default_rng(5)
    M, N, K = 200, 330, 1030
    A = bits(rng.standard_normal((M, K))); Bm = bits(rng.standard_normal((K, N)))
    Cref, S = oracle.gemm(A, Bm, M, N, K)
    try:
        B.dispatch_clear()
        model = B.select_variant(M, N, K, K, N, N, 1, gi.F32)
        for forced in ("umma_n64_sk4", "umma2_n256_sk2", "umma_n128_sk2"):
            assert names[forced] != model
            B.dispatch_set(M, N, K, 1, gi.F32, names[forced])
            assert B.select_variant(M, N, K, K, N, N, 1, gi.F32) == names[forced]
            vals, raw, guards = G.run_gemm(A.ravel(), Bm.ravel(), M, N, K, K, N, N, gi.F32)      # automatic choice
            r = oracle.check(vals[0], Cref, S, G.tol_for(gi.F32))
            assert guards and r.ok, (forced, r)
        assert B.select_variant(M, N, K + 1, K + 1, N, N, 1, gi.F32) != -1
    finally:
        B.dispatch_clear()
