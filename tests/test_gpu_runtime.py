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
        small = torch.zeros(3 << 20, dtype=torch.uint8, device="cuda")   # the header (2 MiB + 256 B) fits, the rest does not
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
        # a class entry with knobs set: used for another shape of the same class, result still right
        B.dispatch_clear()
        code = B.variant_code(names["umma_n128_ts"], 1, 3)
        B.dispatch_set_class(M, N, K, 1, gi.F32, True, code)
        M2, N2, K2 = M - 3, N - 5, K - 5                              # same tile and k-block counts
        A2 = bits(rng.standard_normal((M2, K2))); B2 = bits(rng.standard_normal((K2, N2)))
        A2p, B2p = gi.embed(A2, K2 + 7), gi.embed(B2, N2 + 3)        # pitches that TMA can address
        assert (K2 + 7) % 8 == 0 and (N2 + 3) % 8 == 0
        assert B.select_variant(M2, N2, K2, K2 + 7, N2 + 3, N2, 1, gi.F32) == code
        vals, raw, guards = G.run_gemm(A2p, B2p, M2, N2, K2, K2 + 7, N2 + 3, N2, gi.F32)
        Cref2, S2 = oracle.gemm(A2, B2, M2, N2, K2)
        assert guards and oracle.check(vals[0], Cref2, S2, G.tol_for(gi.F32)).ok
    finally:
        B.dispatch_clear()
        B.dispatch_load_packaged()


def test_bounded_wait_runs_out_and_the_library_recovers():
    """The failure path of the kernels' bounded waits, without hanging anything: the wait
    limit is set to 1 ms and the next split launch raises its hand-over flags to a value
    nobody waits for.  Both units of a one-tile, two-unit product then give up after 1 ms,
    the kernel returns normally, the status word names the wait (epilogue role, flag wait),
    reading it clears the header, and the next ordinary call is correct."""
    names = _names()
    rng = np.random.default_rng(77)
    M, N, K = 128, 64, 256
    A = bits(rng.standard_normal((M, K))); Bm = bits(rng.standard_normal((K, N)))
    dA, dB = G.to_device_bits(A.ravel()), G.to_device_bits(Bm.ravel())
    dC = torch.zeros(M * N, dtype=torch.float32, device="cuda")
    s = torch.cuda.current_stream()
    assert B.device_status(s) == (B.OK, 0)
    try:
        B.debug_set(B.DEBUG_WAIT_LIMIT_NS, 1_000_000)
        B.debug_set(B.DEBUG_MISS_NEXT_SPLIT_FLAGS, 1)
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        st = B.gemm_bf16_variant(names["umma_n64_sk2"], dA, dB, dC, M, N, K, K, N, N, 0, 0, 0, 1, gi.F32, s,
                                 check=False)
        t1.record()
        assert st == B.OK                                  # the launch itself succeeds
        code, detail = B.device_status(s)                  # synchronises
        assert code == B.ERR_DEVICE_TIMEOUT
        assert detail >> 8 == 3 and detail & 0xFF == 0xC0  # epilogue role, wait for another unit's flag
        ms = t0.elapsed_time(t1)
        assert 0.9 <= ms < 500.0, ms                       # gave up after the 1 ms limit, not the default 2 s
        assert "bounded wait" in B.strerror(code)
        assert B.device_status(s) == (B.OK, 0)             # reading cleared it
    finally:
        B.debug_set(B.DEBUG_WAIT_LIMIT_NS, 0)
        B.debug_set(B.DEBUG_MISS_NEXT_SPLIT_FLAGS, 0)
    assert B.debug_set(99, 0, check=False) == B.ERR_INVALID_VARIANT
    # the same launch again, now with its flags as they should be
    Cref, S = oracle.gemm(A, Bm, M, N, K)
    for vn in ("umma_n64_sk2", "umma_n64"):
        vals, _, g = G.run_gemm(A.ravel(), Bm.ravel(), M, N, K, K, N, N, gi.F32, variant=names[vn])
        assert g and oracle.check(vals[0], Cref, S, G.tol_for(gi.F32)).ok, vn
    assert B.device_status(s) == (B.OK, 0)


def test_workspace_per_stream_lets_scratch_users_run_concurrently():
    """Two streams, each with a workspace of its own: products that repack their operands
    (odd pitches) and split tiles along K run on both at once and agree with the oracle;
    each stream has its own status word.  The grids are small enough to be resident together."""
    names = _names()
    rng = np.random.default_rng(91)
    shapes = [(300, 520, 1030, 1031, 523, 521), (260, 390, 1500, 1503, 391, 393)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    work, ops = [], []
    for (M, N, K, lda, ldb, ldc) in shapes:
        A = bits(rng.standard_normal((M, K))); Bm = bits(rng.standard_normal((K, N)))
        need = B.workspace_bytes(M, N, K, lda, ldb, ldc, 1, gi.F32)
        work.append(torch.zeros(need, dtype=torch.uint8, device="cuda"))
        ops.append((A, Bm, G.to_device_bits(gi.embed(A, lda)), G.to_device_bits(gi.embed(Bm, ldb)),
                    torch.zeros(M * ldc, dtype=torch.float32, device="cuda")))
    torch.cuda.synchronize()
    try:
        for st, ws in zip(streams, work):
            B.set_workspace_for_stream(st, ws, ws.numel())
        # a second stream may not be given (part of) the first stream's buffer; too small is refused
        assert B.set_workspace_for_stream(streams[1], work[0].data_ptr() + 256, work[0].numel() - 256,
                                          check=False) == B.ERR_WORKSPACE
        assert B.set_workspace_for_stream(streams[1], work[1], 100, check=False) == B.ERR_WORKSPACE
        for variant in ("umma_n64_sk2", "umma_n128_ts", "auto"):
            v = B.VARIANT_AUTO if variant == "auto" else names[variant]
            for rep in range(8):
                for (M, N, K, lda, ldb, ldc), (A, Bm, dA, dB, dC), st in zip(shapes, ops, streams):
                    B.gemm_bf16_variant(v, dA, dB, dC, M, N, K, lda, ldb, ldc, 0, 0, 0, 1, gi.F32, st)
            for st in streams:
                assert B.device_status(st) == (B.OK, 0), variant
            for (M, N, K, lda, ldb, ldc), (A, Bm, dA, dB, dC) in zip(shapes, ops):
                Cref, S = oracle.gemm(A, Bm, M, N, K)
                got = dC.cpu().numpy().reshape(M, ldc)[:, :N].astype(np.float64)
                assert oracle.check(got, Cref, S, G.tol_for(gi.F32)).ok, variant
                dC.zero_()
        # a call whose needs exceed the stream's workspace is refused, not grown
        bm, bn, bk = 2000, 3000, 4099                      # repacked operands alone: 41 MB
        assert 2 * (bm * bk + bk * bn) > work[0].numel()
        big = torch.ones(bm * (bk + 1), dtype=torch.int16, device="cuda")
        bigB = torch.ones(bk * (bn + 3), dtype=torch.int16, device="cuda")
        bigC = torch.zeros(bm * bn, dtype=torch.float32, device="cuda")
        assert B.gemm_bf16(big, bigB, bigC, bm, bn, bk, bk + 1, bn + 3, bn, gi.F32, streams[0],
                           check=False) == B.ERR_WORKSPACE
    finally:
        for st in streams:
            B.set_workspace_for_stream(st, None, 0)
        torch.cuda.synchronize()


def test_reserve_workspace_then_no_growth_and_shutdown_releases():
    """cudallm_reserve_workspace sizes the library's own workspace ahead of time: calls within
    that size then leave free device memory as it is; cudallm_shutdown gives it back and the
    library works again afterwards."""
    names = _names()
    rng = np.random.default_rng(5)
    M, N, K = 200, 300, 1030
    lda, ldb, ldc = K + 1, N + 3, N
    A = bits(rng.standard_normal((M, K))); Bm = bits(rng.standard_normal((K, N)))
    Ap, Bp = gi.embed(A, lda), gi.embed(Bm, ldb)
    Cref, S = oracle.gemm(A, Bm, M, N, K)
    need = B.workspace_bytes(M, N, K, lda, ldb, ldc, 1, gi.F32)
    B.reserve_workspace(need + (64 << 20))
    torch.cuda.synchronize()
    dA, dB = G.to_device_bits(Ap), G.to_device_bits(Bp)
    dC = torch.zeros(M * ldc, dtype=torch.float32, device="cuda")
    s = torch.cuda.current_stream()
    B.gemm_bf16_variant(names["umma_n128_sk4"], dA, dB, dC, M, N, K, lda, ldb, ldc, 0, 0, 0, 1, gi.F32, s)
    torch.cuda.synchronize()
    free = torch.cuda.mem_get_info()[0]
    for vn in ("umma_n128_sk4", "umma2_n256_sk2", "umma_n64"):
        B.gemm_bf16_variant(names[vn], dA, dB, dC, M, N, K, lda, ldb, ldc, 0, 0, 0, 1, gi.F32, s)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free
    assert B.shutdown() == B.OK
    assert torch.cuda.mem_get_info()[0] > free                      # the workspace went back
    vals, _, g = G.run_gemm(Ap, Bp, M, N, K, lda, ldb, ldc, gi.F32, variant=names["umma_n128_sk4"])
    assert g and oracle.check(vals[0], Cref, S, G.tol_for(gi.F32)).ok


def test_paper_task2_largest_size_closed_form():
    """The last step of the paper's Task 2 ladder, A (2^18 x 4096) x B (4096 x 2048): 2 GiB of A
    and of C.  Integer closed form on every element, checked on the device."""
    cfg = gi.task2_ladder(4)
    assert cfg.M == 1 << 18
    u, v_, p, q = gi.rank1_int_factors(cfg.M, cfg.N, cfg.K, seed=44)
    du = torch.from_numpy(u.astype(np.float32)).cuda()
    dA = torch.outer(du, torch.from_numpy(p.astype(np.float32)).cuda()).to(torch.bfloat16)      # exact: small integers
    dB = torch.outer(torch.from_numpy(q.astype(np.float32)).cuda(),
                     torch.from_numpy(v_.astype(np.float32)).cuda()).to(torch.bfloat16)
    dC = torch.full((cfg.M, cfg.N), float("nan"), dtype=torch.float32, device="cuda")
    B.gemm_bf16(dA, dB, dC, cfg.M, cfg.N, cfg.K, cfg.K, cfg.N, cfg.N, gi.F32, torch.cuda.current_stream())
    assert B.device_status(torch.cuda.current_stream()) == (B.OK, 0)
    scale = float(np.dot(p, q))
    dv = torch.from_numpy(v_.astype(np.float32)).cuda()
    rows = 1 << 14                                                   # compare in slabs to bound the temporaries
    for r0 in range(0, cfg.M, rows):
        want = torch.outer(du[r0:r0 + rows], dv) * scale             # exact in fp32
        assert torch.equal(dC[r0:r0 + rows], want), r0
    del dA, dC
    torch.cuda.empty_cache()
