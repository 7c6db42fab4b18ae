"""Seeded random shapes, leading dimensions, output types and variants against
the fp64 oracle: short and wide, small and square, tall and deep, very short.
Complements the fixed grids of test_gpu_parity.py with shapes nobody chose."""
import numpy as np
import pytest

import gpu_util as G
import oracle
from paper_2506_09092_b200 import binding as B
from paper_2506_09092_b200 import inputs as gi

pytestmark = pytest.mark.gpu


def bits(x):
    return gi.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def draw_shape(rng, kind):
    if kind == 0:
        return rng.integers(1, 80), rng.integers(1, 1500), rng.integers(1, 1200)
    if kind == 1:
        return rng.integers(1, 700), rng.integers(1, 700), rng.integers(1, 700)
    if kind == 2:
        return rng.integers(100, 1200), rng.integers(1, 300), rng.integers(64, 3000)
    return rng.integers(1, 20), rng.integers(500, 6000), rng.integers(1, 400)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes(seed):
    rng = np.random.default_rng(seed)
    nv = B.num_variants()
    for it in range(40):
        M, N, K = (int(x) for x in draw_shape(rng, it % 4))
        mode = it % 3                      # dense / padded to multiples of 8 / arbitrary padding
        if mode == 0:
            lda, ldb, ldc = K, N, N
        elif mode == 1:
            lda, ldb, ldc = (K + 7) // 8 * 8 + 8, (N + 7) // 8 * 8 + 8, (N + 7) // 8 * 8 + 8
        else:
            lda, ldb, ldc = K + int(rng.integers(0, 5)), N + int(rng.integers(0, 5)), N + int(rng.integers(0, 5))
        out_dtype = int(rng.integers(0, 2))
        A = gi.embed(bits(rng.standard_normal((M, K))), lda)
        Bm = gi.embed(bits(rng.uniform(-1, 1, (K, N))), ldb)
        Cref, S = oracle.gemm(A, Bm, M, N, K, lda, ldb)
        cands = [v for v in range(1, nv) if B.variant_supports(v, M, N, K, lda, ldb, ldc, 1, out_dtype) == 1]
        picks = [B.VARIANT_AUTO] + [int(x) for x in rng.choice(cands, size=min(3, len(cands)), replace=False)]
        for v in picks:
            vals, raw, guards = G.run_gemm(A, Bm, M, N, K, lda, ldb, ldc, out_dtype, variant=v)
            r = oracle.check(vals[0], Cref, S, G.tol_for(out_dtype))
            name = B.variant_name(v) if v >= 0 else "auto"
            assert guards, f"padding or guard band overwritten ({name}, {(M, N, K)}, {(lda, ldb, ldc)})"
            assert r.ok, (name, M, N, K, lda, ldb, ldc, out_dtype, r)
