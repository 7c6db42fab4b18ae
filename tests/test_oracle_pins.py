"""Pins for the CPU oracle: what the mathematics fixes about C = A x B
(Task 2 of the paper's benchmark table), checked without any GPU and without
calling the oracle against itself.  A dropped term, a wrong index, a swapped
operand or a transposed access in ``oracle_gemm.c`` fails at least one of
these."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2506_09092_b200 import inputs as gi

HERE = os.path.dirname(os.path.abspath(__file__))


def bits(x):
    return gi.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


# ---------------------------------------------------------------- literals --

def test_hand_computed_2x2():
    # [[1,2],[3,4]] x [[5,6],[7,8]] = [[19,22],[43,50]]
    A = bits([[1, 2], [3, 4]])
    B = bits([[5, 6], [7, 8]])
    for fn in (oracle.gemm, oracle.gemm_naive):
        C, S = fn(A, B, 2, 2, 2)
        assert C.tolist() == [[19.0, 22.0], [43.0, 50.0]]
        assert S.tolist() == [[19.0, 22.0], [43.0, 50.0]]


def test_hand_computed_2x3_3x2_with_signs():
    # [[1,-2,3],[0,4,-1]] x [[2,1],[-1,0],[0.5,-3]] = [[5.5,-8],[-4.5,3]]
    A = bits([[1, -2, 3], [0, 4, -1]])
    B = bits([[2, 1], [-1, 0], [0.5, -3]])
    for fn in (oracle.gemm, oracle.gemm_naive):
        C, S = fn(A, B, 2, 2, 3)
        assert C.tolist() == [[5.5, -8.0], [-4.5, 3.0]]
        # S = |A| x |B| : [[2+2+1.5, 1+0+9],[0+4+0.5, 0+0+3]]
        assert S.tolist() == [[5.5, 10.0], [4.5, 3.0]]


def test_hand_computed_inner_and_outer_product():
    a = bits([[1, 2, 3, 4]])
    b = bits([[1], [0.5], [-2], [0.25]])
    C, S = oracle.gemm(a, b, 1, 1, 4)
    assert C.item() == 1 + 1 - 6 + 1 and S.item() == 1 + 1 + 6 + 1
    C, _ = oracle.gemm(b, a, 4, 4, 1)      # outer product, K = 1
    assert C.tolist() == [[1, 2, 3, 4], [0.5, 1, 1.5, 2], [-2, -4, -6, -8], [0.25, 0.5, 0.75, 1]]


def test_not_symmetric_in_operands():
    # A x B != B x A for these; catches swapped roles of A and B
    A = bits([[0, 1], [0, 0]])
    B = bits([[0, 0], [1, 0]])
    C, _ = oracle.gemm(A, B, 2, 2, 2)
    assert C.tolist() == [[1.0, 0.0], [0.0, 0.0]]
    C, _ = oracle.gemm(B, A, 2, 2, 2)
    assert C.tolist() == [[0.0, 0.0], [0.0, 1.0]]


def test_golden_file_small_case():
    """A 3x4 by 4x2 product worked by hand and stored as text."""
    path = os.path.join(HERE, "golden", "task2_small_3x4x2.txt")
    rows = [ln.split("#")[0].strip() for ln in open(path)]
    rows = [r for r in rows if r]
    sect = {}
    cur = None
    for r in rows:
        if r.endswith(":"):
            cur = r[:-1]
            sect[cur] = []
        else:
            sect[cur].append([float(t) for t in r.split()])
    A, B, C = (np.array(sect[k]) for k in ("A", "B", "C"))
    Cr, _ = oracle.gemm(bits(A), bits(B), 3, 2, 4)
    assert np.array_equal(Cr, C)


# ------------------------------------------------- identity / permutation --

@pytest.mark.parametrize("M,N", [(5, 7), (64, 33), (130, 257)])
def test_identity_left_and_right(M, N):
    rng = np.random.default_rng(3)
    X = bits(rng.standard_normal((M, N)))
    Xd = oracle.bf16_bits_to_f64(X)
    C, S = oracle.gemm(gi.identity_bits(M, M), X, M, N, M)
    assert np.array_equal(C, Xd) and np.array_equal(S, np.abs(Xd))
    C, S = oracle.gemm(X, gi.identity_bits(N, N), M, N, N)
    assert np.array_equal(C, Xd) and np.array_equal(S, np.abs(Xd))


def test_rectangular_identity_selects_rows_and_pads_zero():
    # A = [I_3 | 0] (3x5): picks the first 3 rows of B (5x4)
    B = bits(np.arange(20).reshape(5, 4))
    C, _ = oracle.gemm(gi.identity_bits(3, 5), B, 3, 4, 5)
    assert np.array_equal(C, np.arange(12).reshape(3, 4).astype(np.float64))
    # A = [I_5 ; 0] (7x5): B followed by two zero rows
    C, _ = oracle.gemm(gi.identity_bits(7, 5), B, 7, 4, 5)
    assert np.array_equal(C[:5], np.arange(20).reshape(5, 4)) and not C[5:].any()


@pytest.mark.parametrize("n,N", [(17, 9), (96, 130)])
def test_permutation(n, N):
    P, pi = gi.permutation_bits(n, seed=5)
    rng = np.random.default_rng(9)
    X = bits(rng.standard_normal((n, N)))
    Xd = oracle.bf16_bits_to_f64(X)
    C, _ = oracle.gemm(P, X, n, N, n)         # row i of C = row pi[i] of X
    assert np.array_equal(C, Xd[pi])
    Y = bits(rng.standard_normal((N, n)))
    Yd = oracle.bf16_bits_to_f64(Y)
    C, _ = oracle.gemm(Y, P, N, n, n)         # C[:, pi[i]] = Y[:, i]
    expect = np.empty_like(Yd)
    expect[:, pi] = Yd
    assert np.array_equal(C, expect)


# -------------------------------------------------- integer closed forms --

@pytest.mark.parametrize("M,N,K", [(3, 5, 7), (70, 45, 300), (257, 129, 1000), (16, 300, 8192)])
def test_rank1_integer_closed_form(M, N, K):
    A, B, u, v, p, q = gi.rank1_int_operands(M, N, K, seed=M + N + K)
    C, S = oracle.gemm(A, B, M, N, K)
    assert np.array_equal(C, np.outer(u, v).astype(np.float64) * float(np.dot(p, q)))
    assert np.array_equal(S, np.outer(np.abs(u), np.abs(v)).astype(np.float64)
                          * float(np.dot(np.abs(p), np.abs(q))))


@pytest.mark.parametrize("K", [1, 15, 64, 65, 4096])
def test_ones_and_checkerboard(K):
    M, N = 6, 10
    ones_a, ones_b = bits(np.ones((M, K))), bits(np.ones((K, N)))
    C, S = oracle.gemm(ones_a, ones_b, M, N, K)
    assert np.all(C == K) and np.all(S == K)
    alt = (-1.0) ** np.arange(K)
    Aa = bits(np.tile(alt, (M, 1)))
    Ba = bits(np.tile(alt[:, None], (1, N)))
    C, _ = oracle.gemm(Aa, Ba, M, N, K)
    assert np.all(C == K)
    C, S = oracle.gemm(Aa, ones_b, M, N, K)
    assert np.all(C == (K % 2)) and np.all(S == K)


@pytest.mark.parametrize("k0", [0, 15, 16, 63, 64, 199])
def test_k_marker(k0):
    M, N, K = 4, 5, 200
    Bm = np.zeros((K, N))
    Bm[k0] = np.arange(1, N + 1)
    Am = np.zeros((M, K))
    Am[:, k0] = np.arange(1, M + 1)
    Am += 0  # other columns zero: only k0 contributes
    C, _ = oracle.gemm(bits(Am), bits(Bm), M, N, K)
    assert np.array_equal(C, np.outer(np.arange(1, M + 1), np.arange(1, N + 1)).astype(float))


def test_row_col_index_map():
    M, N, K = 37, 53, 9
    Am = np.zeros((M, K)); Am[:, 0] = np.arange(M)
    Bm = np.zeros((K, N)); Bm[0] = np.arange(N)
    C, _ = oracle.gemm(bits(Am), bits(Bm), M, N, K)
    assert np.array_equal(C, np.outer(np.arange(M), np.arange(N)).astype(float))


# ------------------------------------------------ library special case ----

@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (33, 65, 129), (256, 256, 256), (300, 200, 1100)])
def test_against_fp64_library_product(M, N, K):
    rng = np.random.default_rng(M * 7 + N)
    A = bits(rng.standard_normal((M, K)))
    B = bits(rng.uniform(-1, 1, (K, N)))
    C, S = oracle.gemm(A, B, M, N, K)
    Ad, Bd = oracle.bf16_bits_to_f64(A), oracle.bf16_bits_to_f64(B)
    # same sum in another order: differs by at most ~K * 2^-53 * S
    bound = 2.0 * K * 2.0 ** -53 * S + 1e-300
    assert np.all(np.abs(C - Ad @ Bd) <= bound)
    Ct = (torch.from_numpy(Ad) @ torch.from_numpy(Bd)).numpy()
    assert np.all(np.abs(C - Ct) <= bound)
    assert np.all(np.abs(S - np.abs(Ad) @ np.abs(Bd)) <= bound)


# ----------------------------------------------------------- brute force --

@pytest.mark.parametrize("seed", range(6))
def test_two_loop_orders_agree_bitwise(seed):
    rng = np.random.default_rng(seed)
    M, N, K = (int(x) for x in rng.integers(1, 65, size=3))
    A = bits(rng.standard_normal((M, K)))
    B = bits(rng.standard_normal((K, N)))
    C1, S1 = oracle.gemm(A, B, M, N, K)
    C2, S2 = oracle.gemm_naive(A, B, M, N, K)
    assert C1.tobytes() == C2.tobytes() and S1.tobytes() == S2.tobytes()


def test_python_loop_brute_force():
    rng = np.random.default_rng(42)
    M, N, K = 4, 3, 5
    A = bits(rng.standard_normal((M, K)))
    B = bits(rng.standard_normal((K, N)))
    Ad, Bd = oracle.bf16_bits_to_f64(A).tolist(), oracle.bf16_bits_to_f64(B).tolist()
    C, S = oracle.gemm(A, B, M, N, K)
    for i in range(M):
        for j in range(N):
            c = 0.0
            s = 0.0
            for k in range(K):
                c += Ad[i][k] * Bd[k][j]
                s += abs(Ad[i][k]) * abs(Bd[k][j])
            assert C[i, j] == c and S[i, j] == s


# ------------------------------------------------ strides / rows / batch --

def test_leading_dimensions_and_padding_ignored():
    rng = np.random.default_rng(1)
    M, N, K = 9, 11, 13
    A = bits(rng.standard_normal((M, K)))
    B = bits(rng.standard_normal((K, N)))
    C0, S0 = oracle.gemm(A, B, M, N, K)
    Ap = gi.embed(A, ld=K + 3)           # NaN padding must never be read
    Bp = gi.embed(B, ld=N + 8)
    C1, S1 = oracle.gemm(Ap, Bp, M, N, K, lda=K + 3, ldb=N + 8)
    assert C0.tobytes() == C1.tobytes() and S0.tobytes() == S1.tobytes()
    Cn, _ = oracle.gemm_naive(Ap, Bp, M, N, K, lda=K + 3, ldb=N + 8)
    assert C0.tobytes() == Cn.tobytes()


def test_rows_subset_matches_definition():
    rng = np.random.default_rng(2)
    M, N, K = 40, 17, 23
    A = bits(rng.standard_normal((M, K)))
    B = bits(rng.standard_normal((K, N)))
    Ad, Bd = oracle.bf16_bits_to_f64(A), oracle.bf16_bits_to_f64(B)
    rows = [39, 0, 7, 7, 12]
    C, S = oracle.gemm_rows(A, B, rows, N, K)
    bound = 2.0 * K * 2.0 ** -53 * S
    assert np.all(np.abs(C - Ad[rows] @ Bd) <= bound)
    # identity pin on the row selector itself
    I = gi.identity_bits(M, M)
    X = bits(rng.standard_normal((M, N)))
    C, _ = oracle.gemm_rows(I, X, rows, N, M)
    assert np.array_equal(C, oracle.bf16_bits_to_f64(X)[rows])


def test_batched_items_are_independent_products():
    rng = np.random.default_rng(4)
    M, N, K, batch = 5, 6, 7, 4
    lda, ldb = K + 1, N + 2
    sA, sB = M * lda + 3, K * ldb + 5
    A = np.full((batch - 1) * sA + M * lda, 0x7FC0, dtype=np.uint16)
    B = np.full((batch - 1) * sB + K * ldb, 0x7FC0, dtype=np.uint16)
    items = []
    for t in range(batch):
        a = bits(rng.standard_normal((M, K))); b = bits(rng.standard_normal((K, N)))
        items.append((a, b))
        np.lib.stride_tricks.as_strided(A[t * sA:], (M, K), (lda * 2, 2))[...] = a
        np.lib.stride_tricks.as_strided(B[t * sB:], (K, N), (ldb * 2, 2))[...] = b
    C, S = oracle.gemm_batched(A, B, M, N, K, lda, ldb, sA, sB, batch)
    for t, (a, b) in enumerate(items):
        bound = 2.0 * K * 2.0 ** -53 * S[t]
        assert np.all(np.abs(C[t] - oracle.bf16_bits_to_f64(a) @ oracle.bf16_bits_to_f64(b)) <= bound)
    # batch item with identity A returns B's item
    Ai = np.concatenate([gi.identity_bits(3, 3).ravel()] * 2)
    Bi = bits(np.arange(18).reshape(2, 3, 3)).ravel()
    C, _ = oracle.gemm_batched(Ai, Bi, 3, 3, 3, 3, 3, 9, 9, 2)
    assert np.array_equal(C, np.arange(18).reshape(2, 3, 3).astype(float))


def test_degenerate_sizes():
    A = bits(np.ones((3, 4))); B = bits(np.ones((4, 5)))
    C, S = oracle.gemm(A, B, 3, 5, 0)        # K = 0: empty sum
    assert C.shape == (3, 5) and not C.any() and not S.any()
    C, S = oracle.gemm(A, B, 0, 5, 4)
    assert C.shape == (0, 5)
    C, S = oracle.gemm(A, B, 3, 0, 4)
    assert C.shape == (3, 0)


# ------------------------------------------------------------- invariants --

def test_power_of_two_scaling_is_exact():
    rng = np.random.default_rng(8)
    M, N, K = 20, 30, 70
    Af = rng.standard_normal((M, K)).astype(np.float32)
    Bf = rng.standard_normal((K, N)).astype(np.float32)
    A, B = bits(Af), bits(Bf)
    C, S = oracle.gemm(A, B, M, N, K)
    for p in (-3, 4):
        A2 = bits(gi.bf16_bits_to_f32(A) * np.float32(2.0 ** p))
        C2, S2 = oracle.gemm(A2, B, M, N, K)
        assert np.array_equal(C2, C * 2.0 ** p) and np.array_equal(S2, S * 2.0 ** p)


def test_transpose_identity_exact():
    rng = np.random.default_rng(10)
    M, N, K = 13, 21, 34
    A = bits(rng.standard_normal((M, K)))
    B = bits(rng.standard_normal((K, N)))
    C, S = oracle.gemm(A, B, M, N, K)
    Ct, St = oracle.gemm(np.ascontiguousarray(B.T), np.ascontiguousarray(A.T), N, M, K)
    assert np.array_equal(Ct.T, C) and np.array_equal(St.T, S)


def test_zero_padding_and_row_permutation_invariance():
    rng = np.random.default_rng(11)
    M, N, K = 10, 12, 14
    A = bits(rng.standard_normal((M, K)))
    B = bits(rng.standard_normal((K, N)))
    C, _ = oracle.gemm(A, B, M, N, K)
    Ap = np.zeros((M + 3, K + 5), dtype=np.uint16); Ap[:M, :K] = A
    Bp = np.zeros((K + 5, N + 2), dtype=np.uint16); Bp[:K, :N] = B
    Cp, _ = oracle.gemm(Ap, Bp, M + 3, N + 2, K + 5)
    assert np.array_equal(Cp[:M, :N], C) and not Cp[M:].any() and not Cp[:, N:].any()
    pi = rng.permutation(M)
    Cq, _ = oracle.gemm(np.ascontiguousarray(A[pi]), B, M, N, K)
    assert np.array_equal(Cq, C[pi])


def test_S_is_product_of_absolute_values_and_dominates():
    rng = np.random.default_rng(12)
    M, N, K = 15, 16, 50
    A = bits(rng.standard_normal((M, K)))
    B = bits(rng.standard_normal((K, N)))
    C, S = oracle.gemm(A, B, M, N, K)
    Cabs, _ = oracle.gemm(A & np.uint16(0x7FFF), B & np.uint16(0x7FFF), M, N, K)
    assert np.array_equal(S, Cabs) and np.all(S >= np.abs(C))


# ------------------------------------------------------- bf16 conversions --

def test_bf16_widening_matches_torch():
    allbits = np.arange(1 << 16, dtype=np.uint16)
    ours = oracle.bf16_bits_to_f64(allbits)
    t = torch.from_numpy(allbits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(ours, t, equal_nan=True)


def _torch_bf16_bits(x32):
    t = torch.from_numpy(np.ascontiguousarray(x32, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def test_f32_to_bf16_rne_matches_torch_stratified():
    rng = np.random.default_rng(0)
    u = rng.integers(0, 1 << 32, size=1 << 22, dtype=np.uint64).astype(np.uint32)
    # all patterns adjacent to every tie: low half = 0x7FFF, 0x8000, 0x8001
    hi = np.arange(1 << 16, dtype=np.uint32) << np.uint32(16)
    ties = np.concatenate([hi | np.uint32(l) for l in (0x0000, 0x7FFF, 0x8000, 0x8001, 0xFFFF)])
    u = np.concatenate([u, ties])
    f = u.view(np.float32)
    finite = np.isfinite(f)
    for fn in (oracle.f32_to_bf16_bits, gi.f32_to_bf16_bits):
        assert np.array_equal(fn(f[finite]), _torch_bf16_bits(f[finite]))
    # NaN stays NaN, Inf stays Inf (oracle-side routine only)
    o = oracle.f32_to_bf16_bits(f[~finite])
    w = oracle.bf16_bits_to_f64(o)
    assert np.array_equal(np.isnan(w), np.isnan(f[~finite])) and np.array_equal(np.isinf(w), np.isinf(f[~finite]))


def test_f64_to_bf16_single_rounding():
    # explicit ties in [256, 512): spacing 2, odd integers are ties -> even mantissa
    vals = np.array([257.0, 259.0, 258.0, 261.0, 511.0, -257.0, 0.0, -0.0, 1.0, 65025.0,
                     3.0e38, 3.4e38, 1e-40, 2.0 ** -133, 2.0 ** -134, 2.0 ** -126])
    got = oracle.bf16_bits_to_f64(oracle.f64_to_bf16_bits(vals))
    assert got[:6].tolist() == [256.0, 260.0, 258.0, 260.0, 512.0, -256.0]
    assert got[6] == 0 and got[7] == 0 and np.signbit(got[7]) and got[8] == 1.0
    assert got[9] == 65024.0 or got[9] == 65280.0  # 65025 lies between 65024 and 65280 (spacing 256)
    assert got[9] == 65024.0
    # agreement with torch on every fp32-representable value sampled (fp64 -> fp32 exact there)
    rng = np.random.default_rng(5)
    u = rng.integers(0, 1 << 32, size=1 << 20, dtype=np.uint64).astype(np.uint32)
    f = u.view(np.float32)
    f = f[np.isfinite(f)]
    assert np.array_equal(oracle.f64_to_bf16_bits(f.astype(np.float64)), _torch_bf16_bits(f))
    # a value that double rounding (fp64 -> fp32 -> bf16) gets wrong: 1 + 2^-8 + 2^-30
    x = 1.0 + 2.0 ** -8 + 2.0 ** -30      # above the tie -> rounds up
    assert oracle.bf16_bits_to_f64(oracle.f64_to_bf16_bits(np.array([x])))[0] == 1.0 + 2.0 ** -7
    assert np.isinf(oracle.bf16_bits_to_f64(oracle.f64_to_bf16_bits(np.array([3.4e38]))))[0]


# ------------------------------------------------------------- acceptance --

def test_check_rule():
    Cref = np.array([[10.0, 0.0], [-5.0, 1.0]])
    S = np.array([[20.0, 0.0], [5.0, 1.0]])
    assert oracle.check(Cref.copy(), Cref, S, 1e-3)
    g = Cref.copy(); g[0, 0] += 0.019        # 0.95e-3 * S
    assert oracle.check(g, Cref, S, 1e-3)
    g[0, 0] = 10.0 + 0.021                   # 1.05e-3 * S
    r = oracle.check(g, Cref, S, 1e-3)
    assert not r and r.n_bad == 1 and r.argmax == (0, 0)
    g = Cref.copy(); g[0, 1] = 1e-30         # S == 0 demands equality
    assert not oracle.check(g, Cref, S, 1e-3)
    g = Cref.copy(); g[0, 1] = -0.0          # -0 == +0
    assert oracle.check(g, Cref, S, 1e-3)
    g = Cref.copy(); g[1, 1] = np.nan
    assert not oracle.check(g, Cref, S, 1e-3)


# --------------------------------------------- float32 operands (Task 2) ----

def test_f32_hand_computed_and_golden():
    A = np.array([[1, 2], [3, 4]], dtype=np.float32)
    Bm = np.array([[5, 6], [7, 8]], dtype=np.float32)
    for naive in (False, True):
        C, S = oracle.gemm_f32(A, Bm, 2, 2, 2, naive=naive)
        assert C.tolist() == [[19.0, 22.0], [43.0, 50.0]] and S.tolist() == C.tolist()
    A = np.array([[1, -2, 3], [0, 4, -1]], dtype=np.float32)
    Bm = np.array([[2, 1], [-1, 0], [0.5, -3]], dtype=np.float32)
    C, S = oracle.gemm_f32(A, Bm, 2, 2, 3)
    assert C.tolist() == [[5.5, -8.0], [-4.5, 3.0]] and S.tolist() == [[5.5, 10.0], [4.5, 3.0]]
    # a value that needs all 24 bits: (1 + 2^-23) * (1 - 2^-23) = 1 - 2^-46 exactly in fp64
    a = np.array([[1 + 2.0 ** -23]], dtype=np.float32); b = np.array([[1 - 2.0 ** -23]], dtype=np.float32)
    C, _ = oracle.gemm_f32(a, b, 1, 1, 1)
    assert C.item() == 1.0 - 2.0 ** -46


def test_f32_identity_permutation_and_roles():
    rng = np.random.default_rng(1)
    M, N = 33, 47
    X = rng.standard_normal((M, N)).astype(np.float32)
    C, S = oracle.gemm_f32(np.eye(M, dtype=np.float32), X, M, N, M)
    assert np.array_equal(C, X.astype(np.float64)) and np.array_equal(S, np.abs(X).astype(np.float64))
    C, _ = oracle.gemm_f32(X, np.eye(N, dtype=np.float32), M, N, N)
    assert np.array_equal(C, X.astype(np.float64))
    pi = rng.permutation(M)
    P = np.zeros((M, M), dtype=np.float32); P[np.arange(M), pi] = 1
    C, _ = oracle.gemm_f32(P, X, M, N, M)
    assert np.array_equal(C, X[pi].astype(np.float64))
    A = np.array([[0, 1], [0, 0]], dtype=np.float32); Bm = np.array([[0, 0], [1, 0]], dtype=np.float32)
    assert oracle.gemm_f32(A, Bm, 2, 2, 2)[0].tolist() == [[1.0, 0.0], [0.0, 0.0]]
    assert oracle.gemm_f32(Bm, A, 2, 2, 2)[0].tolist() == [[0.0, 0.0], [0.0, 1.0]]


@pytest.mark.parametrize("M,N,K", [(3, 5, 7), (70, 45, 300), (16, 300, 4096)])
def test_f32_rank1_integer_closed_form(M, N, K):
    u, v, p, q = gi.rank1_int_factors(M, N, K, seed=M + K, umax=20, pmax=3)   # entries up to 60: not bf16-exact
    A = np.outer(u, p).astype(np.float32); Bm = np.outer(q, v).astype(np.float32)
    C, S = oracle.gemm_f32(A, Bm, M, N, K)
    assert np.array_equal(C, np.outer(u, v).astype(np.float64) * float(np.dot(p, q)))
    assert np.array_equal(S, np.outer(np.abs(u), np.abs(v)).astype(np.float64) * float(np.dot(np.abs(p), np.abs(q))))


def test_f32_library_loop_orders_strides_rows():
    rng = np.random.default_rng(6)
    M, N, K = 41, 29, 130
    A = rng.standard_normal((M, K)).astype(np.float32); Bm = rng.uniform(-1, 1, (K, N)).astype(np.float32)
    C, S = oracle.gemm_f32(A, Bm, M, N, K)
    bound = 2.0 * K * 2.0 ** -53 * S + 1e-300
    assert np.all(np.abs(C - A.astype(np.float64) @ Bm.astype(np.float64)) <= bound)
    Ct = (torch.from_numpy(A).double() @ torch.from_numpy(Bm).double()).numpy()
    assert np.all(np.abs(C - Ct) <= bound)
    Cn, Sn = oracle.gemm_f32(A, Bm, M, N, K, naive=True)
    assert C.tobytes() == Cn.tobytes() and S.tobytes() == Sn.tobytes()
    # leading dimensions with NaN padding
    Ap = np.full(M * (K + 3), np.nan, dtype=np.float32); Ap.reshape(M, K + 3)[:, :K] = A
    Bp = np.full(K * (N + 5), np.nan, dtype=np.float32); Bp.reshape(K, N + 5)[:, :N] = Bm
    C2, S2 = oracle.gemm_f32(Ap, Bp, M, N, K, lda=K + 3, ldb=N + 5)
    assert C.tobytes() == C2.tobytes() and S.tobytes() == S2.tobytes()
    rows = [40, 0, 7, 7]
    Cr, Sr = oracle.gemm_f32_rows(A, Bm, rows, N, K)
    assert np.array_equal(Cr, C[rows]) and np.array_equal(Sr, S[rows])
    # bf16-representable inputs: the fp32 oracle and the bf16 oracle agree bit for bit
    Ab = gi.f32_to_bf16_bits(A); Bb = gi.f32_to_bf16_bits(Bm)
    C16, S16 = oracle.gemm(Ab, Bb, M, N, K)
    C32, S32 = oracle.gemm_f32(gi.bf16_bits_to_f32(Ab), gi.bf16_bits_to_f32(Bb), M, N, K)
    assert C16.tobytes() == C32.tobytes() and S16.tobytes() == S32.tobytes()
    # degenerate K
    C0, S0 = oracle.gemm_f32(A, Bm, M, N, 0)
    assert not C0.any() and not S0.any()
