"""CPU oracle for C = A x B on bfloat16 operands (the paper's Task 2, matrix
multiplication), with fp64 accumulation.

THIS PACKAGE IS TEST INFRASTRUCTURE.  Only the test-suite, the smoke check and
the benchmark's CPU-baseline leg may import it; the CUDA library never does, and
this package imports nothing from the CUDA side.

Contents
--------
* ``gemm`` / ``gemm_naive`` / ``gemm_rows`` / ``gemm_batched`` -- thin ctypes
  wrappers over ``oracle_gemm.c`` (the plain triple loop, in two loop orders);
  ``gemm_f32`` / ``gemm_f32_rows`` -- the same for float32 operands.
* ``bf16_bits_to_f64`` / ``f64_to_bf16_bits`` -- exact widening and
  round-to-nearest-even narrowing, written with integer bit operations.
* ``transpose_f32`` / ``sum_f32`` / ``dot_f32`` / ``layernorm_f32`` -- the
  paper's Tasks 8, 14, 15 and 4 on float32 arrays (``oracle_tasks.c``).
* ``check`` -- the element-wise acceptance rule
  ``|C_gpu - C_ref| <= tol * S`` with ``S = sum_k |a_ik| |b_kj|``.

parity unpinned: nothing (see tests/test_oracle_pins.py).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRCS = [os.path.join(_HERE, f) for f in ("oracle_gemm.c", "oracle_mhsa.c", "oracle_tasks.c")]
_SRC = _SRCS[0]
_LIB = os.path.join(_HERE, "liboracle_gemm.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile ``oracle_gemm.c`` with gcc into ``liboracle_gemm.so`` beside it."""
    with _lock:
        if (not force and os.path.exists(_LIB)
                and all(os.path.getmtime(_LIB) >= os.path.getmtime(f) for f in _SRCS)):
            return _LIB
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared",
               "-std=c11", "-Wall", "-o", tmp] + _SRCS + ["-lm"]
        subprocess.run(cmd, check=True, capture_output=True, text=True)
        os.replace(tmp, _LIB)
        return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB)
    u16p = ctypes.POINTER(ctypes.c_uint16)
    f64p = ctypes.POINTER(ctypes.c_double)
    i64 = ctypes.c_int64
    i64p = ctypes.POINTER(ctypes.c_int64)
    for name in ("oracle_gemm_bf16", "oracle_gemm_bf16_naive"):
        fn = getattr(lib, name)
        fn.argtypes = [u16p, u16p, f64p, f64p, i64, i64, i64, i64, i64]
        fn.restype = None
    lib.oracle_gemm_bf16_rows.argtypes = [u16p, u16p, f64p, f64p, i64p, i64,
                                          i64, i64, i64, i64]
    lib.oracle_gemm_bf16_rows.restype = None
    lib.oracle_gemm_bf16_batched.argtypes = [u16p, u16p, f64p, f64p, i64, i64,
                                             i64, i64, i64, i64, i64, i64]
    lib.oracle_gemm_bf16_batched.restype = None
    f32p = ctypes.POINTER(ctypes.c_float)
    for name in ("oracle_gemm_f32", "oracle_gemm_f32_naive"):
        fn = getattr(lib, name)
        fn.argtypes = [f32p, f32p, f64p, f64p, i64, i64, i64, i64, i64]
        fn.restype = None
    lib.oracle_gemm_f32_rows.argtypes = [f32p, f32p, f64p, f64p, i64p, i64, i64, i64, i64, i64]
    lib.oracle_gemm_f32_rows.restype = None
    lib.oracle_mhsa_bf16.argtypes = [u16p, u16p, u16p, f64p, f64p] + [i64] * 6
    lib.oracle_mhsa_bf16.restype = ctypes.c_int
    lib.oracle_transpose_f32.argtypes = [f32p, f32p, i64, i64, i64, i64]
    lib.oracle_transpose_f32.restype = None
    lib.oracle_sum_f32.argtypes = [f32p, i64, f64p]
    lib.oracle_sum_f32.restype = ctypes.c_double
    lib.oracle_dot_f32.argtypes = [f32p, f32p, i64, f64p]
    lib.oracle_dot_f32.restype = ctypes.c_double
    lib.oracle_layernorm_f32.argtypes = [f32p, f32p, f32p, f64p, i64, i64, ctypes.c_double, f64p, f64p]
    lib.oracle_layernorm_f32.restype = None
    lib.oracle_num_threads.restype = ctypes.c_int
    lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
    _lib = lib
    return lib


def num_threads() -> int:
    """Host threads the parallel loops use (OpenMP's current maximum)."""
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def _u16(a: np.ndarray) -> np.ndarray:
    a = np.asarray(a)
    if a.dtype != np.uint16:
        raise TypeError("operands are bfloat16 bit patterns: dtype must be uint16")
    return a


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _operand_view(X: np.ndarray, rows: int, cols: int, ld: int | None):
    """Return (uint16 array whose data pointer is element [0][0], leading
    dimension in elements) for a ``rows x cols`` row-major operand.

    ``X`` is either 2-D (a view with unit column stride is used in place, its
    row stride becoming the leading dimension) or flat with an explicit ``ld``.
    """
    X = _u16(X)
    if X.ndim == 2:
        if X.shape[0] < rows or X.shape[1] < cols:
            raise ValueError("operand smaller than rows x cols")
        if X.strides[1] != 2 or X.strides[0] % 2 or X.strides[0] < 0:
            X = np.ascontiguousarray(X)
        ldx = X.strides[0] // 2
        if X.shape[0] <= 1 or ldx == 0:
            ldx = max(X.shape[1], cols, 1)
        if ld is not None and ld != ldx and X.shape[0] > 1:
            raise ValueError("ld does not match the 2-D operand's row stride")
        return X, ldx
    if X.ndim != 1:
        raise ValueError("operand must be 1-D (with ld) or 2-D")
    if ld is None:
        ld = max(cols, 1)
    if ld < cols:
        raise ValueError("ld smaller than the row length")
    need = (rows - 1) * ld + cols if rows > 0 and cols > 0 else 0
    if X.size < need:
        raise ValueError("flat operand too small for rows, cols, ld")
    return np.ascontiguousarray(X), ld


def gemm(A, B, M, N, K, lda=None, ldb=None, want_S=True):
    """C_ref (and S) as fp64 ``M x N`` arrays for row-major bf16 operands.

    ``A``/``B`` hold bfloat16 bit patterns (uint16), either 2-D or flat with
    ``lda``/``ldb`` in elements.  Definition: Task 2, C[i][j] = sum_k A[i][k] B[k][j].
    """
    lib = _load()
    Ab, lda = _operand_view(A, M, K, lda)
    Bb, ldb = _operand_view(B, K, N, ldb)
    C = np.empty((M, N), dtype=np.float64)
    S = np.empty((M, N), dtype=np.float64) if want_S else None
    lib.oracle_gemm_bf16(_ptr(Ab, ctypes.c_uint16), _ptr(Bb, ctypes.c_uint16),
                         _ptr(C, ctypes.c_double),
                         _ptr(S, ctypes.c_double) if want_S else None,
                         M, N, K, lda, ldb)
    return (C, S) if want_S else C


def gemm_naive(A, B, M, N, K, lda=None, ldb=None):
    """Brute force (i-j-k scalar loop); tiny shapes only.  Returns (C_ref, S)."""
    lib = _load()
    Ab, lda = _operand_view(A, M, K, lda)
    Bb, ldb = _operand_view(B, K, N, ldb)
    C = np.empty((M, N), dtype=np.float64)
    S = np.empty((M, N), dtype=np.float64)
    lib.oracle_gemm_bf16_naive(_ptr(Ab, ctypes.c_uint16), _ptr(Bb, ctypes.c_uint16),
                               _ptr(C, ctypes.c_double), _ptr(S, ctypes.c_double),
                               M, N, K, lda, ldb)
    return C, S


def gemm_rows(A, B, rows, N, K, lda=None, ldb=None):
    """Rows ``rows`` of the product only.  Returns (C_ref, S), each ``len(rows) x N``."""
    lib = _load()
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    Mmax = int(rows.max()) + 1 if rows.size else 0
    Ab, lda = _operand_view(A, Mmax, K, lda)
    Bb, ldb = _operand_view(B, K, N, ldb)
    C = np.empty((rows.size, N), dtype=np.float64)
    S = np.empty((rows.size, N), dtype=np.float64)
    lib.oracle_gemm_bf16_rows(_ptr(Ab, ctypes.c_uint16), _ptr(Bb, ctypes.c_uint16),
                              _ptr(C, ctypes.c_double), _ptr(S, ctypes.c_double),
                              _ptr(rows, ctypes.c_int64), rows.size, N, K, lda, ldb)
    return C, S


def gemm_batched(A, B, M, N, K, lda, ldb, strideA, strideB, batch):
    """``batch`` independent products from flat buffers with element strides.
    Returns (C_ref, S), each ``batch x M x N``."""
    lib = _load()
    Ab = np.ascontiguousarray(_u16(A)).reshape(-1)
    Bb = np.ascontiguousarray(_u16(B)).reshape(-1)
    if batch > 0 and M > 0 and K > 0:
        assert Ab.size >= (batch - 1) * strideA + (M - 1) * lda + K
    if batch > 0 and N > 0 and K > 0:
        assert Bb.size >= (batch - 1) * strideB + (K - 1) * ldb + N
    C = np.empty((batch, M, N), dtype=np.float64)
    S = np.empty((batch, M, N), dtype=np.float64)
    lib.oracle_gemm_bf16_batched(_ptr(Ab, ctypes.c_uint16), _ptr(Bb, ctypes.c_uint16),
                                 _ptr(C, ctypes.c_double), _ptr(S, ctypes.c_double),
                                 M, N, K, lda, ldb, strideA, strideB, batch)
    return C, S


# --------------------------------------------------------------------------
# fp32 operands (the paper's Task 2 as printed)

def _f32_view(X, rows, cols, ld):
    X = np.asarray(X)
    if X.dtype != np.float32:
        raise TypeError("operands are float32")
    if X.ndim == 2:
        if X.shape[0] < rows or X.shape[1] < cols:
            raise ValueError("operand smaller than rows x cols")
        if X.strides[1] != 4 or X.strides[0] % 4 or X.strides[0] < 0:
            X = np.ascontiguousarray(X)
        ldx = X.strides[0] // 4 if X.shape[0] > 1 else max(X.shape[1], cols, 1)
        return X, (ldx or max(cols, 1))
    ld = max(cols, 1) if ld is None else ld
    need = (rows - 1) * ld + cols if rows > 0 and cols > 0 else 0
    if X.ndim != 1 or ld < cols or X.size < need:
        raise ValueError("flat float32 operand does not fit rows, cols, ld")
    return np.ascontiguousarray(X), ld


def gemm_f32(A, B, M, N, K, lda=None, ldb=None, naive=False):
    """(C_ref, S) in fp64 for row-major float32 operands (Task 2 as the paper
    states it).  ``naive=True`` runs the scalar i-j-k brute force."""
    lib = _load()
    Ab, lda = _f32_view(A, M, K, lda)
    Bb, ldb = _f32_view(B, K, N, ldb)
    C = np.empty((M, N), dtype=np.float64)
    S = np.empty((M, N), dtype=np.float64)
    fn = lib.oracle_gemm_f32_naive if naive else lib.oracle_gemm_f32
    fn(_ptr(Ab, ctypes.c_float), _ptr(Bb, ctypes.c_float), _ptr(C, ctypes.c_double),
       _ptr(S, ctypes.c_double), M, N, K, lda, ldb)
    return C, S


def gemm_f32_rows(A, B, rows, N, K, lda=None, ldb=None):
    """Rows ``rows`` of the float32 product.  Returns (C_ref, S)."""
    lib = _load()
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    Mmax = int(rows.max()) + 1 if rows.size else 0
    Ab, lda = _f32_view(A, Mmax, K, lda)
    Bb, ldb = _f32_view(B, K, N, ldb)
    C = np.empty((rows.size, N), dtype=np.float64)
    S = np.empty((rows.size, N), dtype=np.float64)
    lib.oracle_gemm_f32_rows(_ptr(Ab, ctypes.c_float), _ptr(Bb, ctypes.c_float), _ptr(C, ctypes.c_double),
                             _ptr(S, ctypes.c_double), _ptr(rows, ctypes.c_int64), rows.size, N, K, lda, ldb)
    return C, S


def mhsa(Q, K, V, N, d_model, h, ldq=None, ldk=None, ldv=None):
    """Task 6, multi-head self-attention, in fp64 on bfloat16 bit patterns.
    Q, K, V: N x d_model (2-D, or flat with leading dimensions).  Returns
    (out, T), each N x d_model, T[i][c] = sum_j p_ij |V[j][c]|."""
    lib = _load()
    Qb, ldq = _operand_view(Q, N, d_model, ldq)
    Kb, ldk = _operand_view(K, N, d_model, ldk)
    Vb, ldv = _operand_view(V, N, d_model, ldv)
    out = np.empty((N, d_model), dtype=np.float64)
    T = np.empty((N, d_model), dtype=np.float64)
    rc = lib.oracle_mhsa_bf16(_ptr(Qb, ctypes.c_uint16), _ptr(Kb, ctypes.c_uint16), _ptr(Vb, ctypes.c_uint16),
                              _ptr(out, ctypes.c_double), _ptr(T, ctypes.c_double),
                              N, d_model, h, ldq, ldk, ldv)
    if rc != 0:
        raise ValueError("h must divide d_model")
    return out, T


# --------------------------------------------------------------------------
# Tasks 8, 14, 15, 4: transpose, sum, dot product, LayerNorm on float32 arrays
# --------------------------------------------------------------------------

def _f32_flat(x, need: int) -> np.ndarray:
    x = np.ascontiguousarray(np.asarray(x))
    if x.dtype != np.float32:
        raise TypeError("operands are float32")
    x = x.reshape(-1)
    if x.size < need:
        raise ValueError("array too small")
    return x


def transpose_f32(A, rows: int, cols: int, lda: int | None = None, ldat: int | None = None,
                  fill: float = np.nan) -> np.ndarray:
    """Task 8: the ``cols x rows`` transpose of the row-major ``rows x cols`` matrix A
    (row pitch lda).  Returns a flat float32 buffer with row pitch ldat whose
    padding elements hold ``fill``."""
    lda = cols if lda is None else lda
    ldat = rows if ldat is None else ldat
    if lda < cols or ldat < rows:
        raise ValueError("pitch smaller than the row length")
    need = (rows - 1) * lda + cols if rows and cols else 0
    a = _f32_flat(A, need)
    out = np.full((cols - 1) * ldat + rows if rows and cols else 0, fill, dtype=np.float32)
    _load().oracle_transpose_f32(_ptr(a, ctypes.c_float), _ptr(out, ctypes.c_float), rows, cols, lda, ldat)
    return out


def sum_f32(x):
    """Task 14: (sum of x in fp64, sum of |x|)."""
    a = _f32_flat(x, 0)
    s_abs = np.zeros(1)
    s = _load().oracle_sum_f32(_ptr(a, ctypes.c_float), a.size, _ptr(s_abs, ctypes.c_double))
    return float(s), float(s_abs[0])


def dot_f32(a, b):
    """Task 15: (a . b in fp64, sum of |a_i||b_i|)."""
    a = _f32_flat(a, 0)
    b = _f32_flat(b, a.size)
    if a.size != b.size:
        raise ValueError("vectors differ in length")
    s_abs = np.zeros(1)
    s = _load().oracle_dot_f32(_ptr(a, ctypes.c_float), _ptr(b, ctypes.c_float), a.size,
                               _ptr(s_abs, ctypes.c_double))
    return float(s), float(s_abs[0])


def layernorm_f32(x, gamma, beta, batch: int, m: int, eps: float = 1e-5):
    """Task 4: (y as fp64 ``batch x m``, per-sample mean, per-sample 1/sqrt(var + eps)).
    gamma / beta: ``m`` float32 values each, or None."""
    xs = _f32_flat(x, batch * m)
    g = None if gamma is None else _f32_flat(gamma, m)
    b = None if beta is None else _f32_flat(beta, m)
    y = np.empty((batch, m), dtype=np.float64)
    mean = np.empty(batch)
    rstd = np.empty(batch)
    null = ctypes.POINTER(ctypes.c_float)()
    _load().oracle_layernorm_f32(_ptr(xs, ctypes.c_float), null if g is None else _ptr(g, ctypes.c_float),
                                 null if b is None else _ptr(b, ctypes.c_float), _ptr(y, ctypes.c_double),
                                 batch, m, float(eps), _ptr(mean, ctypes.c_double), _ptr(rstd, ctypes.c_double))
    return y, mean, rstd


TOL_MHSA = 1e-2      # |O_gpu - O_ref| <= 1e-2 * T  (probabilities are rounded to bf16 on the GPU)
TOL_F32_IN = 1e-5    # |C_gpu - C_ref| <= 1e-5 * S for the fp32-operand path (three bf16 pieces per operand: ~2^-24 per product)
TOL_TF32 = 2.5e-3    # ... for fp32 operands used as TF32 (ten fraction bits: 2^-10 per truncated operand, 2^-9 per
                     # product, plus K * 2^-24 <= 5e-4 of float32 accumulation)


# --------------------------------------------------------------------------
# bfloat16 <-> fp64 by bit manipulation
# --------------------------------------------------------------------------

def bf16_bits_to_f64(bits) -> np.ndarray:
    """Exact widening: a bfloat16 is the top half of an IEEE binary32."""
    b = np.asarray(bits, dtype=np.uint16)
    with np.errstate(invalid="ignore"):      # signalling-NaN patterns widen quietly
        return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f32_to_bf16_bits(x) -> np.ndarray:
    """binary32 -> bfloat16 bits, round to nearest, ties to the even mantissa.
    NaN stays NaN (quiet bit set); +-Inf and overflow to Inf follow IEEE."""
    f = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = (u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)
    out = (r & np.uint64(0xFFFF)).astype(np.uint16)
    nan = np.isnan(f)
    if np.any(nan):
        out = np.where(nan, ((u >> np.uint64(16)) | np.uint64(0x0040)).astype(np.uint16), out)
    return out


def f64_to_bf16_bits(x) -> np.ndarray:
    """fp64 -> bfloat16 bits with ONE rounding (nearest, ties to even).

    The GPU epilogue rounds an fp32 accumulator; for values that are exactly
    representable in fp32 (every integer-valued test case) the two agree.
    Done directly from the fp64 bit pattern so no double rounding occurs.
    Handles normal bf16 range, zeros, Inf and NaN; fp64 values that would be
    bf16 subnormals are rounded via an exact scaling step.
    """
    d = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    out = np.empty(d.shape, dtype=np.uint16)
    flat = d.reshape(-1)
    o = out.reshape(-1)
    sign = (np.signbit(flat)).astype(np.uint16) << np.uint16(15)
    a = np.abs(flat)
    # bf16: 8 exponent bits (bias 127), 7 mantissa bits.
    res = np.zeros(flat.shape, dtype=np.uint16)
    isnan = np.isnan(a)
    isinf = np.isinf(a)
    nz = (a > 0) & ~isnan & ~isinf
    if np.any(nz):
        m, e = np.frexp(a[nz])            # a = m * 2**e, m in [0.5, 1)
        E = e - 1                         # a = (2m) * 2**E, 2m in [1, 2)
        Emin = -126
        Eeff = np.maximum(E, Emin)        # subnormals share exponent -126
        # quantum = 2**(Eeff-7); q = a / quantum is exact (power-of-two scaling)
        q = np.ldexp(a[nz], (7 - Eeff).astype(np.int64))
        qi = np.rint(q)                   # rint = round half to even
        # qi in [0, 256]; 256 means carry into the next exponent
        qi = qi.astype(np.int64)
        carry = qi >= 256
        Eeff = np.where(carry & (E >= Emin), Eeff + 1, Eeff)
        qi = np.where(carry & (E >= Emin), 128, qi)
        # normal numbers: biased exponent = Eeff + 127, mantissa = qi - 128
        normal = qi >= 128
        biased = np.where(normal, Eeff + 127, 0)
        mant = np.where(normal, qi - 128, qi)
        # subnormal that rounded up to the smallest normal has qi == 128 -> normal (ok)
        bits = (biased.astype(np.int64) << 7) | mant.astype(np.int64)
        bits = np.where(biased >= 255, 0x7F80, bits)   # overflow -> Inf
        res[nz] = bits.astype(np.uint16)
    res[isinf] = 0x7F80
    res[isnan] = 0x7FC0
    o[:] = res | sign
    return out


# --------------------------------------------------------------------------
# acceptance rule
# --------------------------------------------------------------------------

TOL_F32_OUT = 1e-3   # |C_gpu - C_ref| <= 1e-3 * S  for fp32 output
TOL_BF16_OUT = 1e-2  # |C_gpu - C_ref| <= 1e-2 * S  for bf16 output


@dataclass
class CheckResult:
    ok: bool
    n_bad: int
    max_scaled_err: float      # max |dC| / S   (0/0 := 0, x/0 := inf)
    argmax: tuple
    n_nonfinite: int

    def __bool__(self):
        return self.ok


def check(C_gpu_f64: np.ndarray, C_ref: np.ndarray, S: np.ndarray, tol: float) -> CheckResult:
    """Element-wise acceptance: every element must satisfy
    ``|C_gpu - C_ref| <= tol * S``; where S == 0 this demands equality
    (numerically, so -0 == +0).  Non-finite GPU values always fail."""
    G = np.asarray(C_gpu_f64, dtype=np.float64)
    if G.shape != C_ref.shape or G.shape != S.shape:
        raise ValueError(f"shape mismatch {G.shape} vs {C_ref.shape} vs {S.shape}")
    if G.size == 0:
        return CheckResult(True, 0, 0.0, (), 0)
    nonfinite = ~np.isfinite(G)
    diff = np.abs(G - C_ref)
    bad = (diff > tol * S) | nonfinite
    with np.errstate(divide="ignore", invalid="ignore"):
        scaled = np.where(S > 0, diff / np.where(S > 0, S, 1.0),
                          np.where(diff > 0, np.inf, 0.0))
    scaled = np.where(nonfinite, np.inf, scaled)
    idx = np.unravel_index(int(np.argmax(scaled)), scaled.shape)
    return CheckResult(ok=not bool(bad.any()), n_bad=int(bad.sum()),
                       max_scaled_err=float(scaled[idx]), argmax=tuple(int(i) for i in idx),
                       n_nonfinite=int(nonfinite.sum()))
