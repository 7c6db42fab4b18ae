"""Seeded synthetic inputs for the bf16 GEMM path.

This module only *produces operands*: it draws numbers, narrows them to
bfloat16 bit patterns and lays them out row-major.  It contains none of the
contraction's arithmetic and is the one module that the CUDA-side tests, the
benchmark and the CPU checker all take their operands from, so that both sides
see the same bits.

The paper draws its test inputs at random per task and size (Table "Input
size of each task"; Task 2 multiplies A (size x 4096) by B (4096 x 2048)) but
publishes neither seeds nor data, so every input here is synthetic and seeded.

Recipe
------
For a configuration with seed ``s``: A comes from
``numpy.random.default_rng([s, 0])`` and B from ``default_rng([s, 1])``;
values are drawn as float32 (``uniform(-1, 1)`` -- half open -- or
``standard_normal * std``), then narrowed to bfloat16 with round-to-nearest-
even done on the bit pattern.  The arrays returned are ``uint16`` bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

F32, BF16 = 0, 1  # out_dtype codes of the C ABI


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even.
    Inputs here are finite, so no NaN handling is needed."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    # finite inputs far below the float32 maximum: the add cannot wrap
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns -> float32 (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def int_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Small integers (|x| <= 256) -> bfloat16 bit patterns, exactly."""
    x = np.asarray(x)
    assert np.all(np.abs(x) <= 256)
    return f32_to_bf16_bits(x.astype(np.float32))


def _draw(rng: np.random.Generator, shape, dist: str, std: float) -> np.ndarray:
    if dist == "uniform":
        v = rng.uniform(-1.0, 1.0, size=shape).astype(np.float32)
    elif dist == "normal":
        v = rng.standard_normal(size=shape, dtype=np.float32)
        if std != 1.0:
            v = v * np.float32(std)
    else:
        raise ValueError(dist)
    return v


def random_operand(seed, which: int, rows: int, cols: int, ld: int | None = None,
                   dist: str = "normal", std: float = 1.0, batch: int = 1,
                   stride: int | None = None, pad_bits: int = 0x7FC0) -> np.ndarray:
    """Flat uint16 buffer holding ``batch`` row-major ``rows x cols`` operands
    with leading dimension ``ld`` and item stride ``stride`` (elements).
    Padding elements (columns >= cols, gaps between items) hold ``pad_bits``
    (a bfloat16 NaN by default), so a kernel that reads them poisons its result.
    ``which`` is 0 for A and 1 for B."""
    ld = cols if ld is None else ld
    assert ld >= cols
    item = rows * ld
    stride = item if stride is None else stride
    assert batch == 1 or stride >= (rows - 1) * ld + cols
    rng = np.random.default_rng([int(seed), int(which)])
    vals = f32_to_bf16_bits(_draw(rng, (batch, rows, cols), dist, std))
    total = (batch - 1) * stride + (rows - 1) * ld + cols if rows and cols and batch else 0
    buf = np.full(max(total, 1), pad_bits, dtype=np.uint16)
    for t in range(batch):
        if rows and cols:
            view = np.lib.stride_tricks.as_strided(
                buf[t * stride:], shape=(rows, cols), strides=(ld * 2, 2))
            view[...] = vals[t]
    return buf


@dataclass(frozen=True)
class GemmConfig:
    """One workload: shapes, strides, output type and the input recipe."""
    name: str
    M: int
    N: int
    K: int
    out_dtype: int
    seed: int
    dist_a: str = "normal"
    dist_b: str = "normal"
    std_a: float = 1.0
    std_b: float = 1.0
    lda: int | None = None
    ldb: int | None = None
    ldc: int | None = None
    batch: int = 1
    note: str = ""

    @property
    def lda_(self): return self.K if self.lda is None else self.lda
    @property
    def ldb_(self): return self.N if self.ldb is None else self.ldb
    @property
    def ldc_(self): return self.N if self.ldc is None else self.ldc
    @property
    def strideA(self): return self.M * self.lda_
    @property
    def strideB(self): return self.K * self.ldb_
    @property
    def strideC(self): return self.M * self.ldc_
    @property
    def flops(self): return 2 * self.M * self.N * self.K * self.batch
    @property
    def out_bytes(self): return 4 if self.out_dtype == F32 else 2
    @property
    def algorithmic_bytes(self):
        """A and B read once, C written once."""
        return self.batch * (2 * self.M * self.K + 2 * self.K * self.N
                             + self.out_bytes * self.M * self.N)

    def make(self):
        """(A, B) as flat uint16 buffers laid out per this configuration."""
        A = random_operand(self.seed, 0, self.M, self.K, self.lda_, self.dist_a, self.std_a,
                           self.batch, self.strideA)
        B = random_operand(self.seed, 1, self.K, self.N, self.ldb_, self.dist_b, self.std_b,
                           self.batch, self.strideB)
        return A, B


# The benchmark configurations (names C1..C5b) -------------------------------
CONFIGS = {
    "C1": GemmConfig("C1", 256, 256, 256, F32, seed=0, dist_a="uniform", dist_b="uniform",
                     note="small case, launch-latency bound"),
    "C2": GemmConfig("C2", 4096, 4096, 4096, BF16, seed=1,
                     note="square, tensor-core bound; the headline TFLOP/s workload"),
    "C3": GemmConfig("C3", 8192, 11008, 4096, BF16, seed=2, std_b=0.02,
                     note="transformer MLP up-projection: activations x weights"),
    "C4": GemmConfig("C4", 128, 128, 64, F32, seed=3, batch=512,
                     note="batched attention-score shaped products, HBM bound"),
    "C5a": GemmConfig("C5a", 16, 16384, 8192, F32, seed=4, dist_a="uniform", dist_b="uniform",
                      note="skinny, HBM bound; the headline GB/s workload"),
    "C5b": GemmConfig("C5b", 3001, 1999, 5003, F32, seed=5,
                      note="irregular, odd leading dimensions, edge tiles everywhere"),
}


def task2_ladder(step: int) -> GemmConfig:
    """The paper's own Task 2 shapes: A (size x 4096) times B (4096 x 2048) with
    size = 2**(10 + 2*step), step in 0..4, here with bf16 operands."""
    size = 1 << (10 + 2 * step)
    return GemmConfig(f"T2-{step + 1}", size, 2048, 4096, F32, seed=100 + step,
                      note="paper Task 2 size ladder (bf16 operands instead of fp32)")


# Deterministic, exactly representable operand recipes ------------------------
# Each returns dense uint16 arrays (rows x cols) whose product has a closed form.

def identity_bits(rows: int, cols: int) -> np.ndarray:
    """rows x cols matrix with ones on the main diagonal."""
    X = np.zeros((rows, cols), dtype=np.float32)
    n = min(rows, cols)
    X[np.arange(n), np.arange(n)] = 1.0
    return f32_to_bf16_bits(X)


def permutation_bits(n: int, seed: int):
    """(P bits, pi) with P[i][pi[i]] = 1."""
    pi = np.random.default_rng([seed, 7]).permutation(n)
    X = np.zeros((n, n), dtype=np.float32)
    X[np.arange(n), pi] = 1.0
    return f32_to_bf16_bits(X), pi


def rank1_int_factors(M: int, N: int, K: int, seed: int, umax: int = 8, pmax: int = 2):
    """Integer vectors u (M), v (N) in [-umax, umax] and p, q (K) in
    [-pmax, pmax].  A = u p^T and B = q v^T are exact in bfloat16 and
    A B = (p . q) u v^T with every partial sum an integer below 2**24
    when umax**2 * pmax**2 * K < 2**24."""
    assert umax * umax * pmax * pmax * K < (1 << 24)
    rng = np.random.default_rng([seed, 11])
    u = rng.integers(-umax, umax + 1, size=M)
    v = rng.integers(-umax, umax + 1, size=N)
    p = rng.integers(-pmax, pmax + 1, size=K)
    q = rng.integers(-pmax, pmax + 1, size=K)
    return u, v, p, q


def rank1_int_operands(M: int, N: int, K: int, seed: int, umax: int = 8, pmax: int = 2):
    """(A bits, B bits, u, v, p, q) for the integer rank-1 recipe."""
    u, v, p, q = rank1_int_factors(M, N, K, seed, umax, pmax)
    A = int_to_bf16_bits(np.outer(u, p))
    B = int_to_bf16_bits(np.outer(q, v))
    return A, B, u, v, p, q


def embed(X: np.ndarray, ld: int, pad_bits: int = 0x7FC0, lead: int = 0) -> np.ndarray:
    """Copy a dense 2-D uint16 operand into a flat buffer with leading dimension
    ``ld`` and ``lead`` extra elements in front; padding is NaN by default."""
    rows, cols = X.shape
    assert ld >= cols
    total = lead + ((rows - 1) * ld + cols if rows and cols else 0)
    buf = np.full(max(total, 1), pad_bits, dtype=np.uint16)
    if rows and cols:
        view = np.lib.stride_tricks.as_strided(buf[lead:], shape=(rows, cols), strides=(ld * 2, 2))
        view[...] = X
    return buf


def fnv1a64(a: np.ndarray) -> int:
    """64-bit FNV-1a over the bytes of an array, folded 8 bytes at a time
    (a cheap drift detector for the generators, not a cryptographic hash)."""
    b = np.ascontiguousarray(a).view(np.uint8)
    pad = (-b.size) % 8
    if pad:
        b = np.concatenate([b, np.zeros(pad, dtype=np.uint8)])
    w = b.view(np.uint64)
    # fold with xor / rotate so the digest depends on order; python ints for the tail
    h = np.uint64(0xCBF29CE484222325)
    prime = np.uint64(0x100000001B3)
    with np.errstate(over="ignore"):
        idx = np.arange(w.size, dtype=np.uint64)
        mixed = (w ^ (idx * np.uint64(0x9E3779B97F4A7C15))) * prime
        acc = np.bitwise_xor.reduce(mixed) if w.size else np.uint64(0)
        s = np.add.reduce(mixed) if w.size else np.uint64(0)
        h = (h ^ acc) * prime
        h = (h ^ s) * prime
    return int(h)


# Tasks 8, 14, 15, 4: float32 arrays -------------------------------------------
# The paper's sizes (its table of input sizes): transpose N x N with N = 2^10 ..
# 2^14; reduction N = 2^10 .. 2^18 (steps of 4x); dot product N = 2^16 .. 2^20;
# LayerNorm (16, 4, d, d) with d = 2^6 .. 2^10.  Values are seeded float32 draws.

TRANSPOSE_SIZES = [1 << k for k in range(10, 15)]
REDUCTION_SIZES = [1 << k for k in range(10, 19, 2)]
DOT_SIZES = [1 << k for k in range(16, 21)]
LAYERNORM_SHAPES = [(16, 4, 1 << k, 1 << k) for k in range(6, 11)]


def task_array(seed: int, which: int, n: int, dist: str = "normal", std: float = 1.0,
               mean: float = 0.0) -> np.ndarray:
    """``n`` float32 values from ``default_rng([seed, which])``: ``normal`` (times std, plus
    mean) or ``uniform`` on [-1, 1) (plus mean)."""
    rng = np.random.default_rng([int(seed), int(which)])
    if dist == "uniform":
        x = rng.uniform(-1.0, 1.0, n).astype(np.float32)
    else:
        x = rng.standard_normal(n, dtype=np.float32) * np.float32(std)
    if mean:
        x = x + np.float32(mean)
    return np.ascontiguousarray(x, dtype=np.float32)


def layernorm_inputs(seed: int, batch: int, m: int):
    """(x [batch * m], gamma [m], beta [m]) as float32: samples with different means and
    spreads (sample s: mean s - batch / 2, std 0.5 + s / 4), gamma around 1, beta around 0."""
    x = task_array(seed, 0, batch * m).reshape(batch, m)
    s = np.arange(batch, dtype=np.float32)[:, None]
    x = x * (np.float32(0.5) + s / np.float32(4)) + (s - np.float32(batch / 2))
    gamma = task_array(seed, 1, m, "uniform") * np.float32(0.5) + np.float32(1.0)
    beta = task_array(seed, 2, m) * np.float32(0.1)
    return np.ascontiguousarray(x.reshape(-1), dtype=np.float32), gamma, beta
