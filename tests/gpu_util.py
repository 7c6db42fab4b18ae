"""Helpers for the GPU parity tests: move seeded operands to the device, call the
library through its C ABI (via the ctypes binding), bring C back with guard
bands checked, and compare with the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2506_09092_b200 import binding as B
from paper_2506_09092_b200 import inputs as gi

SENTINEL_F32 = 0x7FC0DEAD      # a NaN pattern no kernel produces
SENTINEL_BF16 = 0x7FDE
GUARD = 64                     # guard elements before and after C


def to_device_bits(bits: np.ndarray, lead: int = 0) -> torch.Tensor:
    """uint16 bit patterns -> int16 CUDA tensor; ``lead`` extra elements in front
    (used to offset the base pointer by an odd number of elements)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    if lead:
        buf = torch.empty(bits.size + lead, dtype=torch.int16, device="cuda")
        buf[lead:] = t.cuda()
        return buf
    return t.cuda()


class COut:
    """Device buffer for C with guard bands and sentinel-filled padding."""

    def __init__(self, M, N, ldc, out_dtype, batch=1, strideC=None, lead=0):
        self.M, self.N, self.ldc, self.out_dtype, self.batch = M, N, ldc, out_dtype, batch
        self.strideC = M * ldc if strideC is None else strideC
        self.lead = lead
        n = (batch - 1) * self.strideC + ((M - 1) * ldc + N if M and N else 0) if batch else 0
        self.n = n
        total = GUARD + lead + n + GUARD
        if out_dtype == gi.F32:
            self.buf = torch.full((total,), SENTINEL_F32, dtype=torch.int32, device="cuda")
            self.esz = 4
        else:
            self.buf = torch.full((total,), SENTINEL_BF16, dtype=torch.int16, device="cuda")
            self.esz = 2
        self.ptr = self.buf.data_ptr() + (GUARD + lead) * self.esz

    def fetch(self):
        """(C as fp64 [batch, M, N], raw bits [batch, M, N], untouched_ok)."""
        raw = self.buf.cpu().numpy()
        sentinel = SENTINEL_F32 if self.out_dtype == gi.F32 else SENTINEL_BF16
        raw_u = raw.view(np.uint32 if self.out_dtype == gi.F32 else np.uint16)
        body = raw_u[GUARD + self.lead: GUARD + self.lead + self.n]
        touched = np.zeros(self.n, dtype=bool)
        M, N, ldc = self.M, self.N, self.ldc
        bits = np.empty((self.batch, M, N), dtype=raw_u.dtype)
        for t in range(self.batch):
            if M and N:
                v = np.lib.stride_tricks.as_strided(body[t * self.strideC:], (M, N),
                                                    (ldc * body.itemsize, body.itemsize))
                bits[t] = v
                tv = np.lib.stride_tricks.as_strided(touched[t * self.strideC:], (M, N), (ldc, 1))
                tv[...] = True
        guards_ok = bool(np.all(raw_u[:GUARD + self.lead] == sentinel)
                         and np.all(raw_u[GUARD + self.lead + self.n:] == sentinel)
                         and np.all(body[~touched] == sentinel))
        if self.out_dtype == gi.F32:
            vals = bits.view(np.float32).astype(np.float64)
        else:
            vals = oracle.bf16_bits_to_f64(bits)
        return vals, bits, guards_ok


def run_gemm(A_bits, B_bits, M, N, K, lda, ldb, ldc, out_dtype, batch=1,
             strideA=None, strideB=None, strideC=None, variant=B.VARIANT_AUTO,
             lead_a=0, lead_b=0, lead_c=0, expect_status=B.OK):
    """Run one product on the GPU through ``cudallm_gemm_bf16_variant``.
    Returns (C fp64 [batch,M,N], C bits, guards_ok)."""
    dA = to_device_bits(A_bits, lead_a)
    dB = to_device_bits(B_bits, lead_b)
    out = COut(M, N, ldc, out_dtype, batch, strideC, lead_c)
    sA = M * lda if strideA is None else strideA
    sB = K * ldb if strideB is None else strideB
    st = B.gemm_bf16_variant(variant, dA.data_ptr() + 2 * lead_a, dB.data_ptr() + 2 * lead_b, out.ptr,
                             M, N, K, lda, ldb, ldc, sA, sB, out.strideC, batch, out_dtype,
                             torch.cuda.current_stream(), check=False)
    assert st == expect_status, f"status {st}: {B.strerror(st)}"
    code, detail = B.device_status(torch.cuda.current_stream())
    assert code == B.OK, f"device status {code} detail {detail:#x}"
    return out.fetch()


def run_config(cfg: gi.GemmConfig, variant=B.VARIANT_AUTO, operands=None):
    A, Bm = operands if operands is not None else cfg.make()
    return run_gemm(A, Bm, cfg.M, cfg.N, cfg.K, cfg.lda_, cfg.ldb_, cfg.ldc_, cfg.out_dtype,
                    cfg.batch, cfg.strideA, cfg.strideB, cfg.strideC, variant)


def log_observed_error(family: str, case: str, observed: float, bound: float, what: str, **extra):
    """Append the largest error a parity test observed (in the units of its tolerance) to
    ``observed_errors.jsonl`` in the directory the environment variable CUDALLM_ERROR_LOG_DIR
    names (default: the scratch output directory at the repository root, created on demand), so that the
    share of each tolerance that is actually used can be read off."""
    import json
    import os
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out_dir = os.environ.get("CUDALLM_ERROR_LOG_DIR", os.path.join(root, "gpurun_out"))
    try:
        os.makedirs(out_dir, exist_ok=True)
        rec = dict(family=family, case=case, observed=float(observed), bound=float(bound),
                   share=float(observed) / float(bound) if bound else None, what=what, **extra)
        with open(os.path.join(out_dir, "observed_errors.jsonl"), "a") as f:
            f.write(json.dumps(rec) + "\n")
    except OSError:
        pass


def tol_for(out_dtype):
    return oracle.TOL_F32_OUT if out_dtype == gi.F32 else oracle.TOL_BF16_OUT


def supported_variants(M, N, K, lda, ldb, ldc, batch, out_dtype):
    return [v for v in range(B.num_variants())
            if B.variant_supports(v, M, N, K, lda, ldb, ldc, batch, out_dtype) == 1]
