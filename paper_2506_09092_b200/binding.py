"""ctypes binding of ``libcudallm_gemm.so``: one Python function per C entry
point, same names, argument marshalling only.

Device buffers are passed as integer addresses (``tensor.data_ptr()``) or as
torch tensors (their ``data_ptr()`` is taken); streams as integer handles
(``torch.cuda.current_stream().cuda_stream``).  Nothing here computes: if the
shared library is missing this module raises, it never falls back to the CPU.
"""
from __future__ import annotations

import ctypes
import os

F32, BF16 = 0, 1
VARIANT_AUTO = -1

OK = 0
ERR_INVALID_POINTER = -1
ERR_INVALID_DIM = -2
ERR_INVALID_LD = -3
ERR_INVALID_DTYPE = -4
ERR_INVALID_VARIANT = -5
ERR_UNSUPPORTED_SHAPE = -6
ERR_UNSUPPORTED_DEVICE = -7
ERR_CUDA = -8
ERR_DEVICE_TIMEOUT = -9
ERR_WORKSPACE = -10
ERR_MISALIGNED = -11
ERR_TOO_LARGE = -12
NOALLOC_SCRATCH_BYTES = 8 << 20

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcudallm_gemm.so")
_lib = None

_i64 = ctypes.c_int64
_vp = ctypes.c_void_p
_int = ctypes.c_int
_sz = ctypes.c_size_t

# name -> (restype, argtypes); mirrors include/cudallm_gemm.h and include/cudallm_tasks.h
SIGNATURES = {
    "cudallm_gemm_bf16": (_int, [_vp, _vp, _vp] + [_i64] * 6 + [_int, _vp]),
    "cudallm_gemm_f32": (_int, [_vp, _vp, _vp] + [_i64] * 6 + [_int, _vp]),
    "cudallm_gemm_tf32": (_int, [_vp, _vp, _vp] + [_i64] * 6 + [_vp]),
    "cudallm_mhsa_bf16": (_int, [_vp, _vp, _vp, _vp] + [_i64] * 7 + [_vp]),
    "cudallm_gemm_bf16_batched": (_int, [_vp, _vp, _vp] + [_i64] * 10 + [_int, _vp]),
    "cudallm_gemm_bf16_variant": (_int, [_int, _vp, _vp, _vp] + [_i64] * 10 + [_int, _vp]),
    "cudallm_gemm_bf16_host": (_int, [_vp, _vp, _vp] + [_i64] * 6 + [_int, _vp, _sz, _vp]),
    "cudallm_host_staging_bytes": (_sz, [_i64] * 6 + [_int]),
    "cudallm_gemm_bf16_splitk_noalloc": (_int, [_vp, _vp, _vp] + [_i64] * 6 + [_int, _int, _vp]),
    "cudallm_num_variants": (_int, []),
    "cudallm_dispatch_set": (_int, [_i64, _i64, _i64, _i64, _int, _int]),
    "cudallm_dispatch_get": (_int, [_i64, _i64, _i64, _i64, _int, ctypes.POINTER(ctypes.c_int)]),
    "cudallm_dispatch_set_class": (_int, [_i64, _i64, _i64, _i64, _int, _int, _int]),
    "cudallm_dispatch_get_class": (_int, [_i64, _i64, _i64, _i64, _int, _int, ctypes.POINTER(ctypes.c_int)]),
    "cudallm_dispatch_clear": (_int, []),
    "cudallm_dispatch_load_packaged": (_int, []),
    "cudallm_variant_code": (_int, [_int, _int, _int]),
    "cudallm_variant_name": (ctypes.c_char_p, [_int]),
    "cudallm_variant_supports": (_int, [_int] + [_i64] * 7 + [_int]),
    "cudallm_select_variant": (_int, [_i64] * 7 + [_int]),
    "cudallm_workspace_bytes": (_sz, [_i64] * 7 + [_int]),
    "cudallm_set_workspace": (_int, [_vp, _sz]),
    "cudallm_set_workspace_for_stream": (_int, [_vp, _vp, _sz]),
    "cudallm_reserve_workspace": (_int, [_sz]),
    "cudallm_shutdown": (_int, []),
    "cudallm_debug_set": (_int, [_int, ctypes.c_ulonglong]),
    "cudallm_device_status": (_int, [_vp, ctypes.POINTER(_int), ctypes.POINTER(_int)]),
    "cudallm_strerror": (ctypes.c_char_p, [_int]),
    "cudallm_version": (_int, []),
    "cudallm_transpose_f32": (_int, [_vp, _vp] + [_i64] * 4 + [_vp]),
    "cudallm_sum_f32": (_int, [_vp, _i64, _vp, _vp]),
    "cudallm_dot_f32": (_int, [_vp, _vp, _i64, _vp, _vp]),
    "cudallm_layernorm_f32": (_int, [_vp, _vp, _vp, _vp, _i64, _i64, ctypes.c_float, _vp]),
}


class CudallmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status}: {strerror(status)}")


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2506_09092_b200.build` "
                "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _p(x):
    """Address of a device/host buffer: int, None, or anything with data_ptr()."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(type(x))


def _s(stream):
    if stream is None:
        return None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _check(st: int, where: str, check: bool):
    if check and st != OK:
        raise CudallmError(st, where)
    return st


def gemm_bf16(A, B, C, M, N, K, lda, ldb, ldc, out_dtype, stream=None, check=True):
    st = lib().cudallm_gemm_bf16(_p(A), _p(B), _p(C), M, N, K, lda, ldb, ldc, out_dtype, _s(stream))
    return _check(st, "cudallm_gemm_bf16", check)


def gemm_f32(A, B, C, M, N, K, lda, ldb, ldc, variant=VARIANT_AUTO, stream=None, check=True):
    """fp32 operands and result (the paper's Task 2 as stated), computed on the
    bf16 tensor cores from three-piece splits of the operands."""
    st = lib().cudallm_gemm_f32(_p(A), _p(B), _p(C), M, N, K, lda, ldb, ldc, variant, _s(stream))
    return _check(st, "cudallm_gemm_f32", check)


def gemm_tf32(A, B, C, M, N, K, lda, ldb, ldc, stream=None, check=True):
    """fp32 operands and result with the tensor cores reading the operands as TF32."""
    st = lib().cudallm_gemm_tf32(_p(A), _p(B), _p(C), M, N, K, lda, ldb, ldc, _s(stream))
    return _check(st, "cudallm_gemm_tf32", check)


def mhsa_bf16(Q, K, V, O, N, d_model, h, ldq, ldk, ldv, ldo, stream=None, check=True):
    """Multi-head self-attention (Task 6): bf16 Q, K, V (N x d_model), fp32 O."""
    st = lib().cudallm_mhsa_bf16(_p(Q), _p(K), _p(V), _p(O), N, d_model, h, ldq, ldk, ldv, ldo, _s(stream))
    return _check(st, "cudallm_mhsa_bf16", check)


def transpose_f32(A, AT, rows, cols, lda, ldat, stream=None, check=True):
    """Task 8: AT (cols x rows, pitch ldat) = transpose of A (rows x cols, pitch lda), fp32."""
    st = lib().cudallm_transpose_f32(_p(A), _p(AT), rows, cols, lda, ldat, _s(stream))
    return _check(st, "cudallm_transpose_f32", check)


def sum_f32(x, n, result, stream=None, check=True):
    """Task 14: result[0] (device fp32) = sum of the n fp32 elements of x."""
    st = lib().cudallm_sum_f32(_p(x), n, _p(result), _s(stream))
    return _check(st, "cudallm_sum_f32", check)


def dot_f32(a, b, n, result, stream=None, check=True):
    """Task 15: result[0] (device fp32) = a . b over n fp32 elements."""
    st = lib().cudallm_dot_f32(_p(a), _p(b), n, _p(result), _s(stream))
    return _check(st, "cudallm_dot_f32", check)


def layernorm_f32(x, gamma, beta, y, batch, m, eps=1e-5, stream=None, check=True):
    """Task 4: LayerNorm of ``batch`` samples of ``m`` fp32 elements; gamma / beta may be None."""
    st = lib().cudallm_layernorm_f32(_p(x), _p(gamma), _p(beta), _p(y), batch, m, ctypes.c_float(eps), _s(stream))
    return _check(st, "cudallm_layernorm_f32", check)


def gemm_bf16_batched(A, B, C, M, N, K, lda, ldb, ldc, strideA, strideB, strideC, batch,
                      out_dtype, stream=None, check=True):
    st = lib().cudallm_gemm_bf16_batched(_p(A), _p(B), _p(C), M, N, K, lda, ldb, ldc,
                                         strideA, strideB, strideC, batch, out_dtype, _s(stream))
    return _check(st, "cudallm_gemm_bf16_batched", check)


def gemm_bf16_variant(variant, A, B, C, M, N, K, lda, ldb, ldc, strideA, strideB, strideC, batch,
                      out_dtype, stream=None, check=True):
    st = lib().cudallm_gemm_bf16_variant(variant, _p(A), _p(B), _p(C), M, N, K, lda, ldb, ldc,
                                         strideA, strideB, strideC, batch, out_dtype, _s(stream))
    return _check(st, "cudallm_gemm_bf16_variant", check)


def gemm_bf16_host(A_host, B_host, C_host, M, N, K, lda, ldb, ldc, out_dtype, dev_buf, dev_bytes,
                   stream=None, check=True):
    st = lib().cudallm_gemm_bf16_host(_p(A_host), _p(B_host), _p(C_host), M, N, K, lda, ldb, ldc,
                                      out_dtype, _p(dev_buf), dev_bytes, _s(stream))
    return _check(st, "cudallm_gemm_bf16_host", check)


def gemm_bf16_splitk_noalloc(A, B, C, M, N, K, lda, ldb, ldc, out_dtype, split_k, stream=None,
                             check=True):
    """Split-K product whose scratch is an array built into the library: for
    callers that may not allocate device memory (see the header).  Synchronises
    ``stream``; the first call per device should come before any stream capture;
    calls that overlap on the GPU race on the shared scratch."""
    st = lib().cudallm_gemm_bf16_splitk_noalloc(_p(A), _p(B), _p(C), M, N, K, lda, ldb, ldc,
                                                out_dtype, split_k, _s(stream))
    return _check(st, "cudallm_gemm_bf16_splitk_noalloc", check)


def host_staging_bytes(M, N, K, lda, ldb, ldc, out_dtype) -> int:
    return int(lib().cudallm_host_staging_bytes(M, N, K, lda, ldb, ldc, out_dtype))


def dispatch_set(M, N, K, batch, out_dtype, variant, check=True) -> int:
    """Record ``variant`` as the kernel for products of this shape (-1 removes the entry):
    the library's automatic choice uses it before its cost model."""
    return _check(lib().cudallm_dispatch_set(M, N, K, batch, out_dtype, variant), "cudallm_dispatch_set", check)


def dispatch_get(M, N, K, batch, out_dtype) -> int:
    """The recorded variant for the shape, or -1."""
    v = ctypes.c_int(-1)
    _check(lib().cudallm_dispatch_get(M, N, K, batch, out_dtype, ctypes.byref(v)), "cudallm_dispatch_get", True)
    return int(v.value)


def dispatch_set_class(M, N, K, batch, out_dtype, tma_addressable, variant, check=True) -> int:
    """Record ``variant`` for the whole class of shapes that are tiled like this one."""
    return _check(lib().cudallm_dispatch_set_class(M, N, K, batch, out_dtype, int(bool(tma_addressable)), variant),
                  "cudallm_dispatch_set_class", check)


def dispatch_get_class(M, N, K, batch, out_dtype, tma_addressable) -> int:
    v = ctypes.c_int(-1)
    _check(lib().cudallm_dispatch_get_class(M, N, K, batch, out_dtype, int(bool(tma_addressable)), ctypes.byref(v)),
           "cudallm_dispatch_get_class", True)
    return int(v.value)


def dispatch_load_packaged() -> int:
    """Enter the packaged search results into the class table; returns how many."""
    return int(lib().cudallm_dispatch_load_packaged())


def variant_code(variant: int, group_rows: int = 0, tail_parts: int = 0, check=True) -> int:
    """Variant id plus the two knobs the search varies -> the code the entry points take."""
    code = int(lib().cudallm_variant_code(variant, group_rows, tail_parts))
    if check and code < 0:
        raise CudallmError(code, "cudallm_variant_code")
    return code


def describe_code(code: int) -> str:
    """Human-readable form of a variant code: name, and the knobs that are set."""
    name = variant_name(code)
    g, t = (code >> 8) & 0xF, (code >> 12) & 0x7
    return name + (f"+g{1 << (g - 1)}" if g else "") + (f"+t{t}" if t else "")


def dispatch_clear() -> int:
    """Empty the dispatch table; returns how many entries it held."""
    return int(lib().cudallm_dispatch_clear())


def num_variants() -> int:
    return int(lib().cudallm_num_variants())


def variant_name(variant: int):
    s = lib().cudallm_variant_name(variant)
    return None if s is None else s.decode()


def variant_supports(variant, M, N, K, lda, ldb, ldc, batch, out_dtype) -> int:
    return int(lib().cudallm_variant_supports(variant, M, N, K, lda, ldb, ldc, batch, out_dtype))


def select_variant(M, N, K, lda, ldb, ldc, batch, out_dtype) -> int:
    return int(lib().cudallm_select_variant(M, N, K, lda, ldb, ldc, batch, out_dtype))


def workspace_bytes(M, N, K, lda, ldb, ldc, batch, out_dtype) -> int:
    return int(lib().cudallm_workspace_bytes(M, N, K, lda, ldb, ldc, batch, out_dtype))


def set_workspace(dev_ptr, nbytes: int, check=True):
    return _check(lib().cudallm_set_workspace(_p(dev_ptr), nbytes), "cudallm_set_workspace", check)


def set_workspace_for_stream(stream, dev_ptr, nbytes: int, check=True):
    """Attach a caller-owned workspace to ``stream`` (``dev_ptr=None`` removes it)."""
    return _check(lib().cudallm_set_workspace_for_stream(_s(stream), _p(dev_ptr), nbytes),
                  "cudallm_set_workspace_for_stream", check)


def reserve_workspace(nbytes: int, check=True):
    """Size the library's own workspace of the current device now."""
    return _check(lib().cudallm_reserve_workspace(nbytes), "cudallm_reserve_workspace", check)


def shutdown(check=True):
    """Release the library's workspaces, streams and events on every device."""
    return _check(lib().cudallm_shutdown(), "cudallm_shutdown", check)


DEBUG_WAIT_LIMIT_NS, DEBUG_MISS_NEXT_SPLIT_FLAGS, DEBUG_LAYERNORM_PATH = 1, 2, 3


def debug_set(what: int, value: int, check=True):
    """Test hooks of the kernels' bounded waits (see the header)."""
    return _check(lib().cudallm_debug_set(what, value), "cudallm_debug_set", check)


def device_status(stream=None):
    """(code, detail) after synchronising ``stream``."""
    code, detail = _int(0), _int(0)
    lib().cudallm_device_status(_s(stream), ctypes.byref(code), ctypes.byref(detail))
    return code.value, detail.value


def strerror(status: int) -> str:
    return lib().cudallm_strerror(status).decode()


def version() -> int:
    return int(lib().cudallm_version())
