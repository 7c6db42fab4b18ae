"""B200-native bf16 GEMM library (C = A x B, fp32 accumulate) with an
FSR-style validate / profile / arg-min harness.

The compute path lives in ``csrc/`` behind a C ABI (``include/cudallm_gemm.h``);
``binding`` marshals arguments to it and nothing else.  Importing the package
does not load the CUDA library; ``binding.lib()`` does, and raises if it has
not been built -- there is no CPU fallback.
"""
__all__ = ["inputs", "binding", "harness", "build"]
