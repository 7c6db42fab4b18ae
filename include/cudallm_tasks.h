/*
 * cudallm_tasks.h -- C ABI of the bandwidth-bound benchmark tasks of the paper
 * on arrays of 32-bit floating point numbers (its Table of task prompts):
 *
 *   Task 8   Matrix Transpose   AT[j][i] = A[i][j]
 *   Task 14  Reduction          s = sum_i x_i
 *   Task 15  Dot Product        s = sum_{i<n} A_i * B_i
 *   Task 4   LayerNorm          per sample: normalise over all its elements,
 *                               then scale by gamma and add beta
 *
 * The general conventions of cudallm_gemm.h hold (device pointers owned by the
 * caller, pitches in elements, calls enqueue on `stream` and return without
 * synchronising, negative CUDALLM_ERR_* status codes, argument errors found
 * before any CUDA call, compute capability 10.0 only, no CPU fallback).  The
 * status codes are those of cudallm_gemm.h.  Only the one-pass LayerNorm kernel
 * (see cudallm_layernorm_f32) has CTAs that wait for one another.
 *
 * cudallm_sum_f32 / cudallm_dot_f32 keep their per-block partial sums in one
 * fixed scratch area per device, and cudallm_layernorm_f32 keeps its per-sample
 * partial statistics in the library workspace: calls of these functions must
 * not run concurrently on different streams of one device.
 */
#ifndef CUDALLM_TASKS_H
#define CUDALLM_TASKS_H

#include <stddef.h>
#include <stdint.h>

#include "cudallm_gemm.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Task 8: AT = transpose(A).
 *   A  : fp32, rows x cols, row-major, row pitch lda  >= cols   (read only)
 *   AT : fp32, cols x rows, row-major, row pitch ldat >= rows   (written; padding
 *        columns rows <= i < ldat are left untouched); must not overlap A.
 * Values are moved bit for bit (NaN payloads and signed zeros included).
 * 16-byte aligned bases with rows, cols, lda and ldat all multiples of 4 take
 * the 64 x 64-tile kernel with 16-byte accesses; anything else (4-byte
 * alignment is required) a 32 x 32-tile kernel with element accesses.  rows == 0 or cols == 0: success, nothing written.
 * Errors: INVALID_DIM (negative, or >= 2^31 - 1024), INVALID_LD, INVALID_POINTER,
 * MISALIGNED, UNSUPPORTED_DEVICE, CUDA.
 */
int cudallm_transpose_f32(const float *A, float *AT, int64_t rows, int64_t cols, int64_t lda, int64_t ldat,
                          void *stream);

/*
 * Task 14: *result = sum_{i<n} x[i].
 *   x      : fp32, n elements (read only); result : one fp32 on the DEVICE.
 * Every element is widened to double and added in double; the total is rounded
 * to fp32 once, so |result - exact| <= 2^-24 |exact| + ~1e-13 sum|x_i|.  Equal
 * inputs give bit-equal results.  n == 0 gives 0.  One kernel launch.
 * Errors: INVALID_DIM (n < 0 or n > 2^40), INVALID_POINTER, MISALIGNED (4 bytes),
 * UNSUPPORTED_DEVICE, CUDA.
 */
int cudallm_sum_f32(const float *x, int64_t n, float *result, void *stream);

/*
 * Task 15: *result = sum_{i<n} a[i] * b[i].
 * Products are formed in double (exact) and added in double; one rounding to
 * fp32 at the end.  Otherwise as cudallm_sum_f32.  a and b may be the same array.
 */
int cudallm_dot_f32(const float *a, const float *b, int64_t n, float *result, void *stream);

/*
 * Task 4: LayerNorm of `batch` samples of m elements each (the paper's input of
 * shape (batch_size, features, dim1, dim2) has m = features * dim1 * dim2 and is
 * passed as it lies in memory: sample s occupies x[s*m .. s*m + m)).
 *     mean_s = (1/m) sum_i x[s][i]
 *     var_s  = (1/m) sum_i (x[s][i] - mean_s)^2              (biased estimate)
 *     y[s][i] = (x[s][i] - mean_s) / sqrt(var_s + eps) * gamma[i] + beta[i]
 *   x, y        : fp32, batch * m elements; y may be x itself (in place), else
 *                 must not overlap x
 *   gamma, beta : fp32, m elements each (one per position of a sample), or NULL
 *                 for "all ones" / "all zeros"
 *   eps         : >= 0 (the usual value is 1e-5)
 * Arithmetic: the moments are taken in fp32 about a pilot value close to the
 * data (so a mean far larger than the spread costs no accuracy), combined in
 * double; the output is formed in fp32 from the mean held as two floats and
 * 1/sqrt(var + eps) rounded to fp32.  With z = (x - mean) / sqrt(var + eps):
 * |y - exact| <= 2^-20 (|z| + 1) |gamma| + 2^-22 |beta| for data whose spread is
 * not dominated by a few outliers; squared deviations must stay inside the fp32
 * range (|x - mean| below about 1e19).  batch == 0 or m == 0: success, nothing
 * written.
 * Kernels: when x, y, gamma and beta are 32-byte aligned, m is a multiple of 8,
 * a sample has 8 to 20 MB (from 4 MB with 32 or more samples) and there are at
 * least four samples, ONE persistent kernel (one CTA per SM) takes the moments
 * of a sample and, a sample or two later, reads it again while it is still in
 * L2, so x crosses DRAM once; its CTAs exchange their partial moments through
 * the workspace and wait for one another with a bound (default 2 s; all CTAs
 * must be resident, i.e. no other kernel may hold SMs for that long).  If a
 * wait runs out the kernel returns, y is unspecified and
 * cudallm_device_status(stream, ...) reports CUDALLM_ERR_DEVICE_TIMEOUT.
 * Everything else takes two plain kernels (moments, then normalisation; x is
 * read twice, the second time from L2 when all of it fits).  Both give results
 * within the bound above; they differ in the last bits because the partial
 * moments are grouped differently.  Equal inputs give equal bits on either.
 * Errors: INVALID_DIM (negative, batch >= 2^31, m > 2^40, eps negative or not
 * finite), INVALID_POINTER (x or y NULL), MISALIGNED (4 bytes), WORKSPACE (an
 * external workspace is set and too small), UNSUPPORTED_DEVICE, CUDA.
 */
int cudallm_layernorm_f32(const float *x, const float *gamma, const float *beta, float *y, int64_t batch,
                          int64_t m, float eps, void *stream);

#ifdef __cplusplus
}
#endif

#endif /* CUDALLM_TASKS_H */
