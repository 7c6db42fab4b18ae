/*
 * CPU oracle for the bandwidth-bound benchmark tasks of the paper that work on
 * 32-bit floating point arrays: Task 8 (matrix transpose), Task 14 (reduction:
 * sum of an array), Task 15 (dot product) and Task 4 (LayerNorm).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code with the CUDA path and
 * must never be called from the product path.
 *
 * Every floating-point quantity is computed in double.  A float widens to
 * double exactly, the product of two floats is exact in double, so the only
 * roundings are those of the running double sums (ascending index order) and,
 * for LayerNorm, of the division and the square root.
 *
 * parity unpinned: nothing.  The transpose is pinned by index-map closed forms,
 * involution and a library transpose; the sum and the dot product by integer
 * closed forms (Gauss sums, sums of squares), hand-computed literals, an exactly
 * rounded library sum and invariances; LayerNorm by closed forms on two-valued
 * and arithmetic-progression samples, by the zero-mean / unit-variance property
 * of its output and by an fp64 library computation.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

/*
 * Task 8: AT[j][i] = A[i][j] for i < rows, j < cols; A is rows x cols with row
 * pitch lda, AT is cols x rows with row pitch ldat (pitches in elements).
 * Pure data movement: values are copied bit for bit.
 */
void oracle_transpose_f32(const float *A, float *AT, int64_t rows, int64_t cols,
                          int64_t lda, int64_t ldat)
{
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j)
            AT[j * ldat + i] = A[i * lda + j];
}

/*
 * Task 14: the sum of the n elements of x, in ascending index order, in
 * double.  *sum_abs (may be NULL) receives sum_i |x_i|, the scale the
 * tolerance is stated against.
 */
double oracle_sum_f32(const float *x, int64_t n, double *sum_abs)
{
    double s = 0.0, a = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        s += (double)x[i];
        a += fabs((double)x[i]);
    }
    if (sum_abs) *sum_abs = a;
    return s;
}

/*
 * Task 15: A . B = sum_{i<n} A_i * B_i, ascending i, in double (each product is
 * exact).  *sum_abs (may be NULL) receives sum_i |A_i| |B_i|.
 */
double oracle_dot_f32(const float *a, const float *b, int64_t n, double *sum_abs)
{
    double s = 0.0, t = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        const double p = (double)a[i] * (double)b[i];
        s += p;
        t += fabs(p);
    }
    if (sum_abs) *sum_abs = t;
    return s;
}

/*
 * Task 4: LayerNorm of `batch` samples of `m` elements each (m = features *
 * dim1 * dim2, the sample flattened).  For sample s:
 *     mean = (1/m) sum_i x[s][i]
 *     var  = (1/m) sum_i (x[s][i] - mean)^2          (the biased estimate)
 *     y[s][i] = (x[s][i] - mean) / sqrt(var + eps) * gamma[i] + beta[i]
 * gamma and beta have m elements (one per position of a sample) and may be
 * NULL (then 1 and 0).  y is written as double.  mean_out / rstd_out (may be
 * NULL) receive the per-sample mean and 1 / sqrt(var + eps).
 */
void oracle_layernorm_f32(const float *x, const float *gamma, const float *beta,
                          double *y, int64_t batch, int64_t m, double eps,
                          double *mean_out, double *rstd_out)
{
    for (int64_t s = 0; s < batch; ++s) {
        const float *xs = x + s * m;
        double sum = 0.0;
        for (int64_t i = 0; i < m; ++i) sum += (double)xs[i];
        const double mean = m ? sum / (double)m : 0.0;
        double sq = 0.0;
        for (int64_t i = 0; i < m; ++i) {
            const double d = (double)xs[i] - mean;
            sq += d * d;
        }
        const double var = m ? sq / (double)m : 0.0;
        const double rstd = 1.0 / sqrt(var + eps);
        for (int64_t i = 0; i < m; ++i) {
            const double g = gamma ? (double)gamma[i] : 1.0;
            const double b = beta ? (double)beta[i] : 0.0;
            y[s * m + i] = ((double)xs[i] - mean) * rstd * g + b;
        }
        if (mean_out) mean_out[s] = mean;
        if (rstd_out) rstd_out[s] = rstd;
    }
}
