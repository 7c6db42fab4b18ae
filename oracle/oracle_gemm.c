/*
 * CPU oracle for the dense contraction C = A x B (the paper's benchmark Task 2,
 * "Matrix Multiplication": A is M x K, B is K x N, C is M x N, all row-major).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code with the CUDA path and
 * must never be called from the product path.
 *
 * Inputs are raw bfloat16 bit patterns (uint16_t).  A bfloat16 is the upper 16
 * bits of an IEEE binary32, so widening to double is exact; a product of two
 * bfloat16 values has at most 16 significant bits and is exact in double; the
 * only rounding is in the fp64 running sum (taken in ascending k).
 *
 * Besides C the oracle returns S[i][j] = sum_k |A[i][k]| * |B[k][j]|, the scale
 * that the element-wise tolerance |C_gpu - C_ref| <= tol * S is stated against.
 *
 * parity unpinned: nothing.  Every function here is pinned by tests against
 * identity / permutation operands, integer rank-1 closed forms, hand-computed
 * literals, an fp64 library product and a second, independently ordered loop.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* bfloat16 bits -> double, exactly (Task 2 operands; widening only). */
static inline double bf16_bits_to_double(uint16_t h)
{
    uint32_t w = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/*
 * Brute force: the definition written out, one output element at a time,
 * i - j - k order, scalar.  Task 2: C[i][j] = sum_{k<K} A[i][k] * B[k][j].
 * Single-threaded; meant for tiny shapes and for cross-checking the faster
 * loop below bit for bit.
 */
void oracle_gemm_bf16_naive(const uint16_t *A, const uint16_t *B,
                            double *C, double *S,
                            int64_t M, int64_t N, int64_t K,
                            int64_t lda, int64_t ldb)
{
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double c = 0.0, s = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double a = bf16_bits_to_double(A[i * lda + k]);
                double b = bf16_bits_to_double(B[k * ldb + j]);
                c += a * b;
                s += fabs(a) * fabs(b);
            }
            C[i * N + j] = c;
            if (S) S[i * N + j] = s;
        }
    }
}

/*
 * The same triple loop in i - k - j order (j contiguous), rows of C spread
 * over the host threads.  Every element still sums its K products in
 * ascending k, so the result is bit-identical to the brute force above.
 * C and S are dense M x N (leading dimension N).  S may be NULL.
 */
void oracle_gemm_bf16(const uint16_t *A, const uint16_t *B,
                      double *C, double *S,
                      int64_t M, int64_t N, int64_t K,
                      int64_t lda, int64_t ldb)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < M; ++i) {
        double *c = C + i * N;
        double *s = S ? S + i * N : NULL;
        for (int64_t j = 0; j < N; ++j) c[j] = 0.0;
        if (s) for (int64_t j = 0; j < N; ++j) s[j] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            const double a = bf16_bits_to_double(A[i * lda + k]);
            const double aa = fabs(a);
            const uint16_t *b = B + k * ldb;
            if (s) {
                for (int64_t j = 0; j < N; ++j) {
                    double bj = bf16_bits_to_double(b[j]);
                    c[j] += a * bj;
                    s[j] += aa * fabs(bj);
                }
            } else {
                for (int64_t j = 0; j < N; ++j)
                    c[j] += a * bf16_bits_to_double(b[j]);
            }
        }
    }
}

/*
 * Selected rows only: row r of the output (r < nrows) is row rows[r] of the
 * full product.  Lets the full-size configurations be checked on a sample of
 * rows when the whole product would take minutes.  C and S are nrows x N.
 */
void oracle_gemm_bf16_rows(const uint16_t *A, const uint16_t *B,
                           double *C, double *S,
                           const int64_t *rows, int64_t nrows,
                           int64_t N, int64_t K,
                           int64_t lda, int64_t ldb)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < nrows; ++r) {
        const int64_t i = rows[r];
        double *c = C + r * N;
        double *s = S ? S + r * N : NULL;
        for (int64_t j = 0; j < N; ++j) c[j] = 0.0;
        if (s) for (int64_t j = 0; j < N; ++j) s[j] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            const double a = bf16_bits_to_double(A[i * lda + k]);
            const double aa = fabs(a);
            const uint16_t *b = B + k * ldb;
            for (int64_t j = 0; j < N; ++j) {
                double bj = bf16_bits_to_double(b[j]);
                c[j] += a * bj;
                if (s) s[j] += aa * fabs(bj);
            }
        }
    }
}

/*
 * Batched: `batch` independent products; item t reads A + t*strideA and
 * B + t*strideB (strides in elements) and writes the dense M x N block t of C
 * (and of S).  Items are computed one after another with the loop above.
 */
void oracle_gemm_bf16_batched(const uint16_t *A, const uint16_t *B,
                              double *C, double *S,
                              int64_t M, int64_t N, int64_t K,
                              int64_t lda, int64_t ldb,
                              int64_t strideA, int64_t strideB,
                              int64_t batch)
{
    for (int64_t t = 0; t < batch; ++t)
        oracle_gemm_bf16(A + t * strideA, B + t * strideB,
                         C + t * M * N, S ? S + t * M * N : NULL,
                         M, N, K, lda, ldb);
}

/*
 * The paper's Task 2 as printed: both operands hold 32-bit floating point
 * numbers.  C[i][j] = sum_{k<K} A[i][k] * B[k][j] with the fp32 values widened
 * to double (exact) -- a product of two fp32 values has at most 48 significant
 * bits and is exact in double; the only rounding is in the fp64 running sum,
 * taken in ascending k.  S as above.  i - k - j order, rows over the threads.
 */
void oracle_gemm_f32(const float *A, const float *B, double *C, double *S,
                     int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < M; ++i) {
        double *c = C + i * N;
        double *s = S ? S + i * N : NULL;
        for (int64_t j = 0; j < N; ++j) c[j] = 0.0;
        if (s) for (int64_t j = 0; j < N; ++j) s[j] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            const double a = (double)A[i * lda + k];
            const double aa = fabs(a);
            const float *b = B + k * ldb;
            for (int64_t j = 0; j < N; ++j) {
                const double bj = (double)b[j];
                c[j] += a * bj;
                if (s) s[j] += aa * fabs(bj);
            }
        }
    }
}

/* The same, one element at a time (i - j - k), single-threaded: brute force. */
void oracle_gemm_f32_naive(const float *A, const float *B, double *C, double *S,
                           int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb)
{
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j) {
            double c = 0.0, s = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                const double a = (double)A[i * lda + k], b = (double)B[k * ldb + j];
                c += a * b;
                s += fabs(a) * fabs(b);
            }
            C[i * N + j] = c;
            if (S) S[i * N + j] = s;
        }
}

/* Selected rows of the fp32 product (see oracle_gemm_bf16_rows). */
void oracle_gemm_f32_rows(const float *A, const float *B, double *C, double *S,
                          const int64_t *rows, int64_t nrows, int64_t N, int64_t K,
                          int64_t lda, int64_t ldb)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < nrows; ++r) {
        const int64_t i = rows[r];
        double *c = C + r * N;
        double *s = S ? S + r * N : NULL;
        for (int64_t j = 0; j < N; ++j) c[j] = 0.0;
        if (s) for (int64_t j = 0; j < N; ++j) s[j] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            const double a = (double)A[i * lda + k];
            const double aa = fabs(a);
            const float *b = B + k * ldb;
            for (int64_t j = 0; j < N; ++j) {
                const double bj = (double)b[j];
                c[j] += a * bj;
                if (s) s[j] += aa * fabs(bj);
            }
        }
    }
}

/* Number of host threads the parallel loops above will use. */
int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
