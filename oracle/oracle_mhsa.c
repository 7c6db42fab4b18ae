/*
 * CPU oracle for the paper's benchmark Task 6, "Multi-Head Self-Attention":
 *
 *   MultiHead(Q, K, V) = Concat(head_1, ..., head_h),
 *   head_i = softmax(Q_i K_i^T / sqrt(d_k)) V_i,   d_k = d_model / h,
 *
 * with Q, K, V of size N x d_model (row-major) and Q_i, K_i, V_i the i-th
 * head's partition of the input matrices.  Reading taken: the partition is by
 * columns -- head i owns columns [i d_k, (i+1) d_k) -- and Concat places head
 * i's output in the same columns; softmax runs over the keys (each row of the
 * N x N score matrix sums to one).
 *
 * THIS FILE IS TEST INFRASTRUCTURE: the plain definition in fp64, one query at
 * a time, sharing no code with the CUDA path.  Operands are bfloat16 bit
 * patterns (widened exactly).  Besides the output it returns
 * T[i][c] = sum_j p_ij |V[j][c]|, the scale the element-wise tolerance is
 * stated against.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline double bf16_to_double(uint16_t h)
{
    uint32_t w = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* out and T are dense N x d_model.  Returns 0, or -1 if h does not divide d_model. */
int oracle_mhsa_bf16(const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                     double *out, double *T,
                     int64_t N, int64_t d_model, int64_t h,
                     int64_t ldq, int64_t ldk, int64_t ldv)
{
    if (h <= 0 || d_model % h) return -1;
    const int64_t dk = d_model / h;
    const double scale = 1.0 / sqrt((double)dk);
#pragma omp parallel
    {
        double *p = (double *)malloc((size_t)(N > 0 ? N : 1) * sizeof(double));
#pragma omp for collapse(2) schedule(static)
        for (int64_t head = 0; head < h; ++head) {
            for (int64_t i = 0; i < N; ++i) {
                const int64_t c0 = head * dk;
                /* scores of query i against every key, then a max-shifted softmax */
                double m = -INFINITY;
                for (int64_t j = 0; j < N; ++j) {
                    double s = 0.0;
                    for (int64_t d = 0; d < dk; ++d)
                        s += bf16_to_double(Q[i * ldq + c0 + d]) * bf16_to_double(K[j * ldk + c0 + d]);
                    p[j] = s * scale;
                    if (p[j] > m) m = p[j];
                }
                double z = 0.0;
                for (int64_t j = 0; j < N; ++j) {
                    p[j] = exp(p[j] - m);
                    z += p[j];
                }
                for (int64_t d = 0; d < dk; ++d) {
                    double o = 0.0, t = 0.0;
                    for (int64_t j = 0; j < N; ++j) {
                        const double v = bf16_to_double(V[j * ldv + c0 + d]);
                        o += p[j] * v;
                        t += p[j] * fabs(v);
                    }
                    out[i * d_model + c0 + d] = o / z;
                    if (T) T[i * d_model + c0 + d] = t / z;
                }
            }
        }
        free(p);
    }
    return 0;
}
