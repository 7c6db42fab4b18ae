// Small helper kernels around the tcgen05 path:
//  * simt_gemm_kernel  -- fully predicated CUDA-core GEMM for any shape and
//    alignment (bring-up cross-check on the device; also serves K == 0).
//  * pack_rows_kernel  -- copies operands whose leading dimension or base
//    is not 16-byte aligned into an aligned workspace so that TMA can read them.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"

namespace cudallm {

// One thread per element of C; fp32 FMA accumulation in ascending k
// (Task 2's definition taken literally).  blockIdx.z strides over the batch.
template <bool OUT_BF16>
__global__ void __launch_bounds__(256)
simt_gemm_kernel(const __nv_bfloat16 *__restrict__ A, const __nv_bfloat16 *__restrict__ B, void *C,
                 int M, int N, int K, long long lda, long long ldb, long long ldc,
                 long long strideA, long long strideB, long long strideC, int batch)
{
    const int col = blockIdx.x * 16 + (threadIdx.x & 15);
    const long long row0 = static_cast<long long>(blockIdx.y) * 16 + (threadIdx.x >> 4);
    for (int b = blockIdx.z; b < batch; b += gridDim.z) {
        const __nv_bfloat16 *Ab = A + b * strideA;
        const __nv_bfloat16 *Bb = B + b * strideB;
        for (long long row = row0; row < M; row += static_cast<long long>(gridDim.y) * 16) {
            if (col >= N) continue;
            float acc = 0.f;
            for (int k = 0; k < K; ++k)
                acc = fmaf(__bfloat162float(Ab[row * lda + k]), __bfloat162float(Bb[k * ldb + col]), acc);
            const long long off = b * strideC + row * ldc + col;
            if (OUT_BF16) reinterpret_cast<__nv_bfloat16 *>(C)[off] = __float2bfloat16_rn(acc);
            else          reinterpret_cast<float *>(C)[off] = acc;
        }
    }
}

// One operand to repack: dst[b][r][0..cols) = src[b][r][0..cols), columns up to the next
// multiple of 8 zero; dst is 16-byte aligned and its row pitch ld_dst and batch stride are
// multiples of 8 elements; src needs 2-byte alignment only.
struct PackJob {
    const uint16_t *src;
    uint16_t *dst;
    int rows, cols, batch;
    long long ld_src, ld_dst, stride_src, stride_dst;
    long long total_rows;                                // rows * batch (0 = nothing to do)
};

// Repacks up to two operands in one launch: one thread per 16-byte piece of the
// destination, the pieces of job a first, then those of job b.  A piece whose source lies
// strictly inside its row is read as five 4-byte words from the 4-byte boundary at or
// below it and shifted into place (the source of a row with an odd pitch is 2 bytes past
// such a boundary every other row); the first and the last piece of a row are read element
// by element, so that nothing outside [src, src + cols) of the row is touched.
__global__ void __launch_bounds__(256)
pack_rows_kernel(const PackJob a, const PackJob b)
{
    grid_launch_dependents();
    grid_dependency_wait();                              // the workspace may still be read by the previous kernel
    const long long pieces_a = a.total_rows * ((a.cols + 7) >> 3);
    const long long total = pieces_a + b.total_rows * ((b.cols + 7) >> 3);
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const bool first = i < pieces_a;
        const long long k = first ? i : i - pieces_a;
        const int rows = first ? a.rows : b.rows;
        const int cols = first ? a.cols : b.cols;
        const int chunks = (cols + 7) >> 3;
        const long long row = k / chunks;
        const int c0 = static_cast<int>(k - row * chunks) * 8;
        const long long item = row / rows;
        const long long r = row - item * rows;
        const uint16_t *s = (first ? a.src : b.src) + item * (first ? a.stride_src : b.stride_src)
                          + r * (first ? a.ld_src : b.ld_src) + c0;
        uint16_t *d = (first ? a.dst : b.dst) + item * (first ? a.stride_dst : b.stride_dst)
                    + r * (first ? a.ld_dst : b.ld_dst) + c0;
        uint4 w;
        if (c0 > 0 && c0 + 10 <= cols) {
            const uint32_t odd = (reinterpret_cast<uintptr_t>(s) >> 1) & 1;
            const uint32_t *q = reinterpret_cast<const uint32_t *>(s - odd);
            const uint32_t w0 = q[0], w1 = q[1], w2 = q[2], w3 = q[3], w4 = q[4];
            const uint32_t sh = odd * 16;
            w.x = __funnelshift_r(w0, w1, sh);
            w.y = __funnelshift_r(w1, w2, sh);
            w.z = __funnelshift_r(w2, w3, sh);
            w.w = __funnelshift_r(w3, w4, sh);
        } else {
            uint16_t v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = (c0 + j < cols) ? s[j] : static_cast<uint16_t>(0);
            w.x = v[0] | (static_cast<uint32_t>(v[1]) << 16);
            w.y = v[2] | (static_cast<uint32_t>(v[3]) << 16);
            w.z = v[4] | (static_cast<uint32_t>(v[5]) << 16);
            w.w = v[6] | (static_cast<uint32_t>(v[7]) << 16);
        }
        *reinterpret_cast<uint4 *>(d) = w;
    }
}

// Cuts fp32 values into three bf16 pieces: x = p0 + p1 + p2 exactly for normal
// numbers whose exponent leaves room for the low piece (p0 = bf16(x), p1 =
// bf16(x - p0), p2 = bf16(x - p0 - p1); both differences are exact in fp32, and
// three 8-bit significands cover fp32's 24 bits).  dst holds the pieces as three
// matrices `piece_stride` elements apart, rows ld_dst apart (a multiple of 8),
// columns beyond `cols` zero.  One thread converts 8 consecutive elements.
__global__ void __launch_bounds__(256)
split3_rows_kernel(const float *__restrict__ src, uint16_t *__restrict__ dst, int rows, int cols,
                   long long ld_src, long long ld_dst, long long piece_stride)
{
    grid_launch_dependents();
    grid_dependency_wait();
    const int chunks = (cols + 7) >> 3;
    const long long total = static_cast<long long>(rows) * chunks;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int r = static_cast<int>(i / chunks);
        const int c0 = static_cast<int>(i - static_cast<long long>(r) * chunks) * 8;
        const float *s = src + r * ld_src + c0;
        uint32_t w[3][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float x = (c0 + j < cols) ? s[j] : 0.f;
            const __nv_bfloat16 p0 = __float2bfloat16_rn(x);
            const float r1 = x - __bfloat162float(p0);
            const __nv_bfloat16 p1 = __float2bfloat16_rn(r1);
            const float r2 = r1 - __bfloat162float(p1);
            const __nv_bfloat16 p2 = __float2bfloat16_rn(r2);
            const uint32_t b[3] = {__bfloat16_as_ushort(p0), __bfloat16_as_ushort(p1), __bfloat16_as_ushort(p2)};
#pragma unroll
            for (int q = 0; q < 3; ++q) {
                if (j & 1) w[q][j >> 1] |= b[q] << 16;
                else       w[q][j >> 1] = b[q];
            }
        }
        uint16_t *d = dst + r * ld_dst + c0;
#pragma unroll
        for (int q = 0; q < 3; ++q)
            *reinterpret_cast<uint4 *>(d + q * piece_stride) = make_uint4(w[q][0], w[q][1], w[q][2], w[q][3]);
    }
}

}  // namespace cudallm
