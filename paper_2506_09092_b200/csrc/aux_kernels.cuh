// Small helper kernels around the tcgen05 path:
//  * simt_gemm_kernel  -- fully predicated CUDA-core GEMM for any shape and
//    alignment (bring-up cross-check on the device; also serves K == 0).
//  * pack_rows_kernel  -- copies an operand whose leading dimension or base
//    is not 16-byte aligned into an aligned workspace so that TMA can read it.
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

// dst[b][r][0..cols) = src[b][r][0..cols); dst row stride ld_dst is a multiple
// of 8 elements and dst is 16-byte aligned.  One thread moves 8 elements.
__global__ void __launch_bounds__(256)
pack_rows_kernel(const uint16_t *__restrict__ src, uint16_t *__restrict__ dst,
                 int rows, int cols, long long ld_src, long long ld_dst,
                 long long stride_src, long long stride_dst, int batch)
{
    grid_launch_dependents();
    grid_dependency_wait();                              // the workspace may still be read by the previous kernel
    const int chunks = (cols + 7) >> 3;
    const long long per_item = static_cast<long long>(rows) * chunks;
    const long long total = per_item * batch;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int b = static_cast<int>(i / per_item);
        const long long rem = i - b * per_item;
        const int r = static_cast<int>(rem / chunks);
        const int c0 = static_cast<int>(rem - static_cast<long long>(r) * chunks) * 8;
        const uint16_t *s = src + b * stride_src + r * ld_src + c0;
        uint16_t v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (c0 + j < cols) ? s[j] : static_cast<uint16_t>(0);
        uint4 w;
        w.x = v[0] | (static_cast<uint32_t>(v[1]) << 16);
        w.y = v[2] | (static_cast<uint32_t>(v[3]) << 16);
        w.z = v[4] | (static_cast<uint32_t>(v[5]) << 16);
        w.w = v[6] | (static_cast<uint32_t>(v[7]) << 16);
        *reinterpret_cast<uint4 *>(dst + b * stride_dst + r * ld_dst + c0) = w;
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
