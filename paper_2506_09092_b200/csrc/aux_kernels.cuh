// Small helper kernels around the tcgen05 path:
//  * simt_gemm_kernel  -- fully predicated CUDA-core GEMM for any shape and
//    alignment (bring-up cross-check on the device; also serves K == 0).
//  * pack_rows_kernel  -- copies operands whose leading dimension or base
//    is not 16-byte aligned into an aligned workspace so that TMA can read them
//    (the row copies themselves are in row_copy.cuh).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"
#include "row_copy.cuh"

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

// Repacks up to two operands in one launch.  The unit of work is up to 512 consecutive
// elements of one row, copied by one warp with 16-byte loads and stores (row_copy.cuh); the
// units of job a come first, then those of job b, and the warps of the grid take them in
// turn.  Eight warps per CTA and as many CTAs as fit: the copy then runs at about 80 % of
// what a plain device-to-device copy of the same bytes reaches.
constexpr int kPackThreads = 256;
// The units of one job, taken in turn by the warps of the grid starting with warp `first_warp`
// (so that job b's units continue where job a's ended).  Index = uint32_t where the unit
// count allows it: its divisions are several times cheaper.
template <typename Index>
__device__ __forceinline__ void pack_job_units(const PackJob &j, Index first_warp, Index nwarps, int lane)
{
    const Index groups = static_cast<Index>((j.cols + 511) >> 9);
    const Index total = static_cast<Index>(j.total_rows) * groups;
    const Index rows = static_cast<Index>(j.rows);
    const int cols = j.cols;
    const long long ld_src = j.ld_src, ld_dst = j.ld_dst, s_src = j.stride_src, s_dst = j.stride_dst;
    const bool batched = j.batch > 1;
    for (Index u = first_warp; u < total; u += nwarps) {
        const Index row = groups == 1 ? u : u / groups;
        const int c0 = static_cast<int>(u - row * groups) * 512;
        long long off_src, off_dst;
        if (batched) {
            const Index item = row / rows, r = row - item * rows;
            off_src = item * s_src + r * ld_src + c0;
            off_dst = item * s_dst + r * ld_dst + c0;
        } else {
            off_src = row * ld_src + c0;
            off_dst = row * ld_dst + c0;
        }
        const uint16_t *src = j.src + off_src;
        uint16_t *dst = j.dst + off_dst;
        if (cols - c0 >= 514) {                          // warp-uniform: not the last unit of its row
            row_copy_interior(src, dst, lane);
        } else {
            RowCopy rc;
            row_copy_load(rc, src, cols - c0, lane);
            row_copy_store(rc, src, dst, cols - c0, lane);
        }
    }
}
template <typename Index>
__device__ __forceinline__ void pack_rows_loop(const PackJob &a, const PackJob &b)
{
    const int lane = threadIdx.x & 31;
    const Index nwarps = static_cast<Index>(gridDim.x) * (kPackThreads / 32);
    const Index gwarp = static_cast<Index>(blockIdx.x) * (kPackThreads / 32) + (threadIdx.x >> 5);
    pack_job_units<Index>(a, gwarp, nwarps, lane);
    // job b starts with the warp after the one that took job a's last unit
    const Index units_a = static_cast<Index>(a.total_rows) * static_cast<Index>((a.cols + 511) >> 9);
    const Index shift = units_a % nwarps;
    pack_job_units<Index>(b, gwarp >= shift ? gwarp - shift : gwarp + nwarps - shift, nwarps, lane);
}
__global__ void __launch_bounds__(kPackThreads)
pack_rows_kernel(const PackJob a, const PackJob b)
{
    grid_launch_dependents();
    grid_dependency_wait();                              // the workspace may still be read by the previous kernel
    const unsigned long long total = static_cast<unsigned long long>(a.total_rows) * ((a.cols + 511) >> 9)
                                   + static_cast<unsigned long long>(b.total_rows) * ((b.cols + 511) >> 9);
    const unsigned long long reach = total + static_cast<unsigned long long>(gridDim.x) * (kPackThreads / 32);
    if (reach < (1ull << 32)) pack_rows_loop<uint32_t>(a, b);
    else                      pack_rows_loop<unsigned long long>(a, b);
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
