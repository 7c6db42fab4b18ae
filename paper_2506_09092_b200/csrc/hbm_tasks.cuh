// Bandwidth-bound kernels for the paper's benchmark tasks on float32 arrays:
// Task 8 (matrix transpose), Task 14 (reduction: sum), Task 15 (dot product)
// and Task 4 (LayerNorm).  None of them is a contraction; what matters is that
// every byte crosses HBM once, in full cache lines, with enough of them in
// flight.
#pragma once
#include "ptx.cuh"

namespace cudallm {

// status detail codes of these kernels: (role << 8) | what
enum : int { kRoleLayerNorm = 5 };

__device__ __forceinline__ void task_report_timeout(int *status, int role, int what)
{
    if (atomicCAS(status, 0, -9 /* CUDALLM_ERR_DEVICE_TIMEOUT */) == 0) status[1] = (role << 8) | what;
}

// -------------------------------------------------------- mbarrier helper --
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// ============================================================== Task 8 ====
// AT[j][i] = A[i][j].  One CTA of 256 threads per 64 x 64 tile: 16-byte loads
// along the rows of A (sixteen threads cover the 256 contiguous bytes of a tile
// row), a padded shared tile (65 floats per row: the column reads below are
// conflict-free), 16-byte stores along the rows of AT (again 256 contiguous
// bytes per tile row).  No persistence and 17 KB of shared memory per CTA, so a
// dozen CTAs per SM overlap each other's latencies.
// Measured on B200 at 16384 x 16384: this kernel 6.5 TB/s (the speed of a plain
// copy); the same with 32 x 32 tiles (128-byte segments) 5.2 TB/s; a
// warp-specialised version with TMA loads of 64 x 64 patches, a turn in shared
// memory and TMA stores of 32 x 32 swizzled boxes 5.4 TB/s whatever its ring
// depth, warp count or patch order -- the 128-byte pieces on the store side
// were the limit, not the SM.  rows and cols are multiples of 4 on this path and
// the bases and pitches 16-byte aligned; edge tiles are predicated per 16 bytes.
__global__ void __launch_bounds__(256)
transpose64_kernel(const float *__restrict__ A, float *__restrict__ AT, int rows, int cols, long long lda,
                   long long ldat, int tiles_c)
{
    __shared__ float tile[64][65];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;          // 16 x 16 threads
    const int tr = blockIdx.x / tiles_c, tc = blockIdx.x - tr * tiles_c;
    const int r0 = tr * 64, c0 = tc * 64;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int r = ty + 16 * k;
        if (r0 + r < rows && c0 + 4 * tx < cols) {
            const float4 v = *reinterpret_cast<const float4 *>(A + (r0 + r) * lda + c0 + 4 * tx);
            tile[r][4 * tx] = v.x; tile[r][4 * tx + 1] = v.y; tile[r][4 * tx + 2] = v.z; tile[r][4 * tx + 3] = v.w;
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int c = ty + 16 * k;                                   // row of AT inside the tile
        if (c0 + c < cols && r0 + 4 * tx < rows) {
            const float4 v = make_float4(tile[4 * tx][c], tile[4 * tx + 1][c], tile[4 * tx + 2][c], tile[4 * tx + 3][c]);
            *reinterpret_cast<float4 *>(AT + (c0 + c) * ldat + r0 + 4 * tx) = v;
        }
    }
}

// Any shape, pitch and alignment: 32 x 32 tiles through a padded shared tile.
__global__ void __launch_bounds__(256)
transpose_simple_kernel(const float *__restrict__ A, float *__restrict__ AT, int rows, int cols,
                        long long lda, long long ldat, int tiles_c, long long tiles)
{
    __shared__ float tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;          // 32 x 8
    for (long long t = blockIdx.x; t < tiles; t += gridDim.x) {
        const int tr = static_cast<int>(t / tiles_c), tc = static_cast<int>(t - static_cast<long long>(tr) * tiles_c);
        const int r0 = tr * 32, c0 = tc * 32;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int r = r0 + ty + 8 * k, c = c0 + tx;
            if (r < rows && c < cols) tile[ty + 8 * k][tx] = A[r * lda + c];
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int c = c0 + ty + 8 * k, r = r0 + tx;               // AT[c][r]
            if (r < rows && c < cols) AT[c * ldat + r] = tile[tx][ty + 8 * k];
        }
        __syncthreads();
    }
}

// ===================================================== Tasks 14 and 15 ====
// sum_i x_i  and  sum_i a_i b_i.  Every element is widened to double (exact)
// and accumulated in double, so the result is the exactly rounded sum up to
// ~1e-13 of sum |terms|, whatever the order; it is rounded to float32 once.
// Threads stride over the array in 16-byte pieces, four loads in flight each;
// a block leaves one partial in scratch; the block that arrives last (a ticket
// counter) adds the partials in index order and resets the ticket, so one
// launch does the whole job and equal inputs give bit-equal results.
constexpr int kRedThreads = 512;
constexpr int kRedMaxBlocks = 1024;

struct ReduceScratch {
    double partial[kRedMaxBlocks];
    unsigned int ticket;
};

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum of `v` over the block in a fixed order; valid in thread 0.
__device__ __forceinline__ double block_sum(double v, double *warp_part)
{
    v = warp_sum(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) warp_part[warp] = v;
    __syncthreads();
    double t = 0.0;
    if (warp == 0) {
        t = lane < (blockDim.x >> 5) ? warp_part[lane] : 0.0;
        t = warp_sum(t);
    }
    __syncthreads();
    return t;
}

__device__ __forceinline__ float4 ldg_stream(const float4 *p)
{
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

// DOT = false: sum of a;  DOT = true: a . b.  `head` leading elements (until a
// is 16-byte aligned; b must share a's misalignment on the vector path, else
// VEC = false) and the tail are taken one by one.
template <bool DOT, bool VEC>
__global__ void __launch_bounds__(kRedThreads)
reduce_kernel(const float *__restrict__ a, const float *__restrict__ b, long long n, float *result,
              ReduceScratch *scratch)
{
    __shared__ double warp_part[kRedThreads / 32];
    __shared__ bool is_last;
    const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long long nthreads = static_cast<long long>(gridDim.x) * blockDim.x;
    double acc0 = 0.0, acc1 = 0.0, acc2 = 0.0, acc3 = 0.0;

    long long head = 0, nvec = 0;
    if (VEC) {
        head = ((16 - (reinterpret_cast<uintptr_t>(a) & 15)) & 15) >> 2;
        if (head > n) head = n;
        nvec = (n - head) >> 2;
        const float4 *av = reinterpret_cast<const float4 *>(a + head);
        const float4 *bv = reinterpret_cast<const float4 *>(b + head);
        long long i = tid;
        // four independent 16-byte loads (eight for the dot product) in flight per thread
        for (; i + 3 * nthreads < nvec; i += 4 * nthreads) {
            float4 x[4], y[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) x[u] = ldg_stream(av + i + u * nthreads);
            if (DOT) {
#pragma unroll
                for (int u = 0; u < 4; ++u) y[u] = ldg_stream(bv + i + u * nthreads);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (DOT) {
                    acc0 = fma(static_cast<double>(x[u].x), static_cast<double>(y[u].x), acc0);
                    acc1 = fma(static_cast<double>(x[u].y), static_cast<double>(y[u].y), acc1);
                    acc2 = fma(static_cast<double>(x[u].z), static_cast<double>(y[u].z), acc2);
                    acc3 = fma(static_cast<double>(x[u].w), static_cast<double>(y[u].w), acc3);
                } else {
                    acc0 += static_cast<double>(x[u].x);
                    acc1 += static_cast<double>(x[u].y);
                    acc2 += static_cast<double>(x[u].z);
                    acc3 += static_cast<double>(x[u].w);
                }
            }
        }
        for (; i < nvec; i += nthreads) {
            const float4 x = ldg_stream(av + i);
            if (DOT) {
                const float4 y = ldg_stream(bv + i);
                acc0 = fma(static_cast<double>(x.x), static_cast<double>(y.x), acc0);
                acc1 = fma(static_cast<double>(x.y), static_cast<double>(y.y), acc1);
                acc2 = fma(static_cast<double>(x.z), static_cast<double>(y.z), acc2);
                acc3 = fma(static_cast<double>(x.w), static_cast<double>(y.w), acc3);
            } else {
                acc0 += static_cast<double>(x.x);
                acc1 += static_cast<double>(x.y);
                acc2 += static_cast<double>(x.z);
                acc3 += static_cast<double>(x.w);
            }
        }
    }
    // elements outside the vector body: [0, head) and [head + 4 nvec, n)
    const long long tail0 = head + 4 * nvec;
    for (long long i = tid; i < head + (n - tail0); i += nthreads) {
        const long long k = i < head ? i : tail0 + (i - head);
        acc0 += DOT ? static_cast<double>(a[k]) * static_cast<double>(b[k]) : static_cast<double>(a[k]);
    }

    const double block_total = block_sum((acc0 + acc1) + (acc2 + acc3), warp_part);
    if (threadIdx.x == 0) {
        scratch->partial[blockIdx.x] = block_total;
        __threadfence();
        const unsigned int t = atomicAdd(&scratch->ticket, 1u);
        is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (is_last) {
        __threadfence();
        double v = 0.0;
        for (int i = threadIdx.x; i < static_cast<int>(gridDim.x); i += blockDim.x)
            v += __ldcg(&scratch->partial[i]);
        const double total = block_sum(v, warp_part);
        if (threadIdx.x == 0) {
            *result = static_cast<float>(total);
            scratch->ticket = 0;                         // ready for the next launch
        }
    }
}

// ============================================================== Task 4 ====
// y[s][i] = (x[s][i] - mean_s) / sqrt(var_s + eps) * gamma[i] + beta[i] with the
// mean and the (biased) variance taken over the m elements of sample s.
//
// Work split.  A group of G CTAs owns a sample; CTA g of the group works on
// elements [g * slice, (g + 1) * slice) of it.  Samples are taken T at a time (a
// "bundle", T <= 16): the CTAs compute their moments of the T slices, publish
// them, meet once (a bounded wait on a counter in global memory; the grid never
// exceeds what is resident at once), combine everybody's moments -- the same
// arithmetic in the same order in every CTA -- and normalise the T slices.
//
// Arithmetic.  The fp64 pipe of this GPU is slow (a conversion, an add and a
// multiply-add in double per element cap a streaming kernel at ~4 TB/s), so the
// moments are taken in float32 about a pilot value c (the mean of the first
// eight elements of the CTA's slice, so that x - c is of the size of the data's
// spread, not of its offset): per 32-byte piece, d_j = x_j - c, f1 = sum d_j,
// f2 = sum d_j^2 in float32, and f1, f2 are added to double accumulators (1/4
// double operation per element).  A CTA publishes A = n c + S1 (its sum of x),
// its own mean A / n and B = S2 - S1^2 / n (its sum of squared deviations about
// that mean); the combination is mean = sum A_k / m and
// M2 = sum (B_k + n_k (mean_k - mean)^2): no large numbers are subtracted
// anywhere, so a mean far larger than the spread costs no accuracy.
// Pass 2 is float32 on a two-float mean (ln_apply).
//
// Two kernels:
//  * layernorm_smem_kernel: the T slices of a bundle sit in shared memory between
//    the passes (bulk copies, no registers or warps needed to fetch them); x
//    crosses HBM once.  Used when the whole batch takes at most two bundles per
//    group.
//  * layernorm_stream_kernel: the slices are read from global memory in both
//    passes, the second time in reverse order (what was read last is still in
//    L2) and two samples at a time so that gamma and beta are fetched once per
//    pair.  x crosses HBM up to twice, but the memory system is never idle
//    waiting for a meeting per sample.  Also the path for unaligned data.
struct LayerNormParams {
    const float *x, *gamma, *beta;
    float *y;
    long long m;             // elements per sample
    long long slice;         // shared-memory kernel: elements of shared memory per sample (whole 4 KiB
                             // blocks); streaming kernel, unaligned data: elements per CTA
    int batch;
    int group_size;          // G
    int num_groups;          // groups that run side by side; grid = num_groups * G
    int bundle;              // T: samples per bundle, 1 .. 16 (a power of two for the shared-memory kernel)
    double eps;
    double inv_m;            // 1 / m (the fp64 pipe is slow: no division on the device)
    double *partials;        // [batch][G][4]: A, B, mean and element count of the CTA's share
    unsigned int *arrived;   // [bundles], zero at launch
    int *status;
};

constexpr int kLnThreads = 512;
constexpr int kLnWarps = kLnThreads / 32;
constexpr int kLnMaxBundle = 16;                         // = warps per CTA: one warp combines one sample

// 32-byte loads (sm_100 has 256-bit global accesses; half as many instructions
// per byte in flight) with an L2 eviction priority: plain for the first read of
// x, "evict last" for gamma and beta, which are read again for every sample, and
// "evict first" for the second and last read of x.
struct Float8 {
    float v[8];
};
__device__ __forceinline__ Float8 ld8(const float *p)
{
    Float8 r;
    asm volatile("ld.global.L1::no_allocate.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]),
                   "=f"(r.v[6]), "=f"(r.v[7]) : "l"(p) : "memory");
    return r;
}
__device__ __forceinline__ Float8 ld8_last_use(const float *p)
{
    Float8 r;
    asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]),
                   "=f"(r.v[6]), "=f"(r.v[7]) : "l"(p) : "memory");
    return r;
}
__device__ __forceinline__ Float8 ld8_keep(const float *p)
{
    Float8 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::evict_last.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]),
                   "=f"(r.v[6]), "=f"(r.v[7]) : "l"(p));
    return r;
}
__device__ __forceinline__ void st8_stream(float *p, const Float8 &r)
{
    asm volatile("st.global.L1::no_allocate.L2::evict_first.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "f"(r.v[0]), "f"(r.v[1]), "f"(r.v[2]), "f"(r.v[3]), "f"(r.v[4]), "f"(r.v[5]),
                   "f"(r.v[6]), "f"(r.v[7]) : "memory");
}

// One element of pass 2 in float32.  The mean arrives as mh + ml (mh = the
// double mean rounded to float, ml = the rest): x - mh is exact when x is near
// the mean and has a relative error of 2^-24 otherwise, so (x - mh) - ml is the
// deviation to ~2^-23 of ITS OWN size -- no cancellation against a large mean.
__device__ __forceinline__ float ln_apply(float x, float mh, float ml, float rstd, float g, float b)
{
    return fmaf(((x - mh) - ml) * rstd, g, b);
}

// Moments of one 32-byte piece about the pilot c, in float32 (a tree of depth
// three for the sum), added to the caller's float32 partial sums.  The caller
// widens those to double after at most four pieces, so every float32 sum is a
// tree of depth <= 6 and its error stays below 2^-21 of the sum of magnitudes,
// while the slow fp64 pipe sees one conversion and one add per 16 elements.
__device__ __forceinline__ void ln_add_piece(const Float8 &v, float c, float &f1, float &f2)
{
    const float d0 = v.v[0] - c, d1 = v.v[1] - c, d2 = v.v[2] - c, d3 = v.v[3] - c;
    const float d4 = v.v[4] - c, d5 = v.v[5] - c, d6 = v.v[6] - c, d7 = v.v[7] - c;
    f1 += ((d0 + d1) + (d2 + d3)) + ((d4 + d5) + (d6 + d7));
    float qa = d0 * d0, qb = d4 * d4;
    qa = fmaf(d1, d1, qa); qb = fmaf(d5, d5, qb);
    qa = fmaf(d2, d2, qa); qb = fmaf(d6, d6, qb);
    qa = fmaf(d3, d3, qa); qb = fmaf(d7, d7, qb);
    f2 += qa + qb;
}
__device__ __forceinline__ void ln_add_quad(const float4 &v, float c, float &f1, float &f2)
{
    const float d0 = v.x - c, d1 = v.y - c, d2 = v.z - c, d3 = v.w - c;
    f1 += (d0 + d1) + (d2 + d3);
    float q = d0 * d0;
    q = fmaf(d1, d1, q);
    q = fmaf(d2, d2, q);
    q = fmaf(d3, d3, q);
    f2 += q;
}
__device__ __forceinline__ void ln_flush(float &f1, float &f2, double &s1, double &s2)
{
    s1 += static_cast<double>(f1);
    s2 += static_cast<double>(f2);
    f1 = 0.f;
    f2 = 0.f;
}
__device__ __forceinline__ float ln_pilot(const Float8 &v)
{
    return (((v.v[0] + v.v[1]) + (v.v[2] + v.v[3])) + ((v.v[4] + v.v[5]) + (v.v[6] + v.v[7]))) * 0.125f;
}

// What a CTA publishes for its n elements of a sample: A = sum x, B = sum of
// squared deviations about its own mean, and that mean.
__device__ __forceinline__ void ln_publish(double *slot, double n, float c, double s1, double s2)
{
    const double A = n * static_cast<double>(c) + s1;
    const double mean = n > 0.0 ? A / n : 0.0;
    double B = n > 0.0 ? s2 - s1 * s1 / n : 0.0;
    B = B > 0.0 ? B : 0.0;
    __stcg(slot, A);
    __stcg(slot + 1, B);
    __stcg(slot + 2, mean);
    __stcg(slot + 3, n);
}

__device__ __forceinline__ float warp_sum_f32(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One warp combines the G published entries of a sample: mean, and M2 as the sum
// of the entries' own B plus n_k (mean_k - mean)^2.  Only the sum of the A_k and
// the differences of means need double.  Lane 0 writes (mean high, mean low,
// 1 / sqrt(var + eps)) to out.
__device__ __forceinline__ void ln_combine(const double *slots, int G, double inv_m, double eps, int lane,
                                           float *out)
{
    double a = 0.0;
    for (int k = lane; k < G; k += 32) a += __ldcg(slots + 4 * k);
    a = warp_sum(a);
    const double mean = a * inv_m;
    float m2 = 0.f;
    for (int k = lane; k < G; k += 32) {
        const float dm = static_cast<float>(__ldcg(slots + 4 * k + 2) - mean);
        m2 += static_cast<float>(__ldcg(slots + 4 * k + 1)) + static_cast<float>(__ldcg(slots + 4 * k + 3)) * dm * dm;
    }
    m2 = warp_sum_f32(m2);
    if (lane == 0) {
        const double var = static_cast<double>(m2) * inv_m;
        const float mh = static_cast<float>(mean);
        out[0] = mh;
        out[1] = static_cast<float>(mean - static_cast<double>(mh));
        out[2] = static_cast<float>(rsqrt(var + eps));
    }
}

// Thread 0: announce this CTA's moments of a bundle and wait for the group.
// Returns false (and raises the status) if the wait ran out.
__device__ __forceinline__ bool ln_meet(unsigned int *counter, int group_size, int *status)
{
    atomicAdd(counter, 1u);
    const uint64_t t0 = globaltimer_ns();
    unsigned int seen;
    do {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
        if (seen >= static_cast<unsigned int>(group_size)) return true;
    } while (globaltimer_ns() - t0 <= kWaitLimitNs);
    task_report_timeout(status, kRoleLayerNorm, 0);
    return false;
}

// ---------------------------------------------------------------------------
// Which elements a CTA works on (aligned data).  A sample is cut into blocks of
// 128 pieces of 32 bytes (4 KiB); CTA g of a group takes blocks g, g + G, g + 2G,
// ... .  Measured on this GPU: 148 CTAs that each stream their own contiguous
// 100 KB slice reach 4.5 TB/s, the same loads interleaved block-wise reach
// 6.4 TB/s -- the CTAs then sweep one compact window of DRAM together.
constexpr int kLnBlockPieces = 128;
constexpr int kLnBlockBytes = kLnBlockPieces * 32;
constexpr int kLnBlocksPerRound = kLnThreads / kLnBlockPieces;       // 4 blocks per sweep of the CTA

struct LnSpan {
    long long pieces;        // 32-byte pieces per sample
    int g, G;
    int nblocks;             // blocks of this CTA
    // global piece index of this thread in the CTA's block j (may be >= pieces in the last block)
    __device__ __forceinline__ long long piece(int j, int tid) const
    {
        return (static_cast<long long>(j) * G + g) * kLnBlockPieces + (tid & (kLnBlockPieces - 1));
    }
};
__device__ __forceinline__ LnSpan ln_span(long long m, int g, int G)
{
    LnSpan sp;
    sp.pieces = m >> 3;
    sp.g = g;
    sp.G = G;
    const long long blocks = (sp.pieces + kLnBlockPieces - 1) / kLnBlockPieces;
    sp.nblocks = blocks > g ? static_cast<int>((blocks - 1 - g) / G) + 1 : 0;
    return sp;
}
// elements of the sample that the CTA owns
__device__ __forceinline__ double ln_span_elems(const LnSpan &sp)
{
    long long n = 0;
    for (int j = 0; j < sp.nblocks; ++j) {
        const long long first = (static_cast<long long>(j) * sp.G + sp.g) * kLnBlockPieces;
        n += min(static_cast<long long>(kLnBlockPieces), sp.pieces - first);
    }
    return static_cast<double>(8 * n);
}

// ---------------------------------------------------------------------------
// Blocks in shared memory.  Per bundle:
//   1. warp 0 asks the copy engine for the CTA's blocks of the T samples (bulk
//      copies completing on one mbarrier per chunk position of 16 KiB);
//   2. when they have landed, warp w takes the moments of its share of sample
//      w / (16 / T) out of shared memory; thread t publishes sample t; the group
//      meets;
//   3. warp t combines the group's entries of sample t;
//   4. pass 2 walks the chunk positions: gamma and beta are loaded once per
//      32-byte piece and applied to all T samples (their L2 traffic drops by T),
//      x comes from shared memory, y goes to HBM; as soon as a chunk position has
//      been consumed, the copies of the next bundle for that position are issued,
//      so that HBM reads run under pass 2's writes.
constexpr int kLnChunkBlocks = 4;                        // blocks per chunk position = one sweep of the CTA
constexpr int kLnChunkBytes = kLnChunkBlocks * kLnBlockBytes;
constexpr int kLnMaxChunks = 8;

__device__ __forceinline__ void bulk_load_1d(uint32_t smem_addr, const void *gptr, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr), "l"(gptr), "r"(bytes), "r"(bar) : "memory");
}

__global__ void __launch_bounds__(kLnThreads)
layernorm_smem_kernel(const LayerNormParams p)
{
    static_assert(kLnWarps == kLnMaxBundle, "one warp per sample of a bundle");
    static_assert(kLnChunkBlocks == kLnBlocksPerRound, "a chunk position is one sweep of the CTA");
    extern __shared__ __align__(128) uint8_t ln_smem[];
    __shared__ double wsum[kLnWarps][2];
    __shared__ float stat[kLnMaxBundle][3];              // mean (two floats) and 1/sqrt(var + eps) per sample
    __shared__ __align__(8) unsigned long long bars[kLnMaxChunks];
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int group = blockIdx.x / p.group_size;
    const int g = blockIdx.x - group * p.group_size;
    const int T = p.bundle;
    const LnSpan sp = ln_span(p.m, g, p.group_size);
    const int nchunks = (sp.nblocks + kLnChunkBlocks - 1) / kLnChunkBlocks;
    const uint32_t buf_bytes = static_cast<uint32_t>(p.slice * 4);   // shared memory per sample (whole blocks)
    const uint32_t smem0 = smem_u32(ln_smem);
    const int num_bundles = (p.batch + T - 1) / T;
    const double n_own = ln_span_elems(sp);
    if (tid == 0) {
        abort_flag = 0;
        for (int c = 0; c < kLnMaxChunks; ++c) mbar_init(smem_u32(&bars[c]), 1);
        fence_mbar_init();
        fence_proxy_async_smem();
    }
    __syncthreads();

    // bytes of the CTA's block j that exist (the sample's last block may be short)
    auto block_bytes = [&](int j) -> uint32_t {
        const long long first = (static_cast<long long>(j) * sp.G + sp.g) * kLnBlockPieces;
        return static_cast<uint32_t>(min(static_cast<long long>(kLnBlockPieces), sp.pieces - first)) * 32u;
    };
    // copies of chunk position c of every sample of a bundle (warp 0; one copy per lane and turn)
    auto issue_chunk = [&](int bundle, int c) {
        const int tb = min(T, p.batch - bundle * T);
        const int j0 = c * kLnChunkBlocks, j1 = min(j0 + kLnChunkBlocks, sp.nblocks);
        const uint32_t bar = smem_u32(&bars[c]);
        if (lane == 0) {
            uint32_t bytes = 0;
            for (int j = j0; j < j1; ++j) bytes += block_bytes(j);
            mbar_expect_tx(bar, bytes * tb);
        }
        __syncwarp();
        const int copies = tb * (j1 - j0);
        for (int q = lane; q < copies; q += 32) {
            const int t = q / (j1 - j0), j = j0 + (q - t * (j1 - j0));
            const float *src = p.x + static_cast<long long>(bundle * T + t) * p.m
                             + (static_cast<long long>(j) * sp.G + sp.g) * (kLnBlockPieces * 8);
            bulk_load_1d(smem0 + t * buf_bytes + j * kLnBlockBytes, src, block_bytes(j), bar);
        }
    };

    int bundle = group;
    if (bundle >= num_bundles) return;
    if (warp == 0)
        for (int c = 0; c < nchunks; ++c) issue_chunk(bundle, c);
    uint32_t phase = 0;
    const int W = kLnWarps / T;                          // warps per sample in step 2
    for (; bundle < num_bundles; bundle += p.num_groups) {
        const int tb = min(T, p.batch - bundle * T);     // samples in this bundle
        const int s0 = bundle * T;
        // 1. the blocks have landed
        bool ok = true;
        for (int c = 0; c < nchunks; ++c) ok = mbar_wait(smem_u32(&bars[c]), phase, &abort_flag) && ok;
        phase ^= 1;
        if (!__syncthreads_and(ok)) {
            if (tid == 0) task_report_timeout(p.status, kRoleLayerNorm, 1);
            return;
        }
        // 2. moments per sample about the pilot (the mean of the CTA's first piece of the sample)
        {
            const int t = warp / W, part = warp - t * W;
            double s1 = 0.0, s2 = 0.0;
            if (t < tb && sp.nblocks > 0) {
                const uint32_t base = smem0 + t * buf_bytes;
                Float8 v;
                {
                    const float4 a = ld_shared_v4(base), q = ld_shared_v4(base + 16);
                    v.v[0] = a.x; v.v[1] = a.y; v.v[2] = a.z; v.v[3] = a.w;
                    v.v[4] = q.x; v.v[5] = q.y; v.v[6] = q.z; v.v[7] = q.w;
                }
                const float c = ln_pilot(v);
                // consecutive lanes read consecutive 16 bytes of a block (conflict-free); the warps
                // of the sample take the block's 16-byte quads 32 at a time
                float f1 = 0.f, f2 = 0.f;
                int pending = 0;
                for (int j = 0; j < sp.nblocks; ++j) {
                    const uint32_t nq = block_bytes(j) >> 4;
                    for (uint32_t k = part * 32 + lane; k < nq; k += W * 32) {
                        ln_add_quad(ld_shared_v4(base + j * kLnBlockBytes + k * 16), c, f1, f2);
                        if (++pending == 8) { ln_flush(f1, f2, s1, s2); pending = 0; }
                    }
                }
                ln_flush(f1, f2, s1, s2);
                if (part == 0 && lane == 0) stat[t][0] = c;          // parked for the publishing thread
            }
            s1 = warp_sum(s1);
            s2 = warp_sum(s2);
            if (lane == 0) { wsum[warp][0] = s1; wsum[warp][1] = s2; }
        }
        __syncthreads();
        if (tid < tb) {
            double t1 = 0.0, t2 = 0.0;
            for (int k = 0; k < W; ++k) { t1 += wsum[tid * W + k][0]; t2 += wsum[tid * W + k][1]; }
            ln_publish(p.partials + (static_cast<long long>(s0 + tid) * p.group_size + g) * 4, n_own,
                       sp.nblocks > 0 ? stat[tid][0] : 0.f, t1, t2);
            __threadfence();
        }
        __syncthreads();
        if (tid == 0 && !ln_meet(p.arrived + bundle, p.group_size, p.status)) abort_flag = 1;
        __syncthreads();
        if (abort_flag) return;
        // 3. warp t combines the group's entries of sample t
        if (warp < tb)
            ln_combine(p.partials + static_cast<long long>(s0 + warp) * p.group_size * 4, p.group_size, p.inv_m,
                       p.eps, lane, stat[warp]);
        __syncthreads();
        // 4. pass 2, chunk position by chunk position: thread -> block 4 c + tid / 128, piece tid % 128
        const int next = bundle + p.num_groups;
        for (int c = 0; c < nchunks; ++c) {
            const int j = c * kLnChunkBlocks + (tid >> 7);
            const long long i = sp.piece(j, tid);
            if (j < sp.nblocks && i < sp.pieces) {
                const long long e = 8 * i;
                Float8 gm, bt;
                if (p.gamma) gm = ld8_keep(p.gamma + e);
                if (p.beta) bt = ld8_keep(p.beta + e);
                const uint32_t at = j * kLnBlockBytes + (tid & (kLnBlockPieces - 1)) * 32;
                for (int t = 0; t < tb; ++t) {
                    const float mh = stat[t][0], ml = stat[t][1], rstd = stat[t][2];
                    const float4 a = ld_shared_v4(smem0 + t * buf_bytes + at);
                    const float4 q = ld_shared_v4(smem0 + t * buf_bytes + at + 16);
                    Float8 v;
                    v.v[0] = a.x; v.v[1] = a.y; v.v[2] = a.z; v.v[3] = a.w;
                    v.v[4] = q.x; v.v[5] = q.y; v.v[6] = q.z; v.v[7] = q.w;
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        v.v[u] = ln_apply(v.v[u], mh, ml, rstd, p.gamma ? gm.v[u] : 1.f, p.beta ? bt.v[u] : 0.f);
                    st8_stream(p.y + static_cast<long long>(s0 + t) * p.m + e, v);
                }
            }
            __syncthreads();                             // chunk position c of every buffer has been read
            if (next < num_bundles && warp == 0) issue_chunk(next, c);
        }
    }
}

// ---------------------------------------------------------------------------
// Blocks streamed from global memory in both passes.  VEC: 32-byte accesses on
// the block-interleaved mapping (bases 32-byte aligned, m a multiple of 8);
// otherwise element by element on contiguous slices of p.slice elements.
template <bool VEC>
__global__ void __launch_bounds__(kLnThreads)
layernorm_stream_kernel(const LayerNormParams p)
{
    __shared__ double wsum[kLnMaxBundle][kLnWarps][2];
    __shared__ float stat[kLnMaxBundle][3];
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int group = blockIdx.x / p.group_size;
    const int g = blockIdx.x - group * p.group_size;
    const int T = p.bundle;
    const LnSpan sp = ln_span(p.m, g, p.group_size);
    const long long lo = static_cast<long long>(g) * p.slice;        // scalar path
    const long long hi = min(p.m, lo + p.slice);
    const double n_own = VEC ? ln_span_elems(sp) : static_cast<double>(hi > lo ? hi - lo : 0);
    const int num_bundles = (p.batch + T - 1) / T;
    const int sub = tid >> 7;                                        // block of a sweep this thread is in
    if (tid == 0) abort_flag = 0;
    __syncthreads();

    for (int bundle = group; bundle < num_bundles; bundle += p.num_groups) {
        const int s0 = bundle * T;
        const int tb = min(T, p.batch - s0);
        // ---- pass 1 over the bundle's samples
        if (VEC) {
            // Rounds of four pieces per thread (sixteen blocks per CTA), numbered through all
            // samples of the bundle; the loads of round r + 1 (which may belong to the next
            // sample) are in flight while round r is added up, so the stream never drains.
            const int rps = max(1, (sp.nblocks + 4 * kLnBlocksPerRound - 1) / (4 * kLnBlocksPerRound));
            const int rounds = rps * tb;
            Float8 cur[4], nxt[4], pil_cur, pil_nxt;
            auto fetch = [&](int r, Float8 (&buf)[4], Float8 &pil) {
                const int t = r / rps, jr = r - t * rps;
                const float *xs = p.x + static_cast<long long>(s0 + t) * p.m;
                if (jr == 0 && sp.nblocks > 0) pil = ld8(xs + 8 * sp.piece(0, 0));   // one request per warp
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int j = (4 * jr + u) * kLnBlocksPerRound + sub;
                    const long long i = sp.piece(j, tid);
                    if (j < sp.nblocks && i < sp.pieces) buf[u] = ld8(xs + 8 * i);
                }
            };
            double s1 = 0.0, s2 = 0.0;
            float c = 0.f;
            auto consume = [&](int r, const Float8 (&buf)[4], const Float8 &pil) {
                const int t = r / rps, jr = r - t * rps;
                if (jr == 0 && sp.nblocks > 0) c = ln_pilot(pil);
                float f1 = 0.f, f2 = 0.f;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int j = (4 * jr + u) * kLnBlocksPerRound + sub;
                    const long long i = sp.piece(j, tid);
                    if (j < sp.nblocks && i < sp.pieces) ln_add_piece(buf[u], c, f1, f2);
                }
                ln_flush(f1, f2, s1, s2);
                if (jr == rps - 1) {                     // the sample is complete
                    s1 = warp_sum(s1);
                    s2 = warp_sum(s2);
                    if (lane == 0) { wsum[t][warp][0] = s1; wsum[t][warp][1] = s2; }
                    if (tid == 0) stat[t][0] = sp.nblocks > 0 ? c : 0.f;
                    s1 = 0.0;
                    s2 = 0.0;
                }
            };
            if (rounds > 0) fetch(0, cur, pil_cur);
            for (int r = 0; r < rounds; r += 2) {
                if (r + 1 < rounds) fetch(r + 1, nxt, pil_nxt);
                consume(r, cur, pil_cur);
                if (r + 1 < rounds) {
                    if (r + 2 < rounds) fetch(r + 2, cur, pil_cur);
                    consume(r + 1, nxt, pil_nxt);
                }
            }
        } else {
            for (int t = 0; t < tb; ++t) {
                const float *xb = p.x + static_cast<long long>(s0 + t) * p.m + lo;
                double s1 = 0.0, s2 = 0.0;
                const float c = hi > lo ? __ldcg(xb) : 0.f;
                for (long long i = lo + tid; i < hi; i += kLnThreads) {
                    const double d = static_cast<double>(__ldcg(xb + (i - lo)) - c);
                    s1 += d;
                    s2 = fma(d, d, s2);
                }
                s1 = warp_sum(s1);
                s2 = warp_sum(s2);
                if (lane == 0) { wsum[t][warp][0] = s1; wsum[t][warp][1] = s2; }
                if (tid == 0) stat[t][0] = c;
            }
        }
        __syncthreads();
        if (tid < tb) {
            double t1 = 0.0, t2 = 0.0;
            for (int k = 0; k < kLnWarps; ++k) { t1 += wsum[tid][k][0]; t2 += wsum[tid][k][1]; }
            ln_publish(p.partials + (static_cast<long long>(s0 + tid) * p.group_size + g) * 4, n_own,
                       stat[tid][0], t1, t2);
            __threadfence();
        }
        __syncthreads();
        // ---- the group meets (a group of one has nobody to wait for, but its own
        //      entries still travel through global memory: same code path)
        if (tid == 0 && !ln_meet(p.arrived + bundle, p.group_size, p.status)) abort_flag = 1;
        __syncthreads();
        if (abort_flag) return;
        if (warp < tb)
            ln_combine(p.partials + static_cast<long long>(s0 + warp) * p.group_size * 4, p.group_size, p.inv_m,
                       p.eps, lane, stat[warp]);
        __syncthreads();
        // ---- pass 2, the sample read last first, two samples per sweep
        for (int t = tb - 1; t >= 0; t -= 2) {
            const bool pair = t >= 1;                    // samples t and t - 1 share gamma and beta
            const int ta = t, tc = pair ? t - 1 : t;
            const float *xa = p.x + static_cast<long long>(s0 + ta) * p.m;
            const float *xc = p.x + static_cast<long long>(s0 + tc) * p.m;
            float *ya = p.y + static_cast<long long>(s0 + ta) * p.m;
            float *yc = p.y + static_cast<long long>(s0 + tc) * p.m;
            const float mha = stat[ta][0], mla = stat[ta][1], ra = stat[ta][2];
            const float mhc = stat[tc][0], mlc = stat[tc][1], rc = stat[tc][2];
            if (VEC) {
                for (int j = sub; j < sp.nblocks; j += kLnBlocksPerRound) {
                    const long long i = sp.piece(j, tid);
                    if (i >= sp.pieces) continue;
                    const long long e = 8 * i;
                    Float8 va = ld8_last_use(xa + e), vc, gm, bt;
                    if (pair) vc = ld8_last_use(xc + e);
                    if (p.gamma) gm = ld8_keep(p.gamma + e);
                    if (p.beta) bt = ld8_keep(p.beta + e);
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        va.v[u] = ln_apply(va.v[u], mha, mla, ra, p.gamma ? gm.v[u] : 1.f, p.beta ? bt.v[u] : 0.f);
                    st8_stream(ya + e, va);
                    if (pair) {
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            vc.v[u] = ln_apply(vc.v[u], mhc, mlc, rc, p.gamma ? gm.v[u] : 1.f, p.beta ? bt.v[u] : 0.f);
                        st8_stream(yc + e, vc);
                    }
                }
            } else {
                for (long long i = lo + tid; i < hi; i += kLnThreads) {
                    const float gm = p.gamma ? p.gamma[i] : 1.f;
                    const float bt = p.beta ? p.beta[i] : 0.f;
                    const float a = __ldcg(xa + i);
                    const float cv = pair ? __ldcg(xc + i) : 0.f;    // read before the stores: y may be x
                    ya[i] = ln_apply(a, mha, mla, ra, gm, bt);
                    if (pair) yc[i] = ln_apply(cv, mhc, mlc, rc, gm, bt);
                }
            }
        }
        __syncthreads();                                 // stat[] and wsum[] are rewritten for the next bundle
    }
}

}  // namespace cudallm
