// Bandwidth-bound kernels for the paper's benchmark tasks on float32 arrays:
// Task 8 (matrix transpose), Task 14 (reduction: sum), Task 15 (dot product)
// and Task 4 (LayerNorm).  None of them is a contraction; what matters is that
// every byte crosses HBM once, in full cache lines, with enough of them in
// flight.
#pragma once
#include "ptx.cuh"

namespace cudallm {

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
    grid_launch_dependents();
    grid_dependency_wait();
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
    grid_launch_dependents();
    grid_dependency_wait();
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
    grid_launch_dependents();
    grid_dependency_wait();
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
// General path: two plain kernels of many small CTAs (no CTA waits for another;
// the one-pass kernel for samples that fit in shared memory follows further down):
//  * layernorm_moments_kernel: CTA (s, part) takes the moments of one part of
//    sample s and publishes them;
//  * layernorm_apply_kernel: CTA (pair of samples, chunk) combines the published
//    moments of its two samples -- the same arithmetic in the same order in
//    every CTA -- and normalises its chunk of both, fetching gamma and beta once
//    for the pair.
// x is read twice; for batches that fit in L2 the second read stays on chip.
//
// Arithmetic.  The moments are taken in float32 about a pilot value c (the mean
// of the first eight elements of the CTA's part, so that x - c is of the size of
// the data's spread, not of its offset): per 32-byte piece, d_j = x_j - c,
// f1 = sum d_j, f2 = sum d_j^2 in float32, widened to double every four pieces.
// A CTA publishes A = n c + S1 (its sum of x), its own mean A / n and
// B = S2 - S1^2 / n (its sum of squared deviations about that mean); the
// combination is mean = sum A_k / m and M2 = sum (B_k + n_k (mean_k - mean)^2):
// no large numbers are subtracted anywhere, so a mean far larger than the
// spread costs no accuracy.  Pass 2 is float32 on a two-float mean (ln_apply).
//
// History, measured on (16, 4, 1024, 1024) and (16, 4, 512, 512): persistent
// kernels in which groups of CTAs shared a sample, kept its slices in shared
// memory (bulk async copies) or streamed them twice, and met at counters in
// global memory took 148-192 us and 45 us; every meeting left the memory system
// idle for 5-12 us (the slowest CTA of 148 finishes its stream that much later
// than the first).  The two plain kernels take 144 us and 39 us.

// 32-byte loads (sm_100 has 256-bit global accesses; half as many instructions
// per byte in flight) with an L2 eviction priority: plain for the first read of
// x, "evict last" for gamma and beta, which are read again for every sample, and
// "evict first" for the second and last read of x.  The first read must NOT
// carry L1::no_allocate: measured with ncu, lines fetched that way are not kept
// in L2 either (the second kernel then re-read all of a 17 MB x from DRAM; with
// the plain load it reads 3 KB).
struct Float8 {
    float v[8];
};
__device__ __forceinline__ Float8 ld8(const float *p)
{
    Float8 r;
    asm volatile("ld.global.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
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

// ---------------------------------------------------------------------------
// Pairs are visited last sample first in the second kernel, so that what the
// first kernel read last is read again first.
struct LayerNorm2Params {
    const float *x, *gamma, *beta;
    float *y;
    long long m;             // elements per sample
    long long part_len;      // elements per part of the first kernel (a multiple of 8)
    long long chunk_len;     // elements per CTA of the second kernel (a multiple of 8)
    int batch, parts, chunks;
    double eps, inv_m;
    double *partials;        // [batch][parts][4]
};
constexpr int kLn2Threads = 256;

template <bool VEC>
__global__ void __launch_bounds__(kLn2Threads)
layernorm_moments_kernel(const LayerNorm2Params p)
{
    __shared__ double warp_part[kLn2Threads / 32];
    grid_launch_dependents();
    grid_dependency_wait();
    const int s = blockIdx.x / p.parts, part = blockIdx.x - s * p.parts;
    const int tid = threadIdx.x;
    const long long lo = static_cast<long long>(part) * p.part_len;
    const long long hi = min(p.m, lo + p.part_len);
    const float *xb = p.x + static_cast<long long>(s) * p.m + lo;
    double s1 = 0.0, s2 = 0.0;
    float c = 0.f;
    if (VEC) {
        const long long nv = hi > lo ? (hi - lo) >> 3 : 0;
        if (nv > 0) c = ln_pilot(ld8(xb));               // the same 32 bytes for every thread
        for (long long i = tid; i < nv; i += 4 * kLn2Threads) {
            Float8 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (i + u * kLn2Threads < nv) v[u] = ld8(xb + 8 * (i + u * kLn2Threads));
            float f1 = 0.f, f2 = 0.f;
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (i + u * kLn2Threads < nv) ln_add_piece(v[u], c, f1, f2);
            ln_flush(f1, f2, s1, s2);
        }
    } else {
        if (hi > lo) c = __ldcg(xb);
        for (long long i = tid; i < hi - lo; i += kLn2Threads) {
            const double d = static_cast<double>(__ldcg(xb + i) - c);
            s1 += d;
            s2 = fma(d, d, s2);
        }
    }
    const double t1 = block_sum(s1, warp_part);
    const double t2 = block_sum(s2, warp_part);
    if (tid == 0)
        ln_publish(p.partials + (static_cast<long long>(s) * p.parts + part) * 4,
                   static_cast<double>(hi > lo ? hi - lo : 0), c, t1, t2);
}

template <bool VEC>
__global__ void __launch_bounds__(kLn2Threads)
layernorm_apply_kernel(const LayerNorm2Params p)
{
    __shared__ float stat[2][3];
    grid_launch_dependents();
    grid_dependency_wait();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int npairs = (p.batch + 1) / 2;
    const int pair = npairs - 1 - static_cast<int>(blockIdx.x / p.chunks);       // last samples first
    const int chunk = static_cast<int>(blockIdx.x - static_cast<unsigned>(npairs - 1 - pair) * p.chunks);
    const int sa = 2 * pair, sc = min(2 * pair + 1, p.batch - 1);
    const bool two = sc != sa;
    if (warp < 2)
        ln_combine(p.partials + static_cast<long long>(warp ? sc : sa) * p.parts * 4, p.parts, p.inv_m, p.eps,
                   lane, stat[warp]);
    __syncthreads();
    const float mha = stat[0][0], mla = stat[0][1], ra = stat[0][2];
    const float mhc = stat[1][0], mlc = stat[1][1], rc = stat[1][2];
    const long long lo = static_cast<long long>(chunk) * p.chunk_len;
    const long long hi = min(p.m, lo + p.chunk_len);
    const float *xa = p.x + static_cast<long long>(sa) * p.m, *xc = p.x + static_cast<long long>(sc) * p.m;
    float *ya = p.y + static_cast<long long>(sa) * p.m, *yc = p.y + static_cast<long long>(sc) * p.m;
    if (VEC) {
        const long long nv = hi > lo ? (hi - lo) >> 3 : 0;
        for (long long i = tid; i < nv; i += kLn2Threads) {
            const long long e = lo + 8 * i;
            Float8 va = ld8_last_use(xa + e), vc, gm, bt;
            if (two) vc = ld8_last_use(xc + e);
            if (p.gamma) gm = ld8_keep(p.gamma + e);
            if (p.beta) bt = ld8_keep(p.beta + e);
#pragma unroll
            for (int u = 0; u < 8; ++u)
                va.v[u] = ln_apply(va.v[u], mha, mla, ra, p.gamma ? gm.v[u] : 1.f, p.beta ? bt.v[u] : 0.f);
            st8_stream(ya + e, va);
            if (two) {
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    vc.v[u] = ln_apply(vc.v[u], mhc, mlc, rc, p.gamma ? gm.v[u] : 1.f, p.beta ? bt.v[u] : 0.f);
                st8_stream(yc + e, vc);
            }
        }
    } else {
        for (long long i = lo + tid; i < hi; i += kLn2Threads) {
            const float gm = p.gamma ? p.gamma[i] : 1.f;
            const float bt = p.beta ? p.beta[i] : 0.f;
            const float a = __ldcg(xa + i);
            const float cv = two ? __ldcg(xc + i) : 0.f;             // read before the stores: y may be x
            ya[i] = ln_apply(a, mha, mla, ra, gm, bt);
            if (two) yc[i] = ln_apply(cv, mhc, mlc, rc, gm, bt);
        }
    }
}

// ---------------------------------------------------------------------------
// LayerNorm as ONE persistent kernel that reads x from DRAM once: the second
// read of a sample comes out of L2, a few samples after the first.  G CTAs (one
// per SM); CTA i owns positions [i * slice_len, (i + 1) * slice_len) of EVERY
// sample (so each line of x, gamma and beta is only ever asked for by one SM),
// cut into 16 KB chunks.  All loads are bulk asynchronous copies into shared
// memory: what is in flight is bounded by shared memory (5 chunks from DRAM, 6 to
// 8 from L2), not by registers.  Roles:
//
//   loader A (one lane): chunk after chunk of x, sample after sample, from DRAM
//     into ring A ("evict last": wanted again soon); never more than `lead` chunks ahead of the normalisation,
//     so that what it fetched is still in L2 when it is read again;
//   8 moments warps: take the chunks from ring A, hand each sample's moments to
//     the exchange warp;
//   4 exchange warps (warp w serves samples w, w + 4, ...): publish this CTA's
//     moments of a sample, wait for the G entries of the sample, combine them
//     (the same arithmetic in the same order in every CTA), hand mean and
//     1 / sqrt(var + eps) on; one round trip to L2 takes microseconds while
//     the SM streams, so several samples' exchanges must be in flight;
//   loader B (one lane): for every chunk of a sample whose moments are done,
//     x again (now from L2, "evict first": its last use) and the chunk's gamma
//     and beta (from L2, "evict last") into ring B (3 stages of 48 KB; 4 or 9
//     stages when gamma and / or beta are absent);
//   8 normalising warps: take the stages from ring B, store y (streaming).
//
// DRAM reads and writes therefore run side by side all the time, a CTA meets
// the others' moments a sample or more after it published its own, and no
// kernel boundary drains the memory system.  In place (y == x) is safe: an
// element of y is stored after both copies of that element of x have landed.
//
// All G CTAs must be resident at the same time (G <= number of SMs, one CTA per
// SM by shared memory); every wait is bounded, gives up with a status word
// (role 5: 0x10 + kind of wait) and lets the kernel drain and return.
constexpr int kLnRoleWarps = 8;
constexpr int kLnRoleThreads = kLnRoleWarps * 32;
constexpr int kLnExchangeWarps = 4;                               // exchange warp w serves samples w, w + 4, ...
constexpr int kLnStreamThreads = 2 * kLnRoleThreads + (2 + kLnExchangeWarps) * 32;     // + loader A, loader B, exchange
constexpr int kLnChunkElems = 4096;
constexpr int kLnChunkBytes = kLnChunkElems * 4;                  // 16 KB
constexpr int kLnRingA = 5;                                       // chunks of x on their way from DRAM
constexpr int kLnRingBChunks = 9;                                 // chunks of shared memory for ring B: 9 stages of x alone,
                                                                  // 4 of (x, gamma) or (x, beta), 3 of (x, gamma, beta)
constexpr int kLnStreamSmem = (kLnRingA + kLnRingBChunks) * kLnChunkBytes;    // 224 KB
constexpr int kLnSlots = 16;                             // samples in flight between the roles (see `lead`)
constexpr int kRoleLayerNorm = 5;

struct LayerNormStreamParams {
    const float *x, *gamma, *beta;
    float *y;
    long long m;             // elements per sample
    long long slice_len;     // elements per CTA (a multiple of 8)
    int batch, ctas;
    int lead;                // chunks loader A may run ahead of loader B (at most kLnSlots - 8 samples' worth)
    double eps, inv_m;
    unsigned long long *entries;   // [batch][ctas][6]: the published moments, every word tagged (see LnEntry)
    int epoch;               // the tag of this launch's entries (never 0)
    int tag_post;            // the tag this launch writes: epoch (anything else only in the host's
                             // self-test of the wait limit)
    int *status;
    unsigned long long wait_limit_ns;
};

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// `bytes` (a multiple of 16) from global to this CTA's shared memory; completion is counted on `bar`.
__device__ __forceinline__ void bulk_load_hint(uint32_t smem_dst, const void *src, uint32_t bytes, uint32_t bar,
                                               uint64_t policy)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
                 "[%0], [%1], %2, [%3], %4;"
                 ::"r"(smem_dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
// 16-byte accesses for the persistent LayerNorm kernel: consecutive lanes touch consecutive
// 16 bytes of shared memory (a 32-byte piece per lane costs every access two passes through
// the banks, and with the copies' own writes that made shared memory the kernel's bound).
__device__ __forceinline__ float4 lds4(uint32_t addr)
{
    float4 r;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "r"(addr) : "memory");
    return r;
}
__device__ __forceinline__ void st4_stream(float *p, const float4 &r, uint64_t policy)
{
    asm volatile("st.global.L1::no_allocate.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;"
                 ::"l"(p), "f"(r.x), "f"(r.y), "f"(r.z), "f"(r.w), "l"(policy) : "memory");
}
__device__ __forceinline__ void ln_add_piece4(const float4 &v, float c, float &f1, float &f2)
{
    const float d0 = v.x - c, d1 = v.y - c, d2 = v.z - c, d3 = v.w - c;
    f1 += (d0 + d1) + (d2 + d3);
    float q = d0 * d0;
    q = fmaf(d1, d1, q);
    q = fmaf(d2, d2, q);
    q = fmaf(d3, d3, q);
    f2 += q;
}
__device__ __forceinline__ Float8 lds8(uint32_t addr)
{
    Float8 r;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]) : "r"(addr) : "memory");
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7]) : "r"(addr + 16) : "memory");
    return r;
}
constexpr int kLnMaxCtas = 160;                          // entries per sample: at most five per lane of a warp

// What a CTA publishes for its n elements of a sample, in the form the other CTAs read it:
// six 8-byte words, each a 32-bit payload under a 32-bit tag (the launch's epoch).  A naturally
// aligned 8-byte store is indivisible, so a reader that finds the tag has the payload too: no
// flag, no fence, one round trip to L2.  Payloads: A = sum x (double, two words), the CTA's
// own mean A / n (double, two words), B = sum of squared deviations about that mean (float),
// n (int).
struct LnEntry {
    double A, mean;
    float B;
    int n;
};
__device__ __forceinline__ void ln_entry_store(unsigned long long *dst, int n, float c, double s1, double s2,
                                               int tag, int word)
{
    const double nd = static_cast<double>(n);
    const double A = nd * static_cast<double>(c) + s1;
    const double mean = n > 0 ? A / nd : 0.0;
    double B = n > 0 ? s2 - s1 * s1 / nd : 0.0;
    B = B > 0.0 ? B : 0.0;
    const unsigned long long a = static_cast<unsigned long long>(__double_as_longlong(A));
    const unsigned long long mu = static_cast<unsigned long long>(__double_as_longlong(mean));
    unsigned int payload;
    switch (word) {
    case 0: payload = static_cast<unsigned int>(a); break;
    case 1: payload = static_cast<unsigned int>(a >> 32); break;
    case 2: payload = static_cast<unsigned int>(mu); break;
    case 3: payload = static_cast<unsigned int>(mu >> 32); break;
    case 4: payload = __float_as_uint(static_cast<float>(B)); break;
    default: payload = static_cast<unsigned int>(n); break;
    }
    const unsigned long long v = (static_cast<unsigned long long>(static_cast<unsigned int>(tag)) << 32) | payload;
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(dst + word), "l"(v) : "memory");
}
// Reads one entry; false if any of its words does not carry `tag` yet.
__device__ __forceinline__ bool ln_entry_load(const unsigned long long *src, int tag, LnEntry &e)
{
    unsigned long long w[6];
#pragma unroll
    for (int i = 0; i < 3; ++i)
        asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];"
                     : "=l"(w[2 * i]), "=l"(w[2 * i + 1]) : "l"(src + 2 * i) : "memory");
    bool ok = true;
#pragma unroll
    for (int i = 0; i < 6; ++i) ok = ok && static_cast<int>(w[i] >> 32) == tag;
    e.A = __longlong_as_double(static_cast<long long>((w[1] << 32) | (w[0] & 0xffffffffull)));
    e.mean = __longlong_as_double(static_cast<long long>((w[3] << 32) | (w[2] & 0xffffffffull)));
    e.B = __uint_as_float(static_cast<unsigned int>(w[4]));
    e.n = static_cast<int>(static_cast<unsigned int>(w[5]));
    return ok;
}

__device__ __forceinline__ void ln_report(int *status, int what)
{
    if (atomicCAS(status, 0, -9 /* CUDALLM_ERR_DEVICE_TIMEOUT */) == 0) status[1] = (kRoleLayerNorm << 8) | what;
}

// Bounded wait until the shared counter `*counter` exceeds `value`.
__device__ __forceinline__ bool ln_wait_counter(const volatile int *counter, int value, volatile int *abort_flag,
                                                uint64_t limit_ns)
{
    if (*counter > value) return true;
    const uint64_t t0 = globaltimer_ns();
    while (*counter <= value) {
        __nanosleep(20);
        if (*abort_flag) return false;
        if (globaltimer_ns() - t0 > limit_ns) {
            *abort_flag = 1;
            return false;
        }
    }
    return true;
}

__global__ void __launch_bounds__(kLnStreamThreads, 1)
layernorm_stream_kernel(const LayerNormStreamParams p)
{
    extern __shared__ __align__(128) uint8_t ln_smem[];  // ring A, then ring B's stages of (x, gamma, beta)
    __shared__ __align__(8) uint64_t bars[2 * (kLnRingA + kLnRingBChunks)];
    __shared__ double warp_part[2][2][kLnRoleWarps];
    __shared__ double moments_of[kLnSlots][2];           // a sample's sums about its pilot, from the moments warps
    __shared__ float pilot_of[kLnSlots];
    __shared__ float stat_of[kLnSlots][4];               // a sample's (mean high, mean low, 1 / sqrt(var + eps))
    __shared__ volatile int stat_ready[kLnSlots];        // sample + 1 once stat_of holds its statistics
    __shared__ volatile int moments_done;                // samples the moments warps have finished
    __shared__ volatile int b_issued;                    // chunks loader B has started
    __shared__ int abort_word;
    volatile int *abort_flag = &abort_word;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = p.ctas;
    const uint32_t ring_a = smem_u32(ln_smem);
    const uint32_t ring_b = ring_a + kLnRingA * kLnChunkBytes;
    const uint32_t bar_base = smem_u32(bars);
    auto full_a = [&](int i) { return bar_base + 8u * i; };
    auto empty_a = [&](int i) { return bar_base + 8u * (kLnRingA + i); };
    auto full_b = [&](int i) { return bar_base + 8u * (2 * kLnRingA + i); };
    auto empty_b = [&](int i) { return bar_base + 8u * (2 * kLnRingA + kLnRingBChunks + i); };
    if (tid == 0) {
        abort_word = 0;
        moments_done = 0;
        b_issued = 0;
        for (int i = 0; i < kLnSlots; ++i) stat_ready[i] = 0;
        for (int i = 0; i < kLnRingA; ++i) {
            mbar_init(full_a(i), 1);
            mbar_init(empty_a(i), kLnRoleWarps);
        }
        for (int i = 0; i < kLnRingBChunks; ++i) {
            mbar_init(full_b(i), 1);
            mbar_init(empty_b(i), kLnRoleWarps);
        }
        fence_mbar_init();
    }
    __syncthreads();
    grid_launch_dependents();
    grid_dependency_wait();

    const long long lo = static_cast<long long>(cta) * p.slice_len;
    const long long n_ll = min(p.m, lo + p.slice_len) - lo;
    const int n = n_ll > 0 ? static_cast<int>(n_ll) : 0;                   // this CTA's elements of a sample
    const int C = (n + kLnChunkElems - 1) / kLnChunkElems;                 // ... in chunks (the last may be short)
    auto chunk_bytes = [&](int j) { return 4u * static_cast<uint32_t>(min(kLnChunkElems, n - j * kLnChunkElems)); };
    const int kinds = 1 + (p.gamma ? 1 : 0) + (p.beta ? 1 : 0);            // arrays per stage of ring B
    const int NB = kLnRingBChunks / kinds;                                 // stages of ring B

    int last_a = -1, last_b = -1;                        // loader lanes: the last chunk whose copies they started
    if (n == 0) {
        // nothing of any sample lies here: publish empty entries, so that nobody waits for this CTA
        if (tid < 6)
            for (int s = 0; s < p.batch; ++s)
                ln_entry_store(p.entries + (static_cast<long long>(s) * G + cta) * 6, 0, 0.f, 0.0, 0.0, p.tag_post, tid);
    } else if (warp < kLnRoleWarps) {
        // ------------------------------------------------------------- moments
        bool ok = true;
        int t = 0;
        for (int s = 0; s < p.batch; ++s) {
            double s1 = 0.0, s2 = 0.0;
            float c = 0.f;
            for (int j = 0; j < C; ++j, ++t) {
                const int use = t / kLnRingA, slot = t - use * kLnRingA;
                if (ok && !mbar_wait(full_a(slot), use & 1, abort_flag, p.wait_limit_ns)) {
                    if (lane == 0) ln_report(p.status, 0x11);
                    ok = false;
                }
                if (ok) {
                    const uint32_t chunk = ring_a + slot * kLnChunkBytes;
                    if (j == 0) c = ln_pilot(lds8(chunk));
                    float f1 = 0.f, f2 = 0.f;
#pragma unroll
                    for (int h = 0; h < kLnChunkElems / (4 * kLnRoleThreads); ++h) {
                        const int off = h * kLnRoleThreads * 4 + tid * 4;        // element of the chunk
                        if (j * kLnChunkElems + off < n) ln_add_piece4(lds4(chunk + off * 4), c, f1, f2);
                    }
                    ln_flush(f1, f2, s1, s2);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_a(slot));
            }
            s1 = warp_sum(s1);
            s2 = warp_sum(s2);
            if (lane == 0) {
                warp_part[s & 1][0][warp] = s1;
                warp_part[s & 1][1][warp] = s2;
            }
            named_bar_sync(1, kLnRoleThreads);
            if (tid == 0) {
                // the sample's sums in a fixed order, handed to the exchange warp (which is at most
                // kLnSlots - 2 samples behind: loader A waits for loader B, which waits for it)
                double t1 = 0.0, t2 = 0.0;
                for (int w = 0; w < kLnRoleWarps; ++w) {
                    t1 += warp_part[s & 1][0][w];
                    t2 += warp_part[s & 1][1][w];
                }
                const int k = s % kLnSlots;
                moments_of[k][0] = t1;
                moments_of[k][1] = t2;
                pilot_of[k] = c;
                __threadfence_block();
                moments_done = ok ? s + 1 : 0;
            }
        }
    } else if (warp < 2 * kLnRoleWarps) {
        // ------------------------------------------------------- normalisation
        const int at = tid - kLnRoleThreads;
        const uint64_t stream_out = l2_policy_evict_first();      // y is not read again
        bool ok = true;
        int t = 0;
        for (int q = 0; q < p.batch; ++q) {
            if (ok && !ln_wait_counter(&stat_ready[q % kLnSlots], q, abort_flag, p.wait_limit_ns)) {
                if (lane == 0) ln_report(p.status, 0x13);
                ok = false;
            }
            __threadfence_block();
            const int k = q % kLnSlots;
            const float mh = stat_of[k][0], ml = stat_of[k][1], rstd = stat_of[k][2];
            float *yq = p.y + static_cast<long long>(q) * p.m + lo;
            for (int j = 0; j < C; ++j, ++t) {
                const int use = t / NB, stage = t - use * NB;
                if (ok && !mbar_wait(full_b(stage), use & 1, abort_flag, p.wait_limit_ns)) {
                    if (lane == 0) ln_report(p.status, 0x14);
                    ok = false;
                }
                if (ok) {
                    const uint32_t sx = ring_b + stage * (kinds * kLnChunkBytes);
                    const uint32_t sg = sx + kLnChunkBytes, sb = sg + (p.gamma ? kLnChunkBytes : 0);
#pragma unroll
                    for (int h = 0; h < kLnChunkElems / (4 * kLnRoleThreads); ++h) {
                        const int off = h * kLnRoleThreads * 4 + at * 4;         // element of the chunk
                        const int e = j * kLnChunkElems + off;
                        if (e < n) {
                            float4 v = lds4(sx + off * 4);
                            float4 gm = make_float4(1.f, 1.f, 1.f, 1.f), bt = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (p.gamma) gm = lds4(sg + off * 4);
                            if (p.beta) bt = lds4(sb + off * 4);
                            v.x = ln_apply(v.x, mh, ml, rstd, gm.x, bt.x);
                            v.y = ln_apply(v.y, mh, ml, rstd, gm.y, bt.y);
                            v.z = ln_apply(v.z, mh, ml, rstd, gm.z, bt.z);
                            v.w = ln_apply(v.w, mh, ml, rstd, gm.w, bt.w);
                            st4_stream(yq + e, v, stream_out);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_b(stage));
            }
        }
    } else if (warp == 2 * kLnRoleWarps) {
        // ------------------------------------------------------------ loader A
        if (lane == 0) {
            const uint64_t keep = l2_policy_evict_last();        // these lines are wanted again, `lead` chunks later
            int t = 0;
            for (int s = 0; s < p.batch && t >= 0; ++s) {
                const float *src = p.x + static_cast<long long>(s) * p.m + lo;
                for (int j = 0; j < C; ++j, ++t) {
                    const int use = t / kLnRingA, slot = t - use * kLnRingA;
                    if (t >= p.lead && !ln_wait_counter(&b_issued, t - p.lead, abort_flag, p.wait_limit_ns)) {
                        ln_report(p.status, 0x10);
                        t = -1;
                        break;
                    }
                    if (use > 0 && !mbar_wait(empty_a(slot), (use - 1) & 1, abort_flag, p.wait_limit_ns)) {
                        ln_report(p.status, 0x15);
                        t = -1;
                        break;
                    }
                    fence_proxy_async_smem();            // the warps' reads of the slot come before the copy's writes
                    mbar_expect_tx(full_a(slot), chunk_bytes(j));
                    bulk_load_hint(ring_a + slot * kLnChunkBytes, src + j * kLnChunkElems, chunk_bytes(j), full_a(slot), keep);
                    last_a = t;
                }
            }
        }
    } else if (warp == 2 * kLnRoleWarps + 1) {
        // ------------------------------------------------------------ loader B
        if (lane == 0) {
            const uint64_t once = l2_policy_evict_first(), keep = l2_policy_evict_last();
            int t = 0;
            for (int q = 0; q < p.batch && t >= 0; ++q) {
                // x of sample q has passed through the moments warps: it is in L2 (and, in place,
                // may now be overwritten once this copy of it has landed)
                if (!ln_wait_counter(&moments_done, q, abort_flag, p.wait_limit_ns)) {
                    ln_report(p.status, 0x16);
                    break;
                }
                const float *src = p.x + static_cast<long long>(q) * p.m + lo;
                for (int j = 0; j < C; ++j, ++t) {
                    const int use = t / NB, stage = t - use * NB;
                    if (use > 0 && !mbar_wait(empty_b(stage), (use - 1) & 1, abort_flag, p.wait_limit_ns)) {
                        ln_report(p.status, 0x17);
                        t = -1;
                        break;
                    }
                    const uint32_t bytes = chunk_bytes(j);
                    const uint32_t sx = ring_b + stage * (kinds * kLnChunkBytes);
                    const uint32_t sg = sx + kLnChunkBytes, sb = sg + (p.gamma ? kLnChunkBytes : 0);
                    fence_proxy_async_smem();
                    mbar_expect_tx(full_b(stage), bytes * kinds);
                    bulk_load_hint(sx, src + j * kLnChunkElems, bytes, full_b(stage), once);
                    if (p.gamma) bulk_load_hint(sg, p.gamma + lo + j * kLnChunkElems, bytes, full_b(stage), keep);
                    if (p.beta) bulk_load_hint(sb, p.beta + lo + j * kLnChunkElems, bytes, full_b(stage), keep);
                    last_b = t;
                    b_issued = t + 1;
                }
            }
        }
    } else {
        // ------------------------------------------------------------ exchange
        // The only warps that talk to the other CTAs.  (An acquire or a release in a warp that
        // has loads and stores in flight waits for those, microseconds per sample.)  Each
        // publishes this CTA's moments of its next sample s as soon as the moments warps have
        // handed them over, and works out the statistics of its sample q as soon as all G
        // entries of q are there; neither duty ever blocks the other.
        const int first = warp - (2 * kLnRoleWarps + 2);
        int s = first, q = first;
        uint64_t t_idle = globaltimer_ns();
        while (q < p.batch) {
            bool progress = false;
            if (s < p.batch && moments_done > s) {
                __threadfence_block();
                const int k = s % kLnSlots;
                if (lane < 6)
                    ln_entry_store(p.entries + (static_cast<long long>(s) * G + cta) * 6, n, pilot_of[k],
                                   moments_of[k][0], moments_of[k][1], p.tag_post, lane);
                s += kLnExchangeWarps;
                progress = true;
            }
            if (q < s) {
                // entries lane, lane + 32, ... of sample q: all their loads are in flight together
                const unsigned long long *base = p.entries + static_cast<long long>(q) * G * 6;
                LnEntry e[kLnMaxCtas / 32];
                bool all = true;
#pragma unroll
                for (int u = 0; u < kLnMaxCtas / 32; ++u) {
                    const int k = lane + 32 * u;
                    e[u].A = 0.0; e[u].mean = 0.0; e[u].B = 0.f; e[u].n = 0;
                    if (k < G) all = ln_entry_load(base + k * 6, p.epoch, e[u]) && all;
                }
                if (__all_sync(0xffffffffu, all)) {
                    // mean = sum A_k / m, then M2 = sum (B_k + n_k (mean_k - mean)^2): the same
                    // arithmetic in the same order in every CTA
                    double a = 0.0;
#pragma unroll
                    for (int u = 0; u < kLnMaxCtas / 32; ++u) a += e[u].A;
                    const double mean = warp_sum(a) * p.inv_m;
                    float m2 = 0.f;
#pragma unroll
                    for (int u = 0; u < kLnMaxCtas / 32; ++u) {
                        const float dm = static_cast<float>(e[u].mean - mean);
                        m2 += e[u].B + static_cast<float>(e[u].n) * dm * dm;
                    }
                    m2 = warp_sum_f32(m2);
                    if (lane == 0) {
                        const double var = static_cast<double>(m2) * p.inv_m;
                        const float mh = static_cast<float>(mean);
                        float *out = stat_of[q % kLnSlots];
                        out[0] = mh;
                        out[1] = static_cast<float>(mean - static_cast<double>(mh));
                        out[2] = static_cast<float>(rsqrt(var + p.eps));
                        __threadfence_block();
                        stat_ready[q % kLnSlots] = q + 1;
                    }
                    q += kLnExchangeWarps;
                    progress = true;
                }
            }
            if (progress) {
                t_idle = globaltimer_ns();
            } else {
                __nanosleep(40);
                if (*abort_flag) break;
                if (globaltimer_ns() - t_idle > p.wait_limit_ns) {
                    *abort_flag = 1;
                    if (lane == 0) ln_report(p.status, 0x12);
                    break;
                }
            }
        }
    }
    __syncthreads();
    // After a wait that ran out the warps may have left chunks unread: their copies must still
    // land before the CTA gives up its shared memory.  Each loader lane polls (bounded) the
    // chunks it started last; on the normal path every copy was awaited by the warps.
    if (*abort_flag) {
        for (int t = last_a; t >= 0 && t > last_a - kLnRingA; --t) {
            const int use = t / kLnRingA, slot = t - use * kLnRingA;
            for (int k = 0; k < 20000 && !mbar_try_wait(full_a(slot), use & 1); ++k) __nanosleep(100);
        }
        for (int t = last_b; t >= 0 && t > last_b - NB; --t) {
            const int use = t / NB, stage = t - use * NB;
            for (int k = 0; k < 20000 && !mbar_try_wait(full_b(stage), use & 1); ++k) __nanosleep(100);
        }
    }
}

}  // namespace cudallm
