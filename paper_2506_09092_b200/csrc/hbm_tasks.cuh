// Bandwidth-bound kernels for the paper's benchmark tasks on float32 arrays:
// Task 8 (matrix transpose), Task 14 (reduction: sum), Task 15 (dot product)
// and Task 4 (LayerNorm).  None of them is a contraction; what matters is that
// every byte crosses HBM once, in full cache lines, with enough of them in
// flight.
#pragma once
#include "ptx.cuh"

namespace cudallm {

// status detail codes of these kernels: (role << 8) | what
enum : int { kRoleTranspose = 4, kRoleLayerNorm = 5 };

__device__ __forceinline__ void task_report_timeout(int *status, int role, int what)
{
    if (atomicCAS(status, 0, -9 /* CUDALLM_ERR_DEVICE_TIMEOUT */) == 0) status[1] = (role << 8) | what;
}

// ----------------------------------------------------------- TMA helpers --
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// (the tensor maps are rank 3 with a third extent of 1, like the GEMM's)
__device__ __forceinline__ void tma_load_3d(const CUtensorMap *tm, uint32_t smem_addr, uint32_t bar, int x, int y, int z)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(smem_addr), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}

// ============================================================== Task 8 ====
// AT[j][i] = A[i][j].  Every warp runs its own pipeline over 64 x 64 patches of
// A: lane 0 asks TMA for the patch as four 32 x 32 boxes (128-byte swizzle, so
// that rows AND columns of a box can be read without bank conflicts) into one
// of the warp's ring stages; when the bytes have landed the warp turns each
// box around -- lane c reads column c of the box (one conflict-free 128-byte
// wavefront per row) and writes it as row c of a staging block, again in the
// swizzled layout -- and lane 0 stores the block with TMA to AT.  Both
// directions move whole 128-byte lines, and the patches that run at the same
// time are neighbours along a row of A, so DRAM sees 256 contiguous bytes per
// row of a patch.  Out-of-range parts of a box are zero-filled on load and
// clipped on store (rows and cols are multiples of 4 on this path, so the
// 16-byte clipping granule is exact).
constexpr int kTrWarps = 4;                      // warps per CTA
constexpr int kTrStages = 2;                     // 64 x 64 patches in flight per warp
constexpr int kTrPatch = 64;
constexpr int kTrPatchBytes = kTrPatch * kTrPatch * 4;               // 16 KiB
constexpr int kTrWarpBytes = kTrStages * kTrPatchBytes + 2 * 4096;   // ring + two staging blocks
constexpr int kTrSmemBytes = kTrWarps * kTrWarpBytes + kTrWarps * kTrStages * 8 + 1024;

struct TransposeParams {
    int rows, cols;          // of A
    int patches_r, patches_c;
    int *status;
};

__global__ void __launch_bounds__(kTrWarps * 32)
transpose_tma_kernel(const __grid_constant__ CUtensorMap tmap_in, const __grid_constant__ CUtensorMap tmap_out,
                     const TransposeParams p)
{
    extern __shared__ uint8_t tr_smem_raw[];
    const uint32_t base = (smem_u32(tr_smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ring = base + warp * kTrWarpBytes;
    const uint32_t staging = ring + kTrStages * kTrPatchBytes;
    const uint32_t bars = base + kTrWarps * kTrWarpBytes + warp * kTrStages * 8;
    __shared__ int abort_flag;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        prefetch_tensormap(&tmap_in);
        prefetch_tensormap(&tmap_out);
    }
    if (lane == 0) {
        for (int s = 0; s < kTrStages; ++s) mbar_init(bars + 8 * s, 1);
        fence_mbar_init();
        fence_proxy_async_smem();
    }
    __syncthreads();

    const long long total = static_cast<long long>(p.patches_r) * p.patches_c;
    const long long step = static_cast<long long>(gridDim.x) * kTrWarps;
    const long long first = static_cast<long long>(blockIdx.x) * kTrWarps + warp;

    auto issue = [&](long long patch, int s) {           // lane 0 only
        const int pr = static_cast<int>(patch / p.patches_c);
        const int pc = static_cast<int>(patch - static_cast<long long>(pr) * p.patches_c);
        const uint32_t dst = ring + s * kTrPatchBytes;
        mbar_expect_tx(bars + 8 * s, kTrPatchBytes);
#pragma unroll
        for (int b = 0; b < 4; ++b)                      // box b: rows 32 (b / 2).., columns 32 (b % 2)..
            tma_load_3d(&tmap_in, dst + b * 4096, bars + 8 * s, pc * kTrPatch + 32 * (b & 1),
                        pr * kTrPatch + 32 * (b >> 1), 0);
    };

    // prologue: fill the ring
    if (lane == 0)
        for (int s = 0; s < kTrStages; ++s)
            if (first + s * step < total) issue(first + s * step, s);

    uint32_t sel = 0;
    int s = 0;
    uint32_t phase = 0;
    for (long long patch = first; patch < total; patch += step) {
        bool ok = mbar_wait(bars + 8 * s, phase, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {
            if (lane == 0) task_report_timeout(p.status, kRoleTranspose, s);
            break;
        }
        const int pr = static_cast<int>(patch / p.patches_c);
        const int pc = static_cast<int>(patch - static_cast<long long>(pr) * p.patches_c);
        const uint32_t src = ring + s * kTrPatchBytes;
#pragma unroll 1
        for (int b = 0; b < 4; ++b) {
            const int r0 = pr * kTrPatch + 32 * (b >> 1);            // first row / column of the box in A
            const int c0 = pc * kTrPatch + 32 * (b & 1);
            if (r0 >= p.rows || c0 >= p.cols) continue;               // warp-uniform: nothing to store
            const uint32_t box = src + b * 4096;
            // lane = column c of the box: element (r, c) lies at r * 128 + ((c / 4) ^ (r % 8)) * 16 + (c % 4) * 4
            float v[32];
#pragma unroll
            for (int r = 0; r < 32; ++r)
                v[r] = ld_shared_f32(box + r * 128 + ((((lane >> 2) ^ (r & 7))) << 4) + (lane & 3) * 4);
            const uint32_t blk = staging + sel * 4096u;
            sel ^= 1u;
            if (lane == 0) bulk_wait_group_read<1>();                 // the store before the last has read blk
            __syncwarp();
#pragma unroll
            for (int q = 0; q < 8; ++q)                               // row `lane` of the transposed box
                st_shared_v4(blk + lane * 128 + ((q ^ (lane & 7)) << 4), v[4 * q], v[4 * q + 1], v[4 * q + 2],
                             v[4 * q + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                tma_store_3d(&tmap_out, blk, r0, c0, 0);                 // AT: x = row index of A, y = column of A
                bulk_commit_group();
            }
        }
        __syncwarp();                                                 // every lane has read the ring stage
        if (lane == 0 && patch + kTrStages * step < total) issue(patch + kTrStages * step, s);
        if (++s == kTrStages) { s = 0; phase ^= 1; }
    }
    if (lane == 0) bulk_wait_group_read<0>();
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
// A group of G CTAs owns a sample; CTA g of the group works on elements
// [g * slice, (g + 1) * slice).  Pass 1 reads the slice from HBM and adds x and
// x^2 in double (exact products, so the variance has no cancellation problem);
// the CTAs of the group publish their two sums and meet at a counter in global
// memory (a bounded wait; all CTAs of a launch are resident: one per SM at
// most); every CTA then adds the G partials in index order, so all of them
// derive the same mean and 1/sqrt(var + eps).  Pass 2 reads the slice again --
// it was just read, and the host sizes the number of concurrent groups so that
// the live samples fit in L2 -- and writes y.  The wait for sample s is hidden
// behind pass 1 of the group's next sample.
struct LayerNormParams {
    const float *x, *gamma, *beta;
    float *y;
    long long m;             // elements per sample
    long long slice;         // elements per CTA of a group (a multiple of 4)
    int batch;
    int group_size;          // G
    int num_groups;          // groups that run side by side; grid = num_groups * G
    double eps;
    double *partials;        // [batch][G][2]
    unsigned int *arrived;   // [batch], zero at launch
    int *status;
};

constexpr int kLnThreads = 512;

template <bool VEC>
__global__ void __launch_bounds__(kLnThreads)
layernorm_kernel(const LayerNormParams p)
{
    __shared__ double warp_part[kLnThreads / 32];
    __shared__ double stats[2];
    __shared__ int abort_flag;
    const int group = blockIdx.x / p.group_size;
    const int g = blockIdx.x - group * p.group_size;
    const long long lo = static_cast<long long>(g) * p.slice;
    const long long hi = min(p.m, lo + p.slice);
    if (threadIdx.x == 0) abort_flag = 0;
    __syncthreads();

    // pass 1 of one sample: this CTA's sums of x and x^2, published for the group
    auto pass1 = [&](int s) {
        const float *xs = p.x + static_cast<long long>(s) * p.m;
        double s1 = 0.0, s2 = 0.0;
        if (VEC) {
            const float4 *xv = reinterpret_cast<const float4 *>(xs + lo);
            const long long nv = hi > lo ? (hi - lo) >> 2 : 0;
            long long i = threadIdx.x;
            for (; i + 3 * kLnThreads < nv; i += 4 * kLnThreads) {
                float4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) v[u] = __ldcg(xv + i + u * kLnThreads);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const double a = v[u].x, b = v[u].y, c = v[u].z, d = v[u].w;
                    s1 += (a + b) + (c + d);
                    s2 = fma(a, a, s2); s2 = fma(b, b, s2); s2 = fma(c, c, s2); s2 = fma(d, d, s2);
                }
            }
            for (; i < nv; i += kLnThreads) {
                const float4 v = __ldcg(xv + i);
                const double a = v.x, b = v.y, c = v.z, d = v.w;
                s1 += (a + b) + (c + d);
                s2 = fma(a, a, s2); s2 = fma(b, b, s2); s2 = fma(c, c, s2); s2 = fma(d, d, s2);
            }
        } else {
            for (long long i = lo + threadIdx.x; i < hi; i += kLnThreads) {
                const double a = __ldcg(xs + i);
                s1 += a;
                s2 = fma(a, a, s2);
            }
        }
        const double t1 = block_sum(s1, warp_part);
        const double t2 = block_sum(s2, warp_part);
        if (threadIdx.x == 0) {
            double *slot = p.partials + (static_cast<long long>(s) * p.group_size + g) * 2;
            __stcg(slot, t1);
            __stcg(slot + 1, t2);
            __threadfence();
            atomicAdd(p.arrived + s, 1u);
        }
    };

    int s = group;
    if (s < p.batch) pass1(s);
    for (; s < p.batch; s += p.num_groups) {
        const int next = s + p.num_groups;
        if (next < p.batch) pass1(next);
        // meet the other CTAs of the group
        if (threadIdx.x == 0) {
            bool ok = true;
            const uint64_t t0 = globaltimer_ns();
            unsigned int seen;
            do {
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(p.arrived + s) : "memory");
                if (seen >= static_cast<unsigned int>(p.group_size)) break;
                if (globaltimer_ns() - t0 > kWaitLimitNs) { ok = false; break; }
            } while (true);
            if (!ok) {
                abort_flag = 1;
                task_report_timeout(p.status, kRoleLayerNorm, 0);
            } else {
                double s1 = 0.0, s2 = 0.0;
                const double *slot = p.partials + static_cast<long long>(s) * p.group_size * 2;
                for (int k = 0; k < p.group_size; ++k) {
                    s1 += __ldcg(slot + 2 * k);
                    s2 += __ldcg(slot + 2 * k + 1);
                }
                const double mean = s1 / static_cast<double>(p.m);
                double var = s2 / static_cast<double>(p.m) - mean * mean;
                var = var > 0.0 ? var : 0.0;
                stats[0] = mean;
                stats[1] = rsqrt(var + p.eps);
            }
        }
        __syncthreads();
        if (abort_flag) return;
        const double rstd = stats[1];
        const double mean = stats[0];
        __syncthreads();                                 // stats[] is rewritten for the next sample
        const float *xs = p.x + static_cast<long long>(s) * p.m;
        float *ys = p.y + static_cast<long long>(s) * p.m;
        if (VEC) {
            const float4 *xv = reinterpret_cast<const float4 *>(xs + lo);
            const float4 *gv = reinterpret_cast<const float4 *>(p.gamma + lo);
            const float4 *bv = reinterpret_cast<const float4 *>(p.beta + lo);
            float4 *yv = reinterpret_cast<float4 *>(ys + lo);
            const long long nv = hi > lo ? (hi - lo) >> 2 : 0;
            for (long long i = threadIdx.x; i < nv; i += 2 * kLnThreads) {
                const bool two = i + kLnThreads < nv;
                const float4 v0 = __ldcg(xv + i);
                const float4 v1 = two ? __ldcg(xv + i + kLnThreads) : v0;
                const float4 g0 = p.gamma ? __ldg(gv + i) : make_float4(1.f, 1.f, 1.f, 1.f);
                const float4 g1 = (p.gamma && two) ? __ldg(gv + i + kLnThreads) : g0;
                const float4 b0 = p.beta ? __ldg(bv + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                const float4 b1 = (p.beta && two) ? __ldg(bv + i + kLnThreads) : b0;
                float4 o;
                o.x = fmaf(static_cast<float>((static_cast<double>(v0.x) - mean) * rstd), g0.x, b0.x);
                o.y = fmaf(static_cast<float>((static_cast<double>(v0.y) - mean) * rstd), g0.y, b0.y);
                o.z = fmaf(static_cast<float>((static_cast<double>(v0.z) - mean) * rstd), g0.z, b0.z);
                o.w = fmaf(static_cast<float>((static_cast<double>(v0.w) - mean) * rstd), g0.w, b0.w);
                __stcs(yv + i, o);
                if (two) {
                    o.x = fmaf(static_cast<float>((static_cast<double>(v1.x) - mean) * rstd), g1.x, b1.x);
                    o.y = fmaf(static_cast<float>((static_cast<double>(v1.y) - mean) * rstd), g1.y, b1.y);
                    o.z = fmaf(static_cast<float>((static_cast<double>(v1.z) - mean) * rstd), g1.z, b1.z);
                    o.w = fmaf(static_cast<float>((static_cast<double>(v1.w) - mean) * rstd), g1.w, b1.w);
                    __stcs(yv + i + kLnThreads, o);
                }
            }
        } else {
            for (long long i = lo + threadIdx.x; i < hi; i += kLnThreads) {
                const float gm = p.gamma ? p.gamma[i] : 1.f;
                const float bt = p.beta ? p.beta[i] : 0.f;
                ys[i] = fmaf(static_cast<float>((static_cast<double>(__ldcg(xs + i)) - mean) * rstd), gm, bt);
            }
        }
    }
}

}  // namespace cudallm
