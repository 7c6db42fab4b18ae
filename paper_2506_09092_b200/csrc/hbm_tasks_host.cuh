// Host side of the entry points declared in include/cudallm_tasks.h.  This file
// is included at the end of cudallm_gemm.cu and uses that file's device state,
// workspace, tensor-map cache and error plumbing.
#pragma once

namespace {

__device__ cudallm::ReduceScratch g_reduce_scratch;      // zero-initialised: the ticket starts at 0

constexpr int64_t kTaskMaxElems = int64_t(1) << 40;

int task_device(int *dev_out)
{
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    *dev_out = dev;
    return probe_device(dev);
}

int run_reduce(const float *a, const float *b, int64_t n, float *result, bool dot, void *stream_v)
{
    if (n < 0 || n > kTaskMaxElems) return CUDALLM_ERR_INVALID_DIM;
    if (!result || (n > 0 && (!a || (dot && !b)))) return CUDALLM_ERR_INVALID_POINTER;
    if ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(result)
         | (dot ? reinterpret_cast<uintptr_t>(b) : 0)) & 3)
        return CUDALLM_ERR_MISALIGNED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = 0;
    std::lock_guard<std::mutex> lock(g_mutex);
    int st = task_device(&dev);
    if (st != CUDALLM_OK) return st;
    static ReduceScratch *scratch_of[kMaxDevices] = {};        // looked up once per device (g_mutex is held)
    if (!scratch_of[dev])
        CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void **>(&scratch_of[dev]), g_reduce_scratch));
    ReduceScratch *scratch = scratch_of[dev];
    // one block per 8192 elements, at most four blocks of 512 threads per SM
    int64_t blocks = cdiv(n, int64_t(kRedThreads) * 16);
    const int64_t cap = std::min<int64_t>(kRedMaxBlocks, int64_t(4) * g_dev[dev].sm_count);
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const bool vec = !dot || ((reinterpret_cast<uintptr_t>(a) & 15) == (reinterpret_cast<uintptr_t>(b) & 15));
    const unsigned g = (unsigned)blocks;
    if (dot) {
        if (vec) reduce_kernel<true, true><<<g, kRedThreads, 0, stream>>>(a, b, n, result, scratch);
        else     reduce_kernel<true, false><<<g, kRedThreads, 0, stream>>>(a, b, n, result, scratch);
    } else {
        reduce_kernel<false, true><<<g, kRedThreads, 0, stream>>>(a, a, n, result, scratch);
    }
    CUDA_TRY(cudaGetLastError());
    return CUDALLM_OK;
}

}  // namespace

int cudallm_sum_f32(const float *x, int64_t n, float *result, void *stream)
{
    return run_reduce(x, nullptr, n, result, false, stream);
}

int cudallm_dot_f32(const float *a, const float *b, int64_t n, float *result, void *stream)
{
    return run_reduce(a, b, n, result, true, stream);
}

int cudallm_transpose_f32(const float *A, float *AT, int64_t rows, int64_t cols, int64_t lda, int64_t ldat,
                          void *stream_v)
{
    if (rows < 0 || cols < 0 || rows > kMaxDim || cols > kMaxDim) return CUDALLM_ERR_INVALID_DIM;
    if (rows == 0 || cols == 0) return CUDALLM_OK;
    if (lda < cols || ldat < rows) return CUDALLM_ERR_INVALID_LD;
    if (lda > kTaskMaxElems || ldat > kTaskMaxElems) return CUDALLM_ERR_INVALID_DIM;
    if ((long double)rows * lda > (long double)kMaxElems || (long double)cols * ldat > (long double)kMaxElems)
        return CUDALLM_ERR_INVALID_DIM;
    if (!A || !AT) return CUDALLM_ERR_INVALID_POINTER;
    if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(AT)) & 3) return CUDALLM_ERR_MISALIGNED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = 0;
    std::lock_guard<std::mutex> lock(g_mutex);
    int st = task_device(&dev);
    if (st != CUDALLM_OK) return st;
    DeviceState &d = g_dev[dev];

    const bool vec = ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(AT)) & 15) == 0
                  && rows % 4 == 0 && cols % 4 == 0 && lda % 4 == 0 && ldat % 4 == 0;
    if (!vec) {
        const int64_t tiles_c = cdiv(cols, 32);
        const int64_t tiles = cdiv(rows, 32) * tiles_c;
        const int64_t grid = std::min<int64_t>(tiles, int64_t(d.sm_count) * 16);
        transpose_simple_kernel<<<(unsigned)grid, 256, 0, stream>>>(A, AT, (int)rows, (int)cols, lda, ldat,
                                                                    (int)tiles_c, tiles);
        CUDA_TRY(cudaGetLastError());
        return CUDALLM_OK;
    }
    const int64_t tiles_c = cdiv(cols, 64);
    const int64_t tiles = cdiv(rows, 64) * tiles_c;            // one CTA each
    if (tiles > kMaxDim) return CUDALLM_ERR_INVALID_DIM;
    transpose64_kernel<<<(unsigned)tiles, 256, 0, stream>>>(A, AT, (int)rows, (int)cols, lda, ldat, (int)tiles_c);
    CUDA_TRY(cudaGetLastError());
    return CUDALLM_OK;
}

int cudallm_layernorm_f32(const float *x, const float *gamma, const float *beta, float *y, int64_t batch,
                          int64_t m, float eps, void *stream_v)
{
    if (batch < 0 || m < 0 || batch > kMaxDim || m > kTaskMaxElems) return CUDALLM_ERR_INVALID_DIM;
    if (!(eps >= 0.f) || !(eps <= 3.0e38f)) return CUDALLM_ERR_INVALID_DIM;
    if ((long double)batch * m > (long double)kMaxElems) return CUDALLM_ERR_INVALID_DIM;
    if (batch == 0 || m == 0) return CUDALLM_OK;
    if (!x || !y) return CUDALLM_ERR_INVALID_POINTER;
    const uintptr_t all = reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)
                        | reinterpret_cast<uintptr_t>(gamma) | reinterpret_cast<uintptr_t>(beta);
    if (all & 3) return CUDALLM_ERR_MISALIGNED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = 0;
    std::lock_guard<std::mutex> lock(g_mutex);
    int st = task_device(&dev);
    if (st != CUDALLM_OK) return st;
    DeviceState &d = g_dev[dev];

    const bool vec = (all & 31) == 0 && m % 8 == 0;            // 32-byte loads and stores
    const int sms = d.sm_count;
    // Aligned data is cut into 4 KiB blocks that the CTAs of a group take in turn.
    const int64_t total_blocks = cdiv(m, (int64_t)kLnBlockPieces * 8);
    // Shared-memory kernel: the blocks of a bundle of T samples per CTA, one CTA per SM.
    constexpr int64_t kLnSmemBudget = 227 * 1024 - 2048;
    const int64_t cap = kLnSmemBudget / 4;                     // elements of shared memory per CTA
    int64_t groups = 1, T = 1;
    int64_t G = std::max<int64_t>(1, std::min<int64_t>(sms, total_blocks));
    const int64_t chunks = cdiv(cdiv(total_blocks, G), kLnChunkBlocks);
    int64_t slice = cdiv(total_blocks, G) * (kLnBlockBytes / 4);   // shared memory per sample, in elements
    bool use_smem = vec && slice <= cap && chunks <= kLnMaxChunks;
    if (use_smem) {
        const int64_t max_groups = std::max<int64_t>(1, sms / G);
        // samples per bundle: what fits, but no more than needed to give every group one bundle
        while (T * 2 <= kLnMaxBundle && T * 2 * slice <= cap && T * max_groups < batch) T *= 2;
        groups = std::min<int64_t>(max_groups, cdiv(batch, T));
        // More than two bundles per group: every bundle costs a meeting of the group with
        // the memory system idle; streaming with fewer meetings is cheaper even though x
        // is then read twice.
        if (cdiv(cdiv(batch, T), groups) > 2) use_smem = false;
    }
    if (!use_smem) {
        // Streaming kernel, one CTA per SM: blocks in turn (aligned data) or contiguous
        // slices of at least 1024 elements (anything else).
        G = std::max<int64_t>(1, std::min<int64_t>(sms, vec ? total_blocks : m / 1024));
        slice = round_up(cdiv(m, G), 8);
        if (!vec) G = cdiv(m, slice);                          // no empty CTAs
        const int64_t max_groups = std::max<int64_t>(1, sms / G);
        T = std::min<int64_t>(kLnMaxBundle, std::max<int64_t>(1, cdiv(batch, max_groups)));
        groups = std::min<int64_t>(max_groups, cdiv(batch, T));
    }

    const size_t off_arrived = kHeaderBytes;
    const size_t off_partials = (size_t)round_up((int64_t)(off_arrived + (size_t)batch * 4), 256);
    const size_t total = off_partials + (size_t)batch * (size_t)G * 32;
    st = ensure_workspace(dev, total, stream);
    if (st != CUDALLM_OK) return st;
    uint8_t *ws = static_cast<uint8_t *>(d.ws);
    CUDA_TRY(cudaMemsetAsync(ws + off_arrived, 0, (size_t)batch * 4, stream));

    LayerNormParams lp{};
    lp.x = x; lp.gamma = gamma; lp.beta = beta; lp.y = y;
    lp.m = m; lp.slice = slice;
    lp.batch = (int)batch; lp.group_size = (int)G; lp.num_groups = (int)groups; lp.bundle = (int)T;
    lp.eps = (double)eps;
    lp.inv_m = 1.0 / (double)m;
    lp.partials = reinterpret_cast<double *>(ws + off_partials);
    lp.arrived = reinterpret_cast<unsigned int *>(ws + off_arrived);
    lp.status = reinterpret_cast<int *>(ws);
    const unsigned grid = (unsigned)(groups * G);              // all CTAs are resident at once
    if (use_smem) {
        const size_t smem = (size_t)(T * slice * 4);
        if (!d.smem_attr_set[10]) {
            CUDA_TRY(cudaFuncSetAttribute(layernorm_smem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)kLnSmemBudget));
            d.smem_attr_set[10] = true;
        }
        layernorm_smem_kernel<<<grid, kLnThreads, smem, stream>>>(lp);
    } else if (vec) {
        layernorm_stream_kernel<true><<<grid, kLnThreads, 0, stream>>>(lp);
    } else {
        layernorm_stream_kernel<false><<<grid, kLnThreads, 0, stream>>>(lp);
    }
    CUDA_TRY(cudaGetLastError());
    return CUDALLM_OK;
}
