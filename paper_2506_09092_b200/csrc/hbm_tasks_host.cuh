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
    if (dot) return vec ? launch_serialised(reduce_kernel<true, true>, g, kRedThreads, stream, a, b, (long long)n, result, scratch)
                        : launch_serialised(reduce_kernel<true, false>, g, kRedThreads, stream, a, b, (long long)n, result, scratch);
    return launch_serialised(reduce_kernel<false, true>, g, kRedThreads, stream, a, a, (long long)n, result, scratch);
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
        return launch_serialised(transpose_simple_kernel, (unsigned)grid, 256, stream, A, AT, (int)rows, (int)cols,
                           (long long)lda, (long long)ldat, (int)tiles_c, (long long)tiles);
    }
    const int64_t tiles_c = cdiv(cols, 64);
    const int64_t tiles = cdiv(rows, 64) * tiles_c;            // one CTA each
    if (tiles > kMaxDim) return CUDALLM_ERR_INVALID_DIM;
    return launch_serialised(transpose64_kernel, (unsigned)tiles, 256, stream, A, AT, (int)rows, (int)cols,
                       (long long)lda, (long long)ldat, (int)tiles_c);
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
    // The persistent kernel (x read from DRAM once): one CTA per SM, each with its slice of every
    // sample.  Taken where it was measured faster than the two kernels below: samples of 8 to
    // 20 MB (4 MB with 32 or more of them) -- smaller ones finish before the exchange of the
    // moments between the CTAs (several microseconds) is amortised, larger ones do not stay in
    // L2 between their two reads -- and at least four samples.
    const int ln_path = g_layernorm_path.load();
    if (vec && ln_path != 1) {
        const int64_t G = std::min<int64_t>({int64_t(sms), int64_t(kLnMaxCtas), std::max<int64_t>(1, m / 1024)});
        const int64_t slice_len = round_up(cdiv(m, G), 8);
        const bool worth = (batch >= 4 && m <= (int64_t(5) << 20) && (m >= (int64_t(1) << 21) || (m >= (int64_t(1) << 20) && batch >= 32)))
                        || ln_path == 2;
        if (worth && slice_len < (int64_t(1) << 30)) {
            // Loader A runs ahead of loader B by what keeps about 34 MB of x in L2 between its two
            // reads, at least one sample and a half, at most 8 samples (loader B is at most 3
            // chunks ahead of the normalisation, and the roles hand samples over in 16 slots).
            const int64_t chunks = cdiv(slice_len, kLnChunkElems);
            const int64_t lead = std::max<int64_t>(chunks + (chunks + 1) / 2,
                                                   std::min<int64_t>((kLnSlots - 8) * chunks,
                                                                     (int64_t(34) << 20) / (G * kLnChunkBytes)));
            // The entries live in their own area of the workspace header, whose 8-byte words are
            // zero or an earlier launch's (payload, epoch) pairs: a stale word cannot pass for
            // this launch's tag.  The area holds kEntryBytes / 48 entries; larger batches go in pieces.
            const int64_t per_launch = std::max<int64_t>(1, int64_t(kEntryBytes / 48) / G);
            Workspace &w = workspace_for(d, stream);
            st = ensure_workspace(w, kHeaderBytes, stream);
            if (st != CUDALLM_OK) return st;
            uint8_t *ws = static_cast<uint8_t *>(w.ptr);
            if (!d.layernorm_attr_set) {
                CUDA_TRY(cudaFuncSetAttribute(layernorm_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              kLnStreamSmem));
                d.layernorm_attr_set = true;
            }
            for (int64_t s0 = 0; s0 < batch; s0 += per_launch) {
                LayerNormStreamParams sp{};
                sp.x = x + s0 * m; sp.gamma = gamma; sp.beta = beta; sp.y = y + s0 * m;
                sp.m = m; sp.slice_len = slice_len;
                sp.batch = (int)std::min<int64_t>(per_launch, batch - s0); sp.ctas = (int)G; sp.lead = (int)lead;
                sp.eps = (double)eps;
                sp.inv_m = 1.0 / (double)m;
                sp.entries = reinterpret_cast<unsigned long long *>(ws + kEntryOffset);
                sp.epoch = next_epoch(d);
                sp.tag_post = g_skew_next_flags.exchange(0) ? (sp.epoch ^ 0x40000000) : sp.epoch;
                sp.status = reinterpret_cast<int *>(ws);
                sp.wait_limit_ns = g_wait_limit_ns.load();
                st = launch_serialised_smem(layernorm_stream_kernel, dim3((unsigned)G), dim3(kLnStreamThreads),
                                            (size_t)kLnStreamSmem, stream, sp);
                if (st != CUDALLM_OK) return st;
            }
            return CUDALLM_OK;
        }
    }
    // first kernel: about four CTAs per SM in total (what is resident at once: one wave), at
    // least 4096 elements each, at most 256 parts
    int64_t parts = std::max<int64_t>(1, std::min<int64_t>(cdiv(int64_t(4) * sms, batch), m / 4096));
    parts = std::min<int64_t>(parts, 256);
    const int64_t part_len = round_up(cdiv(m, parts), 8);
    parts = cdiv(m, part_len);
    // second kernel: 8192 elements of each sample of a pair per CTA
    const int64_t chunk_len = 8192;
    const int64_t chunks = cdiv(m, chunk_len);
    const int64_t npairs = (batch + 1) / 2;
    if (batch * parts > kMaxDim || npairs * chunks > kMaxDim) return CUDALLM_ERR_INVALID_DIM;

    const size_t off_partials = kHeaderBytes;
    const size_t total = off_partials + (size_t)batch * (size_t)parts * 32;
    Workspace &w = workspace_for(d, stream);
    st = ensure_workspace(w, total, stream);
    if (st != CUDALLM_OK) return st;
    uint8_t *ws = static_cast<uint8_t *>(w.ptr);

    LayerNorm2Params lp{};
    lp.x = x; lp.gamma = gamma; lp.beta = beta; lp.y = y;
    lp.m = m; lp.part_len = part_len; lp.chunk_len = chunk_len;
    lp.batch = (int)batch; lp.parts = (int)parts; lp.chunks = (int)chunks;
    lp.eps = (double)eps;
    lp.inv_m = 1.0 / (double)m;
    lp.partials = reinterpret_cast<double *>(ws + off_partials);
    st = vec ? launch_serialised(layernorm_moments_kernel<true>, (unsigned)(batch * parts), kLn2Threads, stream, lp)
             : launch_serialised(layernorm_moments_kernel<false>, (unsigned)(batch * parts), kLn2Threads, stream, lp);
    if (st != CUDALLM_OK) return st;
    return vec ? launch_serialised(layernorm_apply_kernel<true>, (unsigned)(npairs * chunks), kLn2Threads, stream, lp)
               : launch_serialised(layernorm_apply_kernel<false>, (unsigned)(npairs * chunks), kLn2Threads, stream, lp);
}
