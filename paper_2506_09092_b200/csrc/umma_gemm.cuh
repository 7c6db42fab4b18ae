// Warp-specialised, persistent tcgen05 GEMM kernel for sm_100a.
//
//   C[i][j] = sum_k A[i][k] * B[k][j]      (Task 2: matrix multiplication)
//
// A is row-major M x K  -> K-major operand, TMA box 64(K) x 128(M), 128B swizzle.
// B is row-major K x N  -> MN-major operand, TMA boxes 64(N) x 64(K), 128B swizzle.
// One CTA owns a 128 x BLOCK_N tile of C; its fp32 accumulator lives in tensor
// memory (two buffers, so the epilogue of one tile overlaps the main loop of
// the next).  Roles: warp 0 = TMA producer, warp 1 = MMA issuer (and TMEM
// owner), warps 2..5 = epilogue (TMEM -> registers -> global).
//
// Work is cut into units (tile, k-split); CTA b runs units b, b+grid, ...
// With split_k > 1 every unit writes its fp32 partial sums to slice `split` of
// a workspace shaped [split][batch][M][ldp]; splitk_reduce_kernel then adds the
// slices in split order 0..S-1 (a fixed order, so results are reproducible)
// and writes C, rounding once.
#pragma once
#include "ptx.cuh"

namespace cudallm {

constexpr int kBlockM = 128;
constexpr int kBlockK = 64;           // one 128-byte swizzle row of bf16
constexpr int kUmmaK = 16;            // K of one tcgen05.mma for 16-bit inputs
constexpr int kNumThreads = 192;      // 6 warps
constexpr int kEpiThreads = 128;

// status detail codes: (role << 8) | barrier kind
enum : int { kRoleProducer = 1, kRoleMma = 2, kRoleEpilogue = 3 };

struct GemmParams {
    void *C;
    long long ldc;          // elements
    long long strideC;      // elements between batch items
    int M, N, K, batch;
    int tiles_m, tiles_n;   // tiles per batch item
    int split_k;            // >= 1, <= kblocks
    int kblocks;            // ceil(K / 64)
    int num_units;          // tiles_m * tiles_n * batch * split_k
    int c_vec_ok;           // C base, ldc, strideC allow 16-byte stores
    int a_box_bytes;        // bytes one TMA box of A delivers (box rows * 128)
    float *partials;        // split-K partial sums [split][batch][M][ldp] (workspace)
    long long ldp;          // row stride of the partial slices (multiple of 4)
    int *status;            // [0] = code, [1] = detail
};

template <int BLOCK_N, int STAGES>
struct SmemLayout {
    static constexpr int kABytes = kBlockM * kBlockK * 2;
    static constexpr int kBBytes = kBlockK * BLOCK_N * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kBarOffset = STAGES * kStageBytes;
    // full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]
    static constexpr int kNumBars = 2 * STAGES + 4;
    static constexpr int kMiscOffset = kBarOffset + kNumBars * 8;
    static constexpr int kBytes = kMiscOffset + 64;
    static constexpr int kDynamicBytes = kBytes + 1024;  // slack for 1024-byte alignment
};

__device__ __forceinline__ void report_timeout(int *status, int role, int what)
{
    if (atomicCAS(status, 0, -9 /* CUDALLM_ERR_DEVICE_TIMEOUT */) == 0)
        status[1] = (role << 8) | what;
}

struct UnitCoord {
    int m_tile, n_tile, b, split, tile_linear;
    int kb_begin, kb_end;
};

__device__ __forceinline__ UnitCoord decode_unit(const GemmParams &p, int u)
{
    UnitCoord c;
    c.split = u % p.split_k;
    int t = u / p.split_k;
    c.tile_linear = t;
    c.m_tile = t % p.tiles_m;
    t /= p.tiles_m;
    c.n_tile = t % p.tiles_n;
    c.b = t / p.tiles_n;
    c.kb_begin = static_cast<int>((static_cast<long long>(p.kblocks) * c.split) / p.split_k);
    c.kb_end = static_cast<int>((static_cast<long long>(p.kblocks) * (c.split + 1)) / p.split_k);
    return c;
}

// Store 32 consecutive fp32 accumulator values of one row, starting at column
// col0 of an n_cols-wide matrix, to `row_ptr + col0` (fp32 or bf16 elements).
template <bool OUT_BF16>
__device__ __forceinline__ void store_row_chunk(void *row_ptr, const float (&v)[32], int col0,
                                                int n_cols, bool vec_ok)
{
    const int n_left = n_cols - col0;
    if (n_left <= 0) return;
    if (OUT_BF16) {
        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(row_ptr) + col0;
        if (vec_ok && n_left >= 32) {
            uint4 *d4 = reinterpret_cast<uint4 *>(dst);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint4 w;
                w.x = pack_bf16x2(v[8 * q + 0], v[8 * q + 1]);
                w.y = pack_bf16x2(v[8 * q + 2], v[8 * q + 3]);
                w.z = pack_bf16x2(v[8 * q + 4], v[8 * q + 5]);
                w.w = pack_bf16x2(v[8 * q + 6], v[8 * q + 7]);
                d4[q] = w;
            }
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (j < n_left) dst[j] = __float2bfloat16_rn(v[j]);
        }
    } else {
        float *dst = reinterpret_cast<float *>(row_ptr) + col0;
        if (vec_ok && n_left >= 32) {
            float4 *d4 = reinterpret_cast<float4 *>(dst);
#pragma unroll
            for (int q = 0; q < 8; ++q)
                d4[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (j < n_left) dst[j] = v[j];
        }
    }
}

// Epilogue of one unit for one thread: `row` is this thread's row of C, `t_addr`
// the TMEM address of its lane at the accumulator's first column.  Reads the
// BLOCK_N accumulator columns 32 at a time and stores them to C (split_k == 1)
// or to this split's slice of the partial sums.  Must be called by whole warps.
template <int BLOCK_N, bool OUT_BF16>
__device__ __forceinline__ void epilogue_tile(const GemmParams &p, const UnitCoord &c, int row,
                                              uint32_t t_addr)
{
    const bool row_ok = row < p.M;
    void *row_ptr;
    bool vec_ok;
    if (p.split_k == 1) {
        const long long off = static_cast<long long>(c.b) * p.strideC
                            + static_cast<long long>(row) * p.ldc;
        row_ptr = OUT_BF16 ? static_cast<void *>(reinterpret_cast<__nv_bfloat16 *>(p.C) + off)
                           : static_cast<void *>(reinterpret_cast<float *>(p.C) + off);
        vec_ok = p.c_vec_ok != 0;
    } else {
        row_ptr = p.partials
                + ((static_cast<long long>(c.split) * p.batch + c.b) * p.M + row) * p.ldp;
        vec_ok = true;
    }
#pragma unroll 1
    for (int ch = 0; ch < BLOCK_N / 32; ++ch) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(t_addr + ch * 32, r);
        tmem_ld_wait();
        if (row_ok) {
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
            const int col0 = c.n_tile * BLOCK_N + ch * 32;
            if (p.split_k == 1) store_row_chunk<OUT_BF16>(row_ptr, v, col0, p.N, vec_ok);
            else                store_row_chunk<false>(row_ptr, v, col0, p.N, vec_ok);
        }
        __syncwarp();                                    // tcgen05.ld needs the whole warp
    }
}

template <int BLOCK_N, int STAGES, bool OUT_BF16>
__global__ void __launch_bounds__(kNumThreads, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a,
                 const __grid_constant__ CUtensorMap tmap_b, const GemmParams p)
{
    using L = SmemLayout<BLOCK_N, STAGES>;
    static_assert(BLOCK_N % 64 == 0 && BLOCK_N >= 64 && BLOCK_N <= 256, "BLOCK_N");
    constexpr uint32_t kTmemCols = 2 * BLOCK_N;          // 128, 256 or 512: power of two
    constexpr uint32_t kIdesc = make_idesc_bf16(kBlockM, BLOCK_N, 0, 1);

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_base + L::kBarOffset;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + L::kMiscOffset);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L::kMiscOffset + 4);

    const int warp_idx = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), 4);     // one arrival per epilogue warp
        }
        fence_mbar_init();
        fence_proxy_async_smem();
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
    }
    if (warp_idx == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp_idx == 0) {
        // ------------------------------------------------ TMA producer ----
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int u = blockIdx.x; ok && u < p.num_units; u += gridDim.x) {
                const UnitCoord c = decode_unit(p, u);
                for (int kb = c.kb_begin; kb < c.kb_end; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1, abort_flag)) {
                        report_timeout(p.status, kRoleProducer, stage);
                        ok = false;
                        break;
                    }
                    const uint32_t sa = smem_base + stage * L::kStageBytes;
                    const uint32_t sb = sa + L::kABytes;
                    mbar_arrive_expect_tx(full_bar(stage), p.a_box_bytes + L::kBBytes);
                    tma_load_3d(sa, &tmap_a, full_bar(stage), kb * kBlockK, c.m_tile * kBlockM, c.b);
#pragma unroll
                    for (int j = 0; j < BLOCK_N / 64; ++j)
                        tma_load_3d(sb + j * (64 * kBlockK * 2), &tmap_b, full_bar(stage),
                                    c.n_tile * BLOCK_N + j * 64, kb * kBlockK, c.b);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp_idx == 1) {
        // -------------------------------------------------- MMA issuer ----
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int u = blockIdx.x; ok && u < p.num_units; u += gridDim.x) {
                const UnitCoord c = decode_unit(p, u);
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1, abort_flag)) {
                    report_timeout(p.status, kRoleMma, 0x40 + acc);
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BLOCK_N;
                for (int kb = c.kb_begin; kb < c.kb_end; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag)) {
                        report_timeout(p.status, kRoleMma, stage);
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = smem_base + stage * L::kStageBytes;
                    const uint32_t sb = sa + L::kABytes;
#pragma unroll
                    for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                        // A: K-major, 8-row groups 1024 B apart; 16 K-elements = 32 B
                        const uint64_t da = make_smem_desc_sw128(sa + k * 32, 16, 1024);
                        // B: MN-major, 64-column chunks 8192 B apart (LBO),
                        //    8-k groups 1024 B apart (SBO); 16 k = 2048 B
                        const uint64_t db = make_smem_desc_sw128(sb + k * 2048, 8192, 1024);
                        umma_bf16(d_tmem, da, db, kIdesc, (kb > c.kb_begin || k > 0) ? 1u : 0u);
                    }
                    umma_commit(empty_bar(stage));       // frees the stage when the MMAs retire
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                umma_commit(tfull_bar(acc));             // accumulator complete
                if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else {
        // ---------------------------------------------------- epilogue ----
        const int quad = warp_idx & 3;                   // TMEM lanes 32*quad .. +31
        const int epi_tid = quad * 32 + lane;            // == row within the tile
        int acc = 0;
        uint32_t acc_phase = 0;
        for (int u = blockIdx.x; u < p.num_units; u += gridDim.x) {
            const UnitCoord c = decode_unit(p, u);
            bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                if (lane == 0) report_timeout(p.status, kRoleEpilogue, 0x80 + acc);
                break;
            }
            tc_fence_after();
            epilogue_tile<BLOCK_N, OUT_BF16>(p, c, c.m_tile * kBlockM + epi_tid,
                                             tmem_base + acc * BLOCK_N + (static_cast<uint32_t>(quad * 32) << 16));
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp_idx == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// Adds the S slices of split-K partial sums in order s = 0..S-1 and writes C
// (fp32, or bf16 rounded once).  One thread handles 4 consecutive columns.
template <bool OUT_BF16>
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float *__restrict__ partials, void *C, int M, int N, int batch, int split_k,
                     long long ldp, long long ldc, long long strideC, int c_vec4_ok)
{
    const int groups = (N + 3) >> 2;
    const long long rows = static_cast<long long>(batch) * M;
    const long long total = rows * groups;
    const long long slice = rows * ldp;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const long long br = i / groups;                 // b * M + row
        const int col = static_cast<int>(i - br * groups) * 4;
        const int b = static_cast<int>(br / M);
        const int row = static_cast<int>(br - static_cast<long long>(b) * M);
        const float *src = partials + br * ldp + col;
        float4 acc = __ldcg(reinterpret_cast<const float4 *>(src));
        for (int s = 1; s < split_k; ++s) {
            const float4 t = __ldcg(reinterpret_cast<const float4 *>(src + s * slice));
            acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
        }
        const long long off = b * strideC + row * ldc + col;
        const int n_left = N - col;
        if (OUT_BF16) {
            __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(C) + off;
            if (c_vec4_ok && n_left >= 4) {
                uint2 w;
                w.x = pack_bf16x2(acc.x, acc.y);
                w.y = pack_bf16x2(acc.z, acc.w);
                *reinterpret_cast<uint2 *>(dst) = w;
            } else {
                const float a[4] = {acc.x, acc.y, acc.z, acc.w};
                for (int j = 0; j < 4 && j < n_left; ++j) dst[j] = __float2bfloat16_rn(a[j]);
            }
        } else {
            float *dst = reinterpret_cast<float *>(C) + off;
            if (c_vec4_ok && n_left >= 4) {
                *reinterpret_cast<float4 *>(dst) = acc;
            } else {
                const float a[4] = {acc.x, acc.y, acc.z, acc.w};
                for (int j = 0; j < 4 && j < n_left; ++j) dst[j] = a[j];
            }
        }
    }
}

}  // namespace cudallm
