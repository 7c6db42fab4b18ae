// Task 2 with float32 operands read by the tensor cores as they lie in memory:
// tcgen05.mma.kind::tf32 takes the operands' float32 words and uses their sign,
// exponent and ten leading fraction bits; products are exact in, and accumulated
// in, float32.  The cheap sibling of the three-piece path (cudallm_gemm_f32): one
// pass over A and B, no conversion kernel, about three decimal digits per
// product instead of seven.
//
// Same skeleton as umma_gemm_kernel (a producer thread, an MMA thread, four
// epilogue warps, a ring of stages guarded by mbarriers, two accumulators in
// tensor memory, the same unit order and the same epilogue), with these
// differences in the operand path:
//  * a k-block is 32 float32 values (the 128 bytes of a swizzle row) deep;
//  * A (row-major M x K, K-major for the MMA): one TMA box of 32 x 128 per
//    k-block, as for bf16 in bytes;
//  * B (row-major K x N, MN-major for the MMA): a swizzle row holds 32 columns,
//    so a 256-column tile takes eight boxes of 32 columns x 32 k, 4 KiB apart
//    (the descriptor's leading-dimension offset).  32-bit operands that the
//    tensor core has to transpose must lie in the "128-byte swizzle on 32-byte
//    units" layout (the row's four 32-byte units exchanged by the row index
//    modulo 4, four-row groups 512 bytes apart: the stride-dimension offset):
//    TMA writes it (CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B), descriptor layout type
//    1 names it; with the 16-byte-unit swizzle of the other operands the
//    products come out as zeros.  One MMA (K = 8) reads 8 rows, 1 KiB, of each box;
//  * four MMAs of 128 x 256 x 8 per k-block.
// The loops are plain (a barrier round trip per 512-clock k-block); the fused
// probe-and-issue steps of the bf16 kernels were not needed to keep the tensor
// pipe the bound here.
#pragma once
#include "umma_gemm.cuh"
#include "umma_gemm_2cta.cuh"

namespace cudallm {

constexpr int kTf32BlockN = 256;
constexpr int kTf32BlockK = 32;
constexpr int kTf32Stages = 4;

struct Tf32Smem {
    static constexpr int kABytes = kBlockM * kTf32BlockK * 4;        // 16 KiB
    static constexpr int kBoxBytes = 32 * kTf32BlockK * 4;           // one box of B: 32 columns x 32 k
    static constexpr int kBBytes = (kTf32BlockN / 32) * kBoxBytes;   // 32 KiB
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kEpiOffset = kTf32Stages * kStageBytes;     // 1024-byte aligned (swizzled staging)
    static constexpr int kBarOffset = kEpiOffset + kEpiStageBytes;
    static constexpr int kNumBars = 2 * kTf32Stages + 4;             // full, empty, tmem_full[2], tmem_empty[2]
    static constexpr int kMiscOffset = kBarOffset + kNumBars * 8;
    static constexpr int kDynamicBytes = kMiscOffset + 64;
};

// Instruction descriptor for kind::tf32: fp32 accumulator, A K-major, B MN-major.
__host__ __device__ constexpr uint32_t make_idesc_tf32(int m, int n)
{
    return (1u << 4)                                  // D format: fp32
         | (2u << 7)                                  // A format: tf32
         | (2u << 10)                                 // B format: tf32
         | (0u << 15)                                 // A K-major
         | (1u << 16)                                 // B MN-major
         | (static_cast<uint32_t>(n >> 3) << 17)
         | (static_cast<uint32_t>(m >> 4) << 24);
}

// Shared-memory descriptor for the 128-byte swizzle on 32-byte units (layout type 1).
__device__ __forceinline__ uint64_t make_smem_desc_sw128_32b(uint32_t smem_addr, uint32_t lbo_bytes,
                                                             uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFF) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(1) << 61;
    return d;
}

__device__ __forceinline__ void tma_load_3d(uint32_t smem_dst, const CUtensorMap *tm, int x, int y, int z,
                                            uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
                 "[%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(z), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// D (tensor memory) = or += A x B, both operands in shared memory, K = 8.
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile("{\n\t"
                 ".reg .pred p;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t"
                 "}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__global__ void __launch_bounds__(kNumThreads, 1)
umma_tf32_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const __grid_constant__ CUtensorMap tmap_c, const GemmParams p)
{
    using L = Tf32Smem;
    constexpr uint32_t kTmemCols = 2 * kTf32BlockN;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = smem_raw;
    const uint32_t smem_base = smem_u32(smem);
    if (smem_base & 1023u) {
        if (threadIdx.x == 0) report_timeout(p.status, 0, 0x7F);
        return;
    }
    const uint32_t bar_base = smem_base + L::kBarOffset;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kTf32Stages + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * kTf32Stages + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * kTf32Stages + 2 + a); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + L::kMiscOffset);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L::kMiscOffset + 4);

    const int warp_idx = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kTf32Stages; ++s) {
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
        if (p.c_tma) prefetch_tensormap(&tmap_c);
    }
    if (warp_idx == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_launch_dependents();

    if (warp_idx == 0) {
        // ------------------------------------------------ TMA producer ----
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            grid_dependency_wait();
            for (int u = blockIdx.x; ok && u < p.num_units; u += gridDim.x) {
                const UnitCoord c = decode_unit(p, u);
                for (int kb = c.kb_begin; kb < c.kb_end; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1, abort_flag, p.wait_limit_ns)) {
                        report_timeout(p.status, kRoleProducer, stage);
                        ok = false;
                        break;
                    }
                    const uint32_t sa = smem_base + stage * L::kStageBytes, sb = sa + L::kABytes;
                    mbar_arrive_expect_tx(full_bar(stage), L::kStageBytes);
                    tma_load_3d(sa, &tmap_a, kb * kTf32BlockK, c.m_tile * kBlockM, c.b, full_bar(stage));
#pragma unroll
                    for (int j = 0; j < kTf32BlockN / 32; ++j)
                        tma_load_3d(sb + j * L::kBoxBytes, &tmap_b, c.n_tile * kTf32BlockN + 32 * j, kb * kTf32BlockK, c.b,
                                    full_bar(stage));
                    if (++stage == kTf32Stages) { stage = 0; phase ^= 1; }
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
            constexpr uint32_t idesc = make_idesc_tf32(kBlockM, kTf32BlockN);
            for (int u = blockIdx.x; ok && u < p.num_units; u += gridDim.x) {
                const UnitCoord c = decode_unit(p, u);
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1, abort_flag, p.wait_limit_ns)) {
                    report_timeout(p.status, kRoleMma, 0x40 + acc);
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kTf32BlockN;
                uint32_t accumulate = 0;
                for (int kb = c.kb_begin; kb < c.kb_end; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.wait_limit_ns)) {
                        report_timeout(p.status, kRoleMma, stage);
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = smem_base + stage * L::kStageBytes, sb = sa + L::kABytes;
                    // A: K-major, 8-row groups 1024 B apart (SBO); 8 K-elements = 32 B.
                    // B: MN-major, 32-column boxes 4096 B apart (LBO), 4-row groups 512 B apart
                    //    (SBO); 8 k = 1024 B.
#pragma unroll
                    for (int i = 0; i < kTf32BlockK / 8; ++i) {
                        umma_tf32(d_tmem, make_smem_desc_sw128(sa + 32 * i, 16, 1024),
                                  make_smem_desc_sw128_32b(sb + 1024 * i, L::kBoxBytes, 512), idesc, accumulate);
                        accumulate = 1;
                    }
                    umma_commit(empty_bar(stage));       // frees the stage when these MMAs retire
                    if (++stage == kTf32Stages) { stage = 0; phase ^= 1; }
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
        uint32_t sel = 0;
        const uint32_t stage_addr = smem_base + L::kEpiOffset + quad * kEpiWarpBytes;
        grid_dependency_wait();
        for (int u = blockIdx.x; u < p.num_units; u += gridDim.x) {
            const UnitCoord c = decode_unit(p, u);
            bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.wait_limit_ns);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                if (lane == 0) report_timeout(p.status, kRoleEpilogue, 0x80 + acc);
                break;
            }
            tc_fence_after();
            if (!epilogue_tile<kTf32BlockN, false>(p, c, c.m_tile * kBlockM + epi_tid,
                                                   tmem_base + acc * kTf32BlockN + (static_cast<uint32_t>(quad * 32) << 16),
                                                   quad, lane, 0, 1, abort_flag, &tmap_c, stage_addr, sel)) {
                if (lane == 0) report_timeout(p.status, kRoleEpilogue, 0xC0);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        if (lane == 0) bulk_wait_group_read<0>();        // shared memory must outlive the TMA stores
    }

    tc_fence_before();
    __syncthreads();
    if (warp_idx == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---------------------------------------------------------------------------
// The same product on CTA pairs (cta_group::2), as umma_gemm_2cta_kernel does it
// for bf16: a cluster of two CTAs owns a 256 x 256 tile, CTA r stages rows
// [128 r, 128 r + 128) of A and columns [128 r, 128 r + 128) of B (32 instead of
// 48 KiB per k-block and SM; three stages of two k-blocks each, so that producer and
// MMA thread pay one barrier round trip per 64 of K), the leader issues
// 256 x 256 x 8 MMAs for both, and the barriers are laid out as there (the
// leader's `full`, each CTA's `empty`, no multicast).
constexpr int kTf32PairStages = 3;
constexpr int kTf32PairSub = 2;                                       // k-blocks per stage: one barrier round trip per 64 of K

struct Tf32PairSmem {
    static constexpr int kABytes = kBlockM * kTf32BlockK * 4;        // 16 KiB: this CTA's 128 rows of A
    static constexpr int kBoxBytes = 32 * kTf32BlockK * 4;
    static constexpr int kBBytes = (kPairN / 2 / 32) * kBoxBytes;    // 16 KiB: this CTA's 128 columns of B
    static constexpr int kSubBytes = kABytes + kBBytes;              // one k-block
    static constexpr int kStageBytes = kTf32PairSub * kSubBytes;
    static constexpr int kEpiOffset = kTf32PairStages * kStageBytes;
    static constexpr int kBarOffset = kEpiOffset + kEpiStageBytes;
    static constexpr int kNumBars = 2 * kTf32PairStages + 4;
    static constexpr int kMiscOffset = kBarOffset + kNumBars * 8;
    static constexpr int kDynamicBytes = kMiscOffset + 64;
};

// TMA load whose bytes are counted on a barrier of the pair's leader (cluster address).
__device__ __forceinline__ void tma_load_3d_pair(uint32_t smem_dst, const CUtensorMap *tm, int x, int y, int z,
                                                 uint32_t bar_cluster_addr)
{
    asm volatile("cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
                 "[%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(z),
                   "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void umma_tf32_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile("{\n\t"
                 ".reg .pred p;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t"
                 "}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kNumThreads, 1)
umma_tf32_2cta_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                      const __grid_constant__ CUtensorMap tmap_c, const GemmParams p)
{
    using L = Tf32PairSmem;
    constexpr int STAGES = kTf32PairStages;
    constexpr uint32_t kTmemCols = 2 * kPairN;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = smem_raw;
    const uint32_t smem_base = smem_u32(smem);
    if (smem_base & 1023u) {                             // (the same in both CTAs of a pair)
        if (threadIdx.x == 0) report_timeout(p.status, 0, 0x7F);
        return;
    }
    const uint32_t bar_base = smem_base + L::kBarOffset;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + L::kMiscOffset);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L::kMiscOffset + 4);

    const int warp_idx = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                         // 0 = leader
    const int pair = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);       // leader's is used: one expect_tx arrival + both CTAs' bytes
            mbar_init(empty_bar(s), 1);      // one commit from the leader
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);      // one commit from the leader
            mbar_init(tempty_bar(a), 8);     // leader's is used: 4 epilogue warps x 2 CTAs
        }
        fence_mbar_init();
        fence_proxy_async_smem();
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
        if (p.c_tma) prefetch_tensormap(&tmap_c);
    }
    if (warp_idx == 1) {
        tmem_alloc_2cta(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
        tmem_relinquish_2cta();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();              // both CTAs' barriers exist before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_launch_dependents();

    if (warp_idx == 0) {
        // ------------------------------------------------ TMA producer ----
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            const uint32_t leader_full0 = map_to_cta(full_bar(0), 0);
            constexpr int half = kPairN / 2;             // columns of B this CTA stages
            grid_dependency_wait();
            for (int u = pair; ok && u < p.num_units; u += num_pairs) {
                const UnitCoord c = decode_unit(p, u);
                const int row0 = c.m_tile * kPairM + static_cast<int>(rank) * kBlockM;
                const int col0 = c.n_tile * kPairN + static_cast<int>(rank) * half;
                for (int kb = c.kb_begin; kb < c.kb_end; kb += kTf32PairSub) {
                    if (!mbar_wait<true>(empty_bar(stage), phase ^ 1, abort_flag, p.wait_limit_ns)) {
                        report_timeout(p.status, kRoleProducer, stage);
                        ok = false;
                        break;
                    }
                    const int nsub = min(kTf32PairSub, c.kb_end - kb);
                    const uint32_t bar = leader_full0 + 8u * stage;
                    if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * nsub * L::kSubBytes);
                    for (int sub = 0; sub < nsub; ++sub) {
                        const uint32_t sa = smem_base + stage * L::kStageBytes + sub * L::kSubBytes, sb = sa + L::kABytes;
                        const int k = (kb + sub) * kTf32BlockK;
                        tma_load_3d_pair(sa, &tmap_a, k, row0, c.b, bar);
#pragma unroll
                        for (int j = 0; j < half / 32; ++j)
                            tma_load_3d_pair(sb + j * L::kBoxBytes, &tmap_b, col0 + 32 * j, k, c.b, bar);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp_idx == 1) {
        // ------------------------------------- MMA issuer (leader only) ----
        if (lane == 0 && rank == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            constexpr uint32_t idesc = make_idesc_tf32(kPairM, kPairN);
            const uint32_t empty0_cta0 = map_to_cta(empty_bar(0), 0);
            const uint32_t empty0_cta1 = map_to_cta(empty_bar(0), 1);
            const uint32_t tfull0_cta0 = map_to_cta(tfull_bar(0), 0);
            const uint32_t tfull0_cta1 = map_to_cta(tfull_bar(0), 1);
            for (int u = pair; ok && u < p.num_units; u += num_pairs) {
                const UnitCoord c = decode_unit(p, u);
                if (!mbar_wait<true>(tempty_bar(acc), acc_phase ^ 1, abort_flag, p.wait_limit_ns)) {
                    report_timeout(p.status, kRoleMma, 0x40 + acc);
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kPairN;
                uint32_t accumulate = 0;
                for (int kb = c.kb_begin; kb < c.kb_end; kb += kTf32PairSub) {
                    if (!mbar_wait<true>(full_bar(stage), phase, abort_flag, p.wait_limit_ns)) {
                        report_timeout(p.status, kRoleMma, stage);
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const int nsub = min(kTf32PairSub, c.kb_end - kb);
                    for (int sub = 0; sub < nsub; ++sub) {
                        const uint32_t sa = smem_base + stage * L::kStageBytes + sub * L::kSubBytes, sb = sa + L::kABytes;
#pragma unroll
                        for (int i = 0; i < kTf32BlockK / 8; ++i) {
                            umma_tf32_pair(d_tmem, make_smem_desc_sw128(sa + 32 * i, 16, 1024),
                                           make_smem_desc_sw128_32b(sb + 1024 * i, L::kBoxBytes, 512), idesc, accumulate);
                            accumulate = 1;
                        }
                    }
                    umma_commit_pair(empty0_cta0 + 8u * stage);      // frees the stage in both CTAs
                    umma_commit_pair(empty0_cta1 + 8u * stage);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                umma_commit_pair(tfull0_cta0 + 8u * acc);
                umma_commit_pair(tfull0_cta1 + 8u * acc);
                if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else {
        // ---------------------------------------------------- epilogue ----
        const int quad = warp_idx & 3;
        const int epi_tid = quad * 32 + lane;
        int acc = 0;
        uint32_t acc_phase = 0;
        uint32_t sel = 0;
        const uint32_t stage_addr = smem_base + L::kEpiOffset + quad * kEpiWarpBytes;
        grid_dependency_wait();
        for (int u = pair; u < p.num_units; u += num_pairs) {
            const UnitCoord c = decode_unit(p, u);
            bool ok = mbar_wait<true>(tfull_bar(acc), acc_phase, abort_flag, p.wait_limit_ns);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                if (lane == 0) report_timeout(p.status, kRoleEpilogue, 0x80 + acc);
                break;
            }
            tc_fence_after();
            if (!epilogue_tile<kPairN, false>(p, c, c.m_tile * kPairM + static_cast<int>(rank) * kBlockM + epi_tid,
                                              tmem_base + acc * kPairN + (static_cast<uint32_t>(quad * 32) << 16),
                                              quad, lane, static_cast<int>(rank), 2, abort_flag, &tmap_c,
                                              stage_addr, sel)) {
                if (lane == 0) report_timeout(p.status, kRoleEpilogue, 0xC0);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(map_to_cta(tempty_bar(acc), 0));
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        if (lane == 0) bulk_wait_group_read<0>();
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();              // nobody leaves while the peer may still signal or read it
    if (warp_idx == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc_2cta(tmem_base, kTmemCols);
    }
}

}  // namespace cudallm
