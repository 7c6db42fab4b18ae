// tcgen05 GEMM with CTA pairs (cta_group::2): a cluster of two CTAs on two SMs
// owns one 256 x 256 tile of C.
//
//   C[i][j] = sum_k A[i][k] * B[k][j]      (Task 2: matrix multiplication)
//
// CTA r of the pair stages rows [128 r, 128 r + 128) of the tile's A panel and
// columns [128 r, 128 r + 128) of its B panel (32 KB per 64-deep k-block per
// CTA instead of 48 KB for a lone 128 x 256 tile, so six stages fit and the
// bytes that each SM must pull per MMA clock drop by a third).  The leader CTA
// (rank 0) issues one 256 x 256 x 16 MMA for both; each CTA's tensor core
// reads its own A rows and both halves of B, and accumulates its 128 rows x
// 256 columns in its own tensor memory.
//
// Synchronisation (no multicast anywhere):
//  * full[s]  lives in the leader.  Both producers' TMA loads complete their
//    bytes on it (the peer's through the cluster address of that barrier).
//  * empty[s] lives in each CTA; the leader commits the stage's MMAs to its
//    own and to the peer's barrier (two commits).
//  * tmem_full[a] likewise: one commit per CTA.
//  * tmem_empty[a] lives in the leader and counts the 8 epilogue warps of both
//    CTAs (the peer's arrive through the cluster address).
#pragma once
#include "umma_gemm.cuh"

namespace cudallm {

constexpr int kPairM = 256;
constexpr int kPairN = 256;

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;"
                 ::: "memory");
}
// address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void umma_commit_pair(uint32_t bar_cluster_addr)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar_cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];"
                 ::"r"(bar_cluster_addr) : "memory");
}

// A stage holds KSUB (1 or 2) 64-deep k-blocks, each [A 128 x 64 | B 64 x 128].
template <int STAGES, int KSUB>
struct PairSmemLayout {
    static constexpr int kABytes = kBlockM * kBlockK * 2;            // 128 rows of A
    static constexpr int kBBytes = kBlockK * (kPairN / 2) * 2;       // 128 columns of B
    static constexpr int kSubBytes = kABytes + kBBytes;              // 32 KB per k-block
    static constexpr int kStageBytes = KSUB * kSubBytes;
    static constexpr int kEpiOffset = STAGES * kStageBytes;          // 1024-byte aligned
    static constexpr int kBarOffset = kEpiOffset + kEpiStageBytes;
    static constexpr int kNumBars = 2 * STAGES + 4;
    static constexpr int kMiscOffset = kBarOffset + kNumBars * 8;
    static constexpr int kBytes = kMiscOffset + 64;
    static constexpr int kDynamicBytes = kBytes;         // the base is declared 1024-byte aligned
};

template <int STAGES, int KSUB, bool OUT_BF16>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kNumThreads, 1)
umma_gemm_2cta_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                      const __grid_constant__ CUtensorMap tmap_c, const GemmParams p)
{
    using L = PairSmemLayout<STAGES, KSUB>;
    constexpr uint32_t kTmemCols = 2 * kPairN;                       // 512: two accumulators

    // The swizzled stages need 1024-byte alignment in the shared window; the declaration asks
    // for it (no slack is reserved) and the kernel refuses to run without it.
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = smem_raw;
    const uint32_t smem_base = smem_u32(smem);
    if (smem_base & 1023u) {
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
            mbar_init(full_bar(s), 1);       // leader's is used: one expect_tx arrival + bytes
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
    // Each role waits for the previous kernel of the stream where it first touches global
    // memory (the producer just before its first load, the epilogue warps before their loop).

    if (warp_idx == 0) {
        // ------------------------------------------------ TMA producer ----
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            uint32_t tok = 1;                            // the first STAGES stages start out free
            bool waited = false;
            const uint32_t leader_full0 = map_to_cta(full_bar(0), 0);
            for (int u = pair; ok && u < p.num_units; u += num_pairs) {
                const UnitCoord c = decode_unit(p, u);
                constexpr int half = kPairN / 2;         // columns of B this CTA stages
                constexpr int boxes = half / 64;
                for (int kb = c.kb_begin; kb < c.kb_end; kb += KSUB) {
                    if (!tok && !mbar_wait<true>(empty_bar(stage), phase ^ 1, abort_flag, p.wait_limit_ns)) {
                        report_timeout(p.status, kRoleProducer, stage);
                        ok = false;
                        break;
                    }
                    // a stage takes up to KSUB k-blocks, all from the same operand segment
                    const KBlockCoord kc = kblock_coord(p, kb, c.b);
                    const int nsub = min(min(c.kb_end - kb, KSUB), kc.left_in_segment);
                    const int nstage = (stage + 1 == STAGES) ? 0 : stage + 1;
                    const uint32_t nphase = (stage + 1 == STAGES) ? phase ^ 1 : phase;
                    const uint32_t sa = smem_base + stage * L::kStageBytes;
                    if (!waited) {
                        grid_dependency_wait();
                        waited = true;
                    }
                    tok = tma_stage_step<true>(empty_bar(nstage), nphase ^ 1, full_bar(stage),
                                               rank == 0 ? 1u : 0u,
                                               2 * nsub * (L::kABytes + boxes * (64 * kBlockK * 2)),
                                               leader_full0 + 8u * stage, &tmap_a, &tmap_b, sa,
                                               sa + L::kABytes, kc.k,
                                               c.m_tile * kPairM + static_cast<int>(rank) * kBlockM,
                                               c.n_tile * kPairN + static_cast<int>(rank) * half, kc.batch_a,
                                               kc.batch_b, boxes, nsub, L::kSubBytes);
                    kb += nsub - KSUB;                   // the loop adds KSUB
                    stage = nstage;
                    phase = nphase;
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
            uint32_t tok = 0;                            // answer of the probe of full[stage]
            // cluster addresses of the barriers this thread signals in both CTAs
            const uint32_t empty0_cta0 = map_to_cta(empty_bar(0), 0);
            const uint32_t empty0_cta1 = map_to_cta(empty_bar(0), 1);
            const uint32_t tfull0_cta0 = map_to_cta(tfull_bar(0), 0);
            const uint32_t tfull0_cta1 = map_to_cta(tfull_bar(0), 1);
            for (int u = pair; ok && u < p.num_units; u += num_pairs) {
                const UnitCoord c = decode_unit(p, u);
                constexpr uint32_t idesc = make_idesc_bf16(kPairM, kPairN, 0, 1);
                if (!mbar_wait<true>(tempty_bar(acc), acc_phase ^ 1, abort_flag, p.wait_limit_ns)) {
                    report_timeout(p.status, kRoleMma, 0x40 + acc);
                    break;
                }
                const uint32_t d_tmem = tmem_base + acc * kPairN;
                bool first_of_unit = true;
                for (int kb = c.kb_begin; kb < c.kb_end; kb += KSUB) {
                    if (!tok && !mbar_wait<true>(full_bar(stage), phase, abort_flag, p.wait_limit_ns)) {
                        report_timeout(p.status, kRoleMma, stage);
                        ok = false;
                        break;
                    }
                    const int nsub = min(min(c.kb_end - kb, KSUB), kblock_coord(p, kb, c.b).left_in_segment);
                    const int nstage = (stage + 1 == STAGES) ? 0 : stage + 1;
                    const uint32_t nphase = (stage + 1 == STAGES) ? phase ^ 1 : phase;
                    const uint32_t sa = smem_base + stage * L::kStageBytes;
                    tok = umma_stage_step<true>(full_bar(nstage), nphase, d_tmem, idesc,
                                                first_of_unit ? 0u : 1u,
                                                make_smem_desc_sw128(sa, 16, 1024),
                                                make_smem_desc_sw128(sa + L::kABytes, 8192, 1024),
                                                L::kSubBytes, nsub, empty0_cta0 + 8u * stage,
                                                empty0_cta1 + 8u * stage);
                    first_of_unit = false;
                    kb += nsub - KSUB;                   // the loop adds KSUB
                    stage = nstage;
                    phase = nphase;
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
            if (!epilogue_tile<kPairN, OUT_BF16>(p, c, c.m_tile * kPairM + static_cast<int>(rank) * kBlockM + epi_tid,
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
