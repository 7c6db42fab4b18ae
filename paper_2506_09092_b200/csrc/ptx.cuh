// Inline-PTX wrappers for the sm_100a features the GEMM kernels use:
// mbarrier, TMA (cp.async.bulk.tensor), tcgen05 (alloc / mma / commit / ld).
// Every wait in here is bounded: it gives up after a wall-clock limit and
// reports failure to the caller, which records a status and leaves the kernel.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace cudallm {

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint64_t globaltimer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// ----------------------------------------- programmatic dependent launch --
// The GEMM kernels are launched with programmatic stream serialisation: their
// CTAs may start while the previous kernel of the stream is still running (as
// soon as SMs free up), set up barriers and tensor memory, and then wait here
// until every earlier kernel has completed and its writes are visible.  No
// global memory is touched before this wait.
__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
// Lets the next kernel of the stream start launching (it will wait as above).
__device__ __forceinline__ void grid_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ------------------------------------------------- asynchronous copies --
// 16 bytes global -> shared without passing through registers; only the first `src_bytes`
// (0 or 16) are read from global memory, the rest of the 16 is zero-filled.
__device__ __forceinline__ void cp_async_16(uint32_t smem_addr, const void *gptr, uint32_t src_bytes)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(smem_addr), "l"(gptr), "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.wait_all;" ::: "memory");
}

// ------------------------------------------------------- named barriers --
// Barrier `id` (1..15; 0 is __syncthreads) over `threads` threads of the CTA: whole
// warps either wait for all of them or only announce their arrival and go on.
__device__ __forceinline__ void named_bar_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void named_bar_arrive(int id, int threads)
{
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// ------------------------------------------------------------- mbarrier --
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Default wall-clock limit of every in-kernel wait.  Far above any legitimate
// wait (a whole GEMM takes well under a second), short enough that a logic
// error ends the kernel instead of hanging the device.  The GEMM kernels take
// their limit from a kernel parameter (this value unless the host changed it).
constexpr uint64_t kWaitLimitNs = 2000000000ull;

// Wait for phase `parity` of `bar`.  Returns false if `*abort_flag` becomes
// non-zero or `limit_ns` expires (then it also sets `*abort_flag`).
template <bool kCluster = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          uint64_t limit_ns = kWaitLimitNs)
{
    for (int i = 0; i < 128; ++i) {
        if (kCluster ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
    }
    const uint64_t t0 = globaltimer_ns();
    while (true) {
        for (int i = 0; i < 64; ++i) {
            if (kCluster ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity))
                return true;
        }
        if (*abort_flag) return false;
        if (globaltimer_ns() - t0 > limit_ns) {
            *abort_flag = 1;
            return false;
        }
    }
}

// ------------------------------------------------- shared-space ld / st --
// Explicit shared-space accesses (the staging pointers lose their address space
// on the way through the 1024-byte alignment arithmetic, and generic accesses
// to shared memory take the slower global path through the load/store unit).
__device__ __forceinline__ void st_shared_v4(uint32_t addr, float a, float b, float c, float d)
{
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}
__device__ __forceinline__ void st_shared_v4_b32(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d)
                 : "memory");
}
__device__ __forceinline__ float ld_shared_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
// ------------------------------------------------------------------ TMA --
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *tm)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tm)) : "memory");
}
// TMA store of one box from shared memory (bulk async-group completion).  The
// issuing thread commits the group and later waits until shared memory has
// been read (`bulk_wait_group_read`) before the block is overwritten.
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *tm, uint32_t smem_addr, int x, int y, int z)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(z), "r"(smem_addr) : "memory");
}
__device__ __forceinline__ void bulk_commit_group()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_group_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
// -------------------------------------------------------------- tcgen05 --
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(slot_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_alloc_2cta(uint32_t slot_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(slot_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_2cta()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_2cta(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tc_fence_before()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// Arrive once on `bar` when all tcgen05.mma issued so far by this thread finish.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread t gets lane (base_lane + t).
__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
          "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),
          "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}


// ------------------------------------------------- fused hot-loop steps --
// Any instruction whose result the issuing thread has to wait for (a barrier
// probe, even a plain shared-memory load) costs the MMA thread about 100 ns
// while the tensor core streams operands out of shared memory, on top of
// about 36 ns per tcgen05.mma it issues.  The hot loops therefore do ONE
// barrier round trip per stage and put as much work behind it as a stage
// holds (one or two 64-deep k-blocks); each step is a single asm block that
// probes the NEXT stage first, issues the current stage's work, and reads the
// probe's predicate last (through a branch, which cannot be hoisted).

// MMA step for one stage of `nsub` (1 or 2) 64-deep k-blocks: four K=16 MMAs
// per k-block, then the commit(s) that free the stage when they retire.
//   returns 1 if `next_bar` has completed phase `next_parity`.
//   first_acc: 0 -> the first MMA overwrites the accumulator.
//   da0 / db0: descriptors of the first k-block; the second one lies
//   `sub_bytes` further in shared memory.  commit_b is used by pairs only.
template <bool kPair>
__device__ __forceinline__ uint32_t umma_stage_step(uint32_t next_bar, uint32_t next_parity,
                                                    uint32_t d_tmem, uint32_t idesc, uint32_t first_acc,
                                                    uint64_t da0, uint64_t db0, uint32_t sub_bytes,
                                                    int nsub, uint32_t commit_a, uint32_t commit_b)
{
    uint32_t tok;
    const uint64_t sub = static_cast<uint64_t>(sub_bytes >> 4);
#define CUDALLM_MMA_STEP(GROUP, TESTW, TRYW, COMMIT2)                                              \
    asm volatile(                                                                                  \
        "{\n\t"                                                                                    \
        ".reg .pred pn, p0, pt, p2;\n\t"                                                           \
        ".reg .b64 a1, a2, a3, a4, a5, a6, a7, b1, b2, b3, b4, b5, b6, b7;\n\t"                    \
        TESTW " pn, [%1], %2;\n\t"                                                                 \
        "tcgen05.fence::after_thread_sync;\n\t"                                                    \
        "setp.ne.b32 p0, %5, 0;\n\t"                                                               \
        "setp.eq.b32 pt, %5, %5;\n\t"                                                              \
        "setp.gt.s32 p2, %9, 1;\n\t"                                                               \
        "add.u64 a1, %6, 2;\n\t add.u64 a2, %6, 4;\n\t add.u64 a3, %6, 6;\n\t"                   \
        "add.u64 b1, %7, 128;\n\t add.u64 b2, %7, 256;\n\t add.u64 b3, %7, 384;\n\t"             \
        "add.u64 a4, %6, %8;\n\t add.u64 a5, a1, %8;\n\t add.u64 a6, a2, %8;\n\t add.u64 a7, a3, %8;\n\t" \
        "add.u64 b4, %7, %8;\n\t add.u64 b5, b1, %8;\n\t add.u64 b6, b2, %8;\n\t add.u64 b7, b3, %8;\n\t" \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%3], %6, %7, %4, p0;\n\t"                     \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%3], a1, b1, %4, pt;\n\t"                     \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%3], a2, b2, %4, pt;\n\t"                     \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%3], a3, b3, %4, pt;\n\t"                     \
        "@p2 tcgen05.mma.cta_group::" GROUP ".kind::f16 [%3], a4, b4, %4, pt;\n\t"                 \
        "@p2 tcgen05.mma.cta_group::" GROUP ".kind::f16 [%3], a5, b5, %4, pt;\n\t"                 \
        "@p2 tcgen05.mma.cta_group::" GROUP ".kind::f16 [%3], a6, b6, %4, pt;\n\t"                 \
        "@p2 tcgen05.mma.cta_group::" GROUP ".kind::f16 [%3], a7, b7, %4, pt;\n\t"                 \
        "tcgen05.commit.cta_group::" GROUP ".mbarrier::arrive::one.shared::cluster.b64 [%10];\n\t" \
        COMMIT2                                                                                    \
        "@pn bra LDONE;\n\t"                                                                       \
        TRYW " pn, [%1], %2;\n\t"                                                                  \
        "LDONE:\n\t"                                                                               \
        "selp.u32 %0, 1, 0, pn;\n\t"                                                               \
        "}"                                                                                        \
        : "=r"(tok)                                                                                \
        : "r"(next_bar), "r"(next_parity), "r"(d_tmem), "r"(idesc), "r"(first_acc), "l"(da0),      \
          "l"(db0), "l"(sub), "r"(nsub), "r"(commit_a), "r"(commit_b)                              \
        : "memory")
    if (kPair) {
        CUDALLM_MMA_STEP("2", "mbarrier.test_wait.parity.acquire.cluster.shared::cta.b64",
                         "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64",
                         "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%11];\n\t");
    } else {
        CUDALLM_MMA_STEP("1", "mbarrier.test_wait.parity.shared::cta.b64",
                         "mbarrier.try_wait.parity.shared::cta.b64", "");
    }
#undef CUDALLM_MMA_STEP
    return tok;
}

// Producer step for one stage of `nsub` (1 or 2) k-blocks: arm `full_bar` with
// `tx_bytes` (if arm != 0); per k-block load one box of A and `boxes` boxes of
// B (64 columns wide, 8 KB apart in shared memory; up to 4 per k-block).  The second k-block's tiles lie
// `sub_bytes` after the first's.  Returns 1 if `next_bar` has completed phase
// `next_parity`.  `signal_bar` is where the loads complete their bytes (the
// leader's barrier for CTA pairs).
template <bool kPair>
__device__ __forceinline__ uint32_t tma_stage_step(uint32_t next_bar, uint32_t next_parity,
                                                   uint32_t full_bar, uint32_t arm, uint32_t tx_bytes,
                                                   uint32_t signal_bar, const CUtensorMap *tm_a,
                                                   const CUtensorMap *tm_b, uint32_t sa, uint32_t sb,
                                                   int k0, int row0, int col0, int batch_a, int batch_b,
                                                   int boxes, int nsub, uint32_t sub_bytes)
{
    uint32_t tok;
    const uint64_t ta = reinterpret_cast<uint64_t>(tm_a), tb = reinterpret_cast<uint64_t>(tm_b);
#define CUDALLM_TMA_STEP(TESTW, TRYW, LOAD)                                                        \
    asm volatile(                                                                                  \
        "{\n\t"                                                                                    \
        ".reg .pred pn, pa, p1, p2, p3, q0, q1, q2, q3;\n\t"                                       \
        ".reg .b32 c1, c2, c3, s1, s2, s3, k1, ta1, tb1, tb2, tb3, tb4;\n\t"                       \
        TESTW " pn, [%1], %2;\n\t"                                                                 \
        "setp.ne.b32 pa, %4, 0;\n\t"                                                               \
        "setp.gt.s32 p1, %15, 1;\n\t"                                                              \
        "setp.gt.s32 p2, %15, 2;\n\t"                                                              \
        "setp.gt.s32 p3, %15, 3;\n\t"                                                              \
        "setp.gt.s32 q0, %16, 1;\n\t"                                                              \
        "and.pred q1, q0, p1;\n\t"                                                                 \
        "and.pred q2, q0, p2;\n\t"                                                                 \
        "and.pred q3, q0, p3;\n\t"                                                                 \
        "add.s32 c1, %13, 64;\n\t add.s32 c2, %13, 128;\n\t add.s32 c3, %13, 192;\n\t"           \
        "add.u32 s1, %10, 8192;\n\t add.u32 s2, %10, 16384;\n\t add.u32 s3, %10, 24576;\n\t"     \
        "add.s32 k1, %11, 64;\n\t add.u32 ta1, %9, %17;\n\t add.u32 tb1, %10, %17;\n\t add.u32 tb2, s1, %17;\n\t" \
        "add.u32 tb3, s2, %17;\n\t add.u32 tb4, s3, %17;\n\t"                                    \
        "@pa mbarrier.arrive.expect_tx.shared::cta.b64 _, [%3], %5;\n\t"                           \
        LOAD " [%9], [%7, {%11, %12, %14}], [%6];\n\t"                                             \
        LOAD " [%10], [%8, {%13, %11, %18}], [%6];\n\t"                                            \
        "@p1 " LOAD " [s1], [%8, {c1, %11, %18}], [%6];\n\t"                                       \
        "@p2 " LOAD " [s2], [%8, {c2, %11, %18}], [%6];\n\t"                                       \
        "@p3 " LOAD " [s3], [%8, {c3, %11, %18}], [%6];\n\t"                                       \
        "@q0 " LOAD " [ta1], [%7, {k1, %12, %14}], [%6];\n\t"                                      \
        "@q0 " LOAD " [tb1], [%8, {%13, k1, %18}], [%6];\n\t"                                      \
        "@q1 " LOAD " [tb2], [%8, {c1, k1, %18}], [%6];\n\t"                                       \
        "@q2 " LOAD " [tb3], [%8, {c2, k1, %18}], [%6];\n\t"                                       \
        "@q3 " LOAD " [tb4], [%8, {c3, k1, %18}], [%6];\n\t"                                       \
        "@pn bra LDONE;\n\t"                                                                       \
        TRYW " pn, [%1], %2;\n\t"                                                                  \
        "LDONE:\n\t"                                                                               \
        "selp.u32 %0, 1, 0, pn;\n\t"                                                               \
        "}"                                                                                        \
        : "=r"(tok)                                                                                \
        : "r"(next_bar), "r"(next_parity), "r"(full_bar), "r"(arm), "r"(tx_bytes), "r"(signal_bar), \
          "l"(ta), "l"(tb), "r"(sa), "r"(sb), "r"(k0), "r"(row0), "r"(col0), "r"(batch_a), "r"(boxes), \
          "r"(nsub), "r"(sub_bytes), "r"(batch_b)                                                  \
        : "memory")
    if (kPair) {
        CUDALLM_TMA_STEP("mbarrier.test_wait.parity.acquire.cluster.shared::cta.b64",
                         "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64",
                         "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes");
    } else {
        CUDALLM_TMA_STEP("mbarrier.test_wait.parity.shared::cta.b64",
                         "mbarrier.try_wait.parity.shared::cta.b64",
                         "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes");
    }
#undef CUDALLM_TMA_STEP
    return tok;
}

// ---------------------------------------------------------- descriptors --
// Shared-memory matrix descriptor (64 bit): start address, leading-dimension
// byte offset and stride-dimension byte offset in 16-byte units, descriptor
// version 1 in bits [46,48), swizzle mode in bits [61,64) (2 = 128 bytes).
__device__ __forceinline__ uint64_t make_smem_desc_sw128(uint32_t smem_addr, uint32_t lbo_bytes,
                                                         uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFF) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}

// Instruction descriptor for kind::f16 with bf16 A and B, fp32 accumulator,
// A K-major, B MN-major (row-major K x N storage), shape M x N (K = 16).
__host__ __device__ constexpr uint32_t make_idesc_bf16(int m, int n, int a_mn_major, int b_mn_major)
{
    return (1u << 4)                                  // D format: fp32
         | (1u << 7)                                  // A format: bf16
         | (1u << 10)                                 // B format: bf16
         | (static_cast<uint32_t>(a_mn_major) << 15)
         | (static_cast<uint32_t>(b_mn_major) << 16)
         | (static_cast<uint32_t>(n >> 3) << 17)
         | (static_cast<uint32_t>(m >> 4) << 24);
}

// fp32 pair -> packed bf16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

}  // namespace cudallm
