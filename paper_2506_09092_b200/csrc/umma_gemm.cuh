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
// Work is cut into units; CTA b runs units b, b+grid, ... in that order.  The
// first dp_tiles tiles are one unit each.  Every later tile is cut along K into
// split_k units with consecutive indices (these units come first in the unit
// order, so their epilogues overlap later main loops), and its 32-column chunks are dealt
// round-robin to those units, two adjacent chunks at a time where the tile has at least two
// chunks per unit: unit j owns group q iff q mod split_k == j.  In
// its epilogue a unit first writes the chunks it does not own (its fp32 partial
// sums) to the workspace and raises a flag; then, for each chunk it owns, it
// waits for the other units' flags, adds the partial chunks in split order
// 0..S-1 -- a fixed order, so results are reproducible -- and stores C, rounding
// once.  The units of a tile thus exchange data among themselves; a unit never
// waits for a tile with a larger index, so the waits cannot form a cycle, and
// they are bounded like every other wait in the kernel.
// dp_tiles = 0 is plain split-K; dp_tiles = tiles - tiles % grid splits only the
// ragged last wave of a launch so that it takes about 1/split_k of a tile's time.
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

// Division of a 32-bit unsigned number by a divisor fixed on the host (1 <= d <
// 2^31): q = (t + ((n - t) >> sh1)) >> sh2 with t = the high half of mul * n
// (the round-up method for invariant divisors).  Exact for every 32-bit n.
struct FastDiv {
    uint32_t mul;
    uint16_t sh1, sh2;
};
__device__ __forceinline__ uint32_t fast_div(uint32_t n, FastDiv d)
{
    const uint32_t t = __umulhi(d.mul, n);
    return (t + ((n - t) >> d.sh1)) >> d.sh2;
}
inline FastDiv make_fast_div(uint32_t d)
{
    int l = 0;
    while ((1ull << l) < d) ++l;                         // l = ceil(log2 d)
    FastDiv f;
    f.mul = static_cast<uint32_t>((((1ull << 32) * ((1ull << l) - d)) / d) + 1);
    f.sh1 = static_cast<uint16_t>(l < 1 ? l : 1);
    f.sh2 = static_cast<uint16_t>(l ? l - 1 : 0);
    return f;
}

struct GemmParams {
    void *C;
    long long ldc;          // elements
    long long strideC;      // elements between batch items
    int M, N, K, batch;
    int tiles_m, tiles_n;   // tiles per batch item
    int group_m;            // tile rows per raster group (see decode_unit)
    int kblocks;            // 64-deep k-blocks each unit range is cut from: ceil(K / 64), or 6x that
    int piece_kblocks;      // 0, or k-blocks per operand-piece pair (see KBlockCoord)
    int dp_tiles;           // leading tiles that are not split
    int split_k;            // K parts per tile for tiles >= dp_tiles (1 = none), <= kblocks
    int num_units;          // dp_tiles + (tiles - dp_tiles) * split_k
    int c_tma;              // C base, ldc and strideC are 16-byte aligned: the epilogue stores by TMA
    int n_edge_tma;         // ... including the box that straddles column N (N * element size % 16 == 0)
    int a_box_bytes;        // bytes one TMA box of A delivers (box rows * 128)
    int epoch;              // value that marks a flag as raised in this launch (never 0)
    int flag_post;          // value a unit raises its flags to: epoch (anything else only in the host's
                            // self-test of the timeout path, where no wait may ever be satisfied)
    unsigned long long wait_limit_ns;   // wall-clock limit of every bounded wait in the kernel
    float *partials;        // partial tiles of split units (workspace), 128 x BLOCK_N fp32 each
    int *flags;             // one per (partial tile, epilogue warp) (workspace)
    int *status;            // [0] = code, [1] = detail
    // divisors of decode_unit: split_k, tiles per item, tiles per raster group,
    // group_m, and the height of the last (possibly shorter) raster group
    FastDiv div_split, div_item, div_group, div_gm, div_gm_last;
};

// Epilogue staging: 8 KiB per epilogue warp, 1024-byte aligned -- two 4 KiB
// blocks of 32 rows x 128 bytes that TMA stores read in turn, or one block of
// 32 rows x 36 floats for the element-wise path of unaligned C.
constexpr int kEpiPitch = 36;
constexpr int kEpiWarpBytes = 8192;
constexpr int kEpiStageBytes = 4 * kEpiWarpBytes;
static_assert(32 * kEpiPitch * 4 <= kEpiWarpBytes, "element-wise staging block");

// A stage holds KSUB (1 or 2) 64-deep k-blocks, each [A A_ROWS x 64 | B 64 x BLOCK_N]: with
// two, the producer and the MMA thread pay one barrier round trip per 128 of K.
// A_ROWS < 128 is for products with M <= A_ROWS: the TMA box of A then has at most
// A_ROWS rows, and the shared memory saved buys more stages, i.e. more bytes of B in
// flight per SM, which is what bounds a short, wide product.  The MMA still reads
// 128 rows: rows >= A_ROWS are whatever follows in the stage (B's data), and the rows of
// the accumulator they produce are never stored.
template <int BLOCK_N, int STAGES, int KSUB = 1, int A_ROWS = kBlockM>
struct SmemLayout {
    static_assert(A_ROWS % 8 == 0 && A_ROWS >= 8 && A_ROWS <= kBlockM, "rows of A per stage");
    static_assert(A_ROWS * kBlockK * 2 + kBlockK * BLOCK_N * 2 >= kBlockM * kBlockK * 2,
                  "the 128 rows the MMA reads must lie inside the k-block's own bytes");
    static constexpr int kABytes = A_ROWS * kBlockK * 2;
    static constexpr int kBBytes = kBlockK * BLOCK_N * 2;
    static constexpr int kSubBytes = kABytes + kBBytes;
    static constexpr int kStageBytes = KSUB * kSubBytes;
    static constexpr int kEpiOffset = STAGES * kStageBytes;          // 1024-byte aligned (swizzled staging)
    static constexpr int kBarOffset = kEpiOffset + kEpiStageBytes;
    // full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]
    static constexpr int kNumBars = 2 * STAGES + 4;
    static constexpr int kMiscOffset = kBarOffset + kNumBars * 8;
    static constexpr int kBytes = kMiscOffset + 64;
    static constexpr int kDynamicBytes = kBytes;         // the base is declared 1024-byte aligned
};

__device__ __forceinline__ void report_timeout(int *status, int role, int what)
{
    if (atomicCAS(status, 0, -9 /* CUDALLM_ERR_DEVICE_TIMEOUT */) == 0)
        status[1] = (role << 8) | what;
}

struct UnitCoord {
    int m_tile, n_tile, b;
    int split, nsplit;      // this unit's part of K and how many parts its tile has
    int slot0;              // (tile - dp_tiles) * split_k: partial-tile index of this tile's split 0
    int kb_begin, kb_end;
};

__device__ __forceinline__ UnitCoord decode_unit(const GemmParams &p, int u)
{
    UnitCoord c;
    int t;
    // Split units come FIRST in the unit order (their tiles are the last
    // tiles - dp_tiles ones): the exchange of partial sums in their epilogue
    // then overlaps with the main loops of the unsplit tiles that follow.
    const int split_units = p.num_units - p.dp_tiles;
    if (u >= split_units) {
        t = u - split_units;
        c.split = 0;
        c.nsplit = 1;
        c.slot0 = 0;
        c.kb_begin = 0;
        c.kb_end = p.kblocks;
    } else {
        const int ts = static_cast<int>(fast_div(u, p.div_split));
        t = p.dp_tiles + ts;
        c.split = u - ts * p.split_k;
        c.nsplit = p.split_k;
        c.slot0 = ts * p.split_k;
        // kblocks * split_k < 2^32 (kblocks < 6 * 2^25, split_k <= 16)
        const uint32_t lo = static_cast<uint32_t>(p.kblocks) * static_cast<uint32_t>(c.split);
        c.kb_begin = static_cast<int>(fast_div(lo, p.div_split));
        c.kb_end = static_cast<int>(fast_div(lo + static_cast<uint32_t>(p.kblocks), p.div_split));
    }
    // Raster order inside a batch item: groups of group_m tile rows; inside a
    // group the row index runs fastest, then the column.  The CTAs that run at
    // the same time then share one slice of A (group_m tile rows, sized by the
    // host to stay in L2) and a few column panels of B.
    const int per_item = p.tiles_m * p.tiles_n;
    c.b = static_cast<int>(fast_div(t, p.div_item));
    const int r = t - c.b * per_item;
    const int g = static_cast<int>(fast_div(r, p.div_group));
    const int r2 = r - g * p.group_m * p.tiles_n;
    const bool last = (g + 1) * p.group_m > p.tiles_m;   // the shorter group at the bottom
    const int gm = last ? p.tiles_m - g * p.group_m : p.group_m;
    c.n_tile = static_cast<int>(fast_div(r2, last ? p.div_gm_last : p.div_gm));
    c.m_tile = g * p.group_m + (r2 - c.n_tile * gm);
    return c;
}

// Where k-block g of a unit's range lies in the operands.  Normally that is
// column block g of A / row block g of B of batch item b.  In three-piece mode
// (piece_kblocks > 0) the operands are fp32 values cut into three bf16 pieces
// each, stored as "batch" items 0..2 of the tensor maps, and the K range is six
// segments long: segment s multiplies piece kPieceA[s] of A with piece
// kPieceB[s] of B (the six products of magnitude >= 2^-16 of the leading one,
// smallest first so that they are not absorbed by the large ones too early).
struct KBlockCoord {
    int k;                  // first K index of the block
    int batch_a, batch_b;   // third tensor-map coordinate for the A and the B load
    int left_in_segment;    // k-blocks from g to the end of its segment (>= 1)
};
__device__ __forceinline__ KBlockCoord kblock_coord(const GemmParams &p, int g, int b)
{
    KBlockCoord c;
    if (p.piece_kblocks == 0) {
        c.k = g * kBlockK;
        c.batch_a = c.batch_b = b;
        c.left_in_segment = p.kblocks - g;
    } else {
        const int seg = g / p.piece_kblocks;
        const int kb = g - seg * p.piece_kblocks;
        c.k = kb * kBlockK;
        // segments: a3*b1, a1*b3, a2*b2, a2*b1, a1*b2, a1*b1
        c.batch_a = (0x001102 >> (4 * seg)) & 0xF;
        c.batch_b = (0x010120 >> (4 * seg)) & 0xF;
        c.left_in_segment = p.piece_kblocks - kb;
    }
    return c;
}

__device__ __forceinline__ int ld_acquire_gpu(const int *p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_gpu(int *p, int v)
{
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded wait until *flag == epoch.
__device__ __forceinline__ bool wait_flag(const int *flag, int epoch, volatile int *abort_flag,
                                          uint64_t limit_ns)
{
    if (ld_acquire_gpu(flag) == epoch) return true;
    const uint64_t t0 = globaltimer_ns();
    while (true) {
        for (int i = 0; i < 16; ++i) {
            if (ld_acquire_gpu(flag) == epoch) return true;
            __nanosleep(100);
        }
        if (*abort_flag) return false;
        if (globaltimer_ns() - t0 > limit_ns) {
            *abort_flag = 1;
            return false;
        }
    }
}

// One thread's row of a 32-column block -> staging block `blk`, in the swizzled layout
// that store_block_staged describes.
template <bool OUT_BF16>
__device__ __forceinline__ void stage_row_swizzled(uint32_t blk, int lane, const float (&v)[32])
{
    if (OUT_BF16) {
        const uint32_t row = blk + lane * 64;
        const uint32_t x = (lane >> 1) & 3;
#pragma unroll
        for (int q = 0; q < 4; ++q)
            st_shared_v4_b32(row + ((q ^ x) << 4), pack_bf16x2(v[8 * q], v[8 * q + 1]),
                             pack_bf16x2(v[8 * q + 2], v[8 * q + 3]), pack_bf16x2(v[8 * q + 4], v[8 * q + 5]),
                             pack_bf16x2(v[8 * q + 6], v[8 * q + 7]));
    } else {
        const uint32_t row = blk + lane * 128;
        const uint32_t x = lane & 7;
#pragma unroll
        for (int q = 0; q < 8; ++q)
            st_shared_v4(row + ((q ^ x) << 4), v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
    }
}

// One thread's row of 32 floats -> its row of a staging block (36 floats per row), moved
// right by A elements: position A + i holds v[i], so that the 16-byte pieces of the row
// in shared memory are the 16-byte-aligned pieces of the row in a C whose element (row, col0)
// lies A elements behind a 16-byte boundary.  (Positions outside A .. A + 31 get zeros that
// nobody stores.)
template <int A>
__device__ __forceinline__ void stage_row_shifted(uint32_t row_addr, const float (&v)[32])
{
#pragma unroll
    for (int q = 0; q < (A ? 9 : 8); ++q) {
        float w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = 4 * q + j - A;
            w[j] = (i >= 0 && i < 32) ? v[i < 0 ? 0 : (i > 31 ? 31 : i)] : 0.f;
        }
        st_shared_v4(row_addr + 16 * q, w[0], w[1], w[2], w[3]);
    }
}

// Stores one 32 x 32 block of the accumulator (this warp's 32 rows, 32
// consecutive columns from col0) to C.  Each thread arrives with the 32 values
// of ITS row (v); writing them as they are would make every store instruction
// touch 32 different rows, so the block goes through shared memory.
//  * C aligned for TMA (p.c_tma): every thread writes its row (128 bytes of
//    fp32, 64 bytes of bf16) into one of the warp's two staging blocks in the
//    tensor map's swizzled layout -- 16-byte piece q of row r lies at piece
//    q ^ (r % 8) (128-byte rows) or q ^ ((r / 2) % 4) (64-byte rows), which
//    keeps the 16-byte stores of a quarter-warp on distinct banks -- and lane 0
//    issues one TMA store of the box; the hardware clips it at M and N.  The
//    block is reused two stores later, after lane 0 has waited for the older
//    store to have read it.  The clipping works in units of 16 bytes (measured:
//    with N = 127 column 127 is written), so a box that straddles an N whose
//    row length is not a multiple of 16 bytes takes the other path.
//  * fp32 C that TMA cannot address (rows only 4-byte aligned), block inside N: the
//    thread writes its row moved right by the row's own misalignment (0 to 3
//    elements), so that the 16-byte pieces of the staged row are the 16-byte-aligned
//    pieces of the row of C; those go out in 16-byte stores, four rows per
//    instruction, and the up to three elements before and after them in element
//    stores, eight rows per instruction (12 store instructions per block, not 32).
//  * otherwise (bf16 C, or the block that straddles column N): rows 36 floats apart,
//    read back one row per instruction and written with element stores that are
//    contiguous per row.
// `stage` = shared-memory address of the warp's 8 KiB; `sel` alternates between
// its two blocks; row0 = global row of lane 0; b = batch item.
template <bool OUT_BF16>
__device__ __forceinline__ void store_block_staged(const GemmParams &p, const CUtensorMap *tmap_c,
                                                   uint32_t stage, uint32_t &sel, const float (&v)[32],
                                                   int b, int row0, int col0, int lane)
{
    if (p.c_tma && (col0 + 32 <= p.N || p.n_edge_tma)) {
        const uint32_t blk = stage + sel * 4096u;
        sel ^= 1u;
        if (lane == 0) bulk_wait_group_read<1>();        // the store before the last one has read `blk`
        __syncwarp();
        stage_row_swizzled<OUT_BF16>(blk, lane, v);
        fence_proxy_async_smem();                        // generic-proxy writes -> visible to the TMA unit
        __syncwarp();
        if (lane == 0) {
            tma_store_3d(tmap_c, blk, col0, row0, b);
            bulk_commit_group();
        }
        return;
    }
    if (p.c_tma) {                                       // earlier TMA stores may still read the staging blocks
        if (lane == 0) bulk_wait_group_read<0>();
        __syncwarp();
    }
    if (!OUT_BF16 && col0 + 32 <= p.N) {
        // fp32 rows that are only 4-byte aligned: each row's 16-byte-aligned body goes out in
        // 16-byte stores (four rows per instruction), the up to three elements before and
        // after it in element stores (eight rows per instruction).
        const long long e0 = static_cast<long long>(reinterpret_cast<uintptr_t>(p.C) >> 2)
                           + static_cast<long long>(b) * p.strideC + static_cast<long long>(row0) * p.ldc + col0;
        const uint32_t my_row = stage + lane * (kEpiPitch * 4);
        switch (static_cast<int>((e0 + lane * p.ldc) & 3)) {
        case 0:  stage_row_shifted<0>(my_row, v); break;
        case 1:  stage_row_shifted<1>(my_row, v); break;
        case 2:  stage_row_shifted<2>(my_row, v); break;
        default: stage_row_shifted<3>(my_row, v); break;
        }
        __syncwarp();
        const int rows = min(32, p.M - row0);
        float *c0 = reinterpret_cast<float *>(p.C) + (static_cast<long long>(b) * p.strideC
                                                      + static_cast<long long>(row0) * p.ldc + col0);
        float4 body[8];
        float edge[4];
#pragma unroll
        for (int g = 0; g < 8; ++g) {                    // rows 4g .. 4g + 3, lane k of a row: piece k (+ 1)
            const int r = 4 * g + (lane >> 3);
            const int a = static_cast<int>((e0 + r * p.ldc) & 3);
            const int piece = (lane & 7) + (a ? 1 : 0);
            const uint32_t src = stage + (r * kEpiPitch + 4 * piece) * 4;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                         : "=f"(body[g].x), "=f"(body[g].y), "=f"(body[g].z), "=f"(body[g].w) : "r"(src) : "memory");
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {                    // rows 8g .. 8g + 7, lane e of a row: its e-th edge element
            const int r = 8 * g + (lane >> 2), e = lane & 3;
            const int a = static_cast<int>((e0 + r * p.ldc) & 3);
            edge[g] = ld_shared_f32(stage + (r * kEpiPitch + (e >= a ? e : 32 + e)) * 4);
        }
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            const int r = 4 * g + (lane >> 3);
            const int a = static_cast<int>((e0 + r * p.ldc) & 3);
            const int piece = (lane & 7) + (a ? 1 : 0);
            if (r < rows && piece < 8)
                *reinterpret_cast<float4 *>(c0 + r * p.ldc - a + 4 * piece) = body[g];
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const int r = 8 * g + (lane >> 2), e = lane & 3;
            const int a = static_cast<int>((e0 + r * p.ldc) & 3);
            if (r < rows && a) c0[r * p.ldc - a + (e >= a ? e : 32 + e)] = edge[g];
        }
        __syncwarp();                                    // the block is reused for the next chunk
        return;
    }
#pragma unroll
    for (int q = 0; q < 8; ++q)
        st_shared_v4(stage + (lane * kEpiPitch + 4 * q) * 4, v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
    __syncwarp();
    const int rows = min(32, p.M - row0);                // > 0 for at least lane 0's row by construction
    const bool col_ok = col0 + lane < p.N;
    const long long off0 = static_cast<long long>(b) * p.strideC + static_cast<long long>(row0) * p.ldc + col0 + lane;
#pragma unroll
    for (int r0 = 0; r0 < 32; r0 += 8) {
        float x[8];                                      // reads first: C may alias nothing, but the compiler cannot tell
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = ld_shared_f32(stage + ((r0 + i) * kEpiPitch + lane) * 4);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (r0 + i < rows && col_ok) {
                const long long off = off0 + static_cast<long long>(r0 + i) * p.ldc;
                if (OUT_BF16) reinterpret_cast<__nv_bfloat16 *>(p.C)[off] = __float2bfloat16_rn(x[i]);
                else          reinterpret_cast<float *>(p.C)[off] = x[i];
            }
        }
    }
    __syncwarp();                                        // the block is reused for the next chunk
}

// Two adjacent 32-column blocks (columns col0 .. col0 + 63) at once, both by TMA: the
// same steps as two calls of store_block_staged, but with one wait for the staging
// blocks, one proxy fence and one warp barrier, whose latencies (about 600 clocks per
// block in all) are what an epilogue that is not hidden behind a main loop consists of.
template <bool OUT_BF16>
__device__ __forceinline__ void store_two_blocks_staged(const CUtensorMap *tmap_c, uint32_t stage, uint32_t sel,
                                                        const float (&va)[32], const float (&vb)[32], int b,
                                                        int row0, int col0, int lane)
{
    const uint32_t blk_a = stage + sel * 4096u, blk_b = stage + (sel ^ 1u) * 4096u;
    if (lane == 0) bulk_wait_group_read<0>();            // both staging blocks have been read
    __syncwarp();
    stage_row_swizzled<OUT_BF16>(blk_a, lane, va);
    stage_row_swizzled<OUT_BF16>(blk_b, lane, vb);
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
        tma_store_3d(tmap_c, blk_a, col0, row0, b);
        bulk_commit_group();                             // a group each, as store_block_staged counts them
        tma_store_3d(tmap_c, blk_b, col0 + 32, row0, b);
        bulk_commit_group();
    }
}

// Epilogue of one unit, called by the four epilogue warps.  `row` is this
// thread's row of C, `t_addr` the TMEM address of its lane at the accumulator's
// first column, `quad`/`lane` identify the thread (row within the tile =
// 32*quad + lane), `cta_slot` = index of this CTA among the CTAs that share a
// tile (0 for lone CTAs, the cluster rank for pairs) and `ctas_per_tile` their
// number.  Works on the BLOCK_N accumulator columns 32 at a time (a "chunk").
// Partial tile layout: float4 index ((chunk*8 + q) * 128 + row_in_tile), so
// that a warp writes and reads 512 contiguous bytes.  Returns false if a wait
// for another unit's flag ran out.
template <int BLOCK_N, bool OUT_BF16>
__device__ __forceinline__ bool epilogue_tile(const GemmParams &p, const UnitCoord &c, int row,
                                              uint32_t t_addr, int quad, int lane, int cta_slot,
                                              int ctas_per_tile, volatile int *abort_flag,
                                              const CUtensorMap *tmap_c, uint32_t stage, uint32_t &sel)
{
    constexpr int kTileF4 = kBlockM * BLOCK_N / 4;
    constexpr int kChunks = BLOCK_N / 32;
    const bool row_ok = row < p.M;
    const int row_in_tile = quad * 32 + lane;
    const int S = c.nsplit;
    bool ok = true;

    if (S > 1) {
        // Ownership goes by groups of two adjacent chunks where the tile has at least two
        // chunks per unit (unit j owns group q iff q mod S == j), else by single chunks: an
        // owner then fetches both chunks' partial sums in one round trip and stores 64 columns.
        const int g = (kChunks >= 2 * S) ? 2 : 1;
        // 1. hand the chunks other units own to them
        const long long my_slot = static_cast<long long>(c.slot0 + c.split) * ctas_per_tile + cta_slot;
        float4 *mine = reinterpret_cast<float4 *>(p.partials) + my_slot * kTileF4;
#pragma unroll 1
        for (int ch = 0; ch < kChunks; ++ch) {
            if ((ch / g) % S == c.split) continue;
            uint32_t r[32];
            tmem_ld_32x32b_x32(t_addr + ch * 32, r);
            tmem_ld_wait();
            if (row_ok) {
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    __stcg(mine + (ch * 8 + q) * kBlockM + row_in_tile,
                           make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]),
                                       __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3])));
            }
            __syncwarp();                                // tcgen05.ld needs the whole warp
        }
        // The warp barrier orders every lane's partial sums before lane 0's release store,
        // whose fence is cumulative over them (the order a grid-wide barrier relies on too):
        // one fence per warp instead of one per lane plus the store's own.
        __syncwarp();
        if (lane == 0) st_release_gpu(p.flags + my_slot * 4 + quad, p.flag_post);
        if (c.split * g >= kChunks) return true;         // this unit owns no chunk
        // 2. the same epilogue warp of every other unit wrote the rows this warp needs
        for (int s = 0; s < S; ++s) {
            if (s == c.split) continue;
            const long long slot = static_cast<long long>(c.slot0 + s) * ctas_per_tile + cta_slot;
            ok = wait_flag(p.flags + slot * 4 + quad, p.epoch, abort_flag, p.wait_limit_ns) && ok;
        }
        ok = __all_sync(0xffffffffu, ok);          // (every lane polled with acquire loads itself)

        const int row0 = row - lane;                     // global row of this warp's lane 0
        if (row0 >= p.M) return ok;                      // the whole warp is below the matrix
        const float4 *tile0 = reinterpret_cast<const float4 *>(p.partials)
                            + (static_cast<long long>(c.slot0) * ctas_per_tile + cta_slot) * kTileF4;
        // 3. the groups this unit owns: sum over the units in index order (this unit's own
        //    term comes from TMEM), round once, store
#pragma unroll 1
        for (int grp = c.split; grp * g < kChunks; grp += S) {
            const int ch = grp * g;
            const int col0 = c.n_tile * BLOCK_N + ch * 32;
            if (col0 >= p.N) break;                      // warp-uniform: nothing further to store
            const bool two = g == 2 && col0 + 32 < p.N;
            uint32_t ra[32], rb[32];
            tmem_ld_32x32b_x32(t_addr + ch * 32, ra);
            if (two) tmem_ld_32x32b_x32(t_addr + ch * 32 + 32, rb);
            tmem_ld_wait();
            float va[32], vb[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) va[j] = vb[j] = 0.f;
            for (int s = 0; s < S; ++s) {
                if (s == c.split) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        va[j] += __uint_as_float(ra[j]);
                        if (two) vb[j] += __uint_as_float(rb[j]);
                    }
                } else if (row_ok) {
                    const float4 *part = tile0 + static_cast<long long>(s) * ctas_per_tile * kTileF4
                                       + (ch * 8) * kBlockM + row_in_tile;
                    float4 ta[8], tb[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) ta[q] = __ldcg(part + q * kBlockM);
                    if (two) {
#pragma unroll
                        for (int q = 0; q < 8; ++q) tb[q] = __ldcg(part + (8 + q) * kBlockM);
                    }
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        va[4 * q] += ta[q].x; va[4 * q + 1] += ta[q].y;
                        va[4 * q + 2] += ta[q].z; va[4 * q + 3] += ta[q].w;
                    }
                    if (two) {
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            vb[4 * q] += tb[q].x; vb[4 * q + 1] += tb[q].y;
                            vb[4 * q + 2] += tb[q].z; vb[4 * q + 3] += tb[q].w;
                        }
                    }
                }
            }
            if (two && p.c_tma && (col0 + 64 <= p.N || p.n_edge_tma)) {
                store_two_blocks_staged<OUT_BF16>(tmap_c, stage, sel, va, vb, c.b, row0, col0, lane);
            } else {
                store_block_staged<OUT_BF16>(p, tmap_c, stage, sel, va, c.b, row0, col0, lane);
                if (two) store_block_staged<OUT_BF16>(p, tmap_c, stage, sel, vb, c.b, row0, col0 + 32, lane);
            }
        }
        return ok;
    }

    const int row0 = row - lane;                         // global row of this warp's lane 0
    if (row0 >= p.M) return ok;                          // the whole warp is below the matrix
#pragma unroll 1
    for (int ch = 0; ch < kChunks; ++ch) {
        const int col0 = c.n_tile * BLOCK_N + ch * 32;
        if (col0 >= p.N) break;                          // warp-uniform: nothing further to store
        if (p.c_tma && (ch & 1) == 0 && (col0 + 64 <= p.N || (p.n_edge_tma && col0 + 32 < p.N))) {
            uint32_t ra[32], rb[32];
            tmem_ld_32x32b_x32(t_addr + ch * 32, ra);
            tmem_ld_32x32b_x32(t_addr + ch * 32 + 32, rb);
            tmem_ld_wait();
            float va[32], vb[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                va[j] = __uint_as_float(ra[j]);
                vb[j] = __uint_as_float(rb[j]);
            }
            store_two_blocks_staged<OUT_BF16>(tmap_c, stage, sel, va, vb, c.b, row0, col0, lane);
            ++ch;
            continue;
        }
        uint32_t r[32];
        tmem_ld_32x32b_x32(t_addr + ch * 32, r);
        tmem_ld_wait();
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
        store_block_staged<OUT_BF16>(p, tmap_c, stage, sel, v, c.b, row0, col0, lane);
    }
    return ok;
}

// (Instantiations whose shared memory lets two CTAs share an SM must also fit two CTAs'
// registers: 65536 / (2 x 192) = 170 per thread.)
template <int BLOCK_N, int STAGES, int KSUB, bool OUT_BF16, int A_ROWS = kBlockM>
__global__ void __launch_bounds__(kNumThreads,
                                  SmemLayout<BLOCK_N, STAGES, KSUB, A_ROWS>::kDynamicBytes <= 112 * 1024 ? 2 : 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const __grid_constant__ CUtensorMap tmap_c, const GemmParams p)
{
    using L = SmemLayout<BLOCK_N, STAGES, KSUB, A_ROWS>;
    static_assert(KSUB == 1 || KSUB == 2, "k-blocks per stage");
    static_assert(BLOCK_N % 64 == 0 && BLOCK_N >= 64 && BLOCK_N <= 256, "BLOCK_N");
    constexpr uint32_t kTmemCols = 2 * BLOCK_N;          // 128, 256 or 512: power of two

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
        if (p.c_tma) prefetch_tensormap(&tmap_c);
    }
    if (warp_idx == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
        tmem_relinquish();
    }
    // The producer needs the barriers, which its own thread 0 has just initialised, but
    // not tensor memory: warp 0 announces its arrival and goes on (the first loads are
    // on their way while the allocation completes); the other warps wait for everything.
    uint32_t tmem_base = 0;
    if (warp_idx == 0) {
        __syncwarp();
        named_bar_arrive(1, kNumThreads);
    } else {
        tc_fence_before();
        named_bar_sync(1, kNumThreads);
        tc_fence_after();
        tmem_base = *tmem_slot;
    }
    grid_launch_dependents();
    // Each role waits for the previous kernel of the stream where it first touches global
    // memory: the producer just before its first load (the first unit's coordinates are
    // worked out before), the epilogue warps before their loop; the MMA thread never does.

    if (warp_idx == 0) {
        // ------------------------------------------------ TMA producer ----
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            uint32_t tok = 1;                            // the first STAGES stages start out free
            bool waited = false;
            for (int u = blockIdx.x; ok && u < p.num_units; u += gridDim.x) {
                const UnitCoord c = decode_unit(p, u);
                constexpr int boxes = BLOCK_N / 64;
                for (int kb = c.kb_begin; kb < c.kb_end; kb += KSUB) {
                    if (!tok && !mbar_wait(empty_bar(stage), phase ^ 1, abort_flag, p.wait_limit_ns)) {
                        report_timeout(p.status, kRoleProducer, stage);
                        ok = false;
                        break;
                    }
                    // probes the next stage, then issues this stage's loads (one asm block);
                    // a stage takes up to KSUB k-blocks, all from the same operand segment
                    const int nstage = (stage + 1 == STAGES) ? 0 : stage + 1;
                    const uint32_t nphase = (stage + 1 == STAGES) ? phase ^ 1 : phase;
                    const uint32_t sa = smem_base + stage * L::kStageBytes;
                    const KBlockCoord kc = kblock_coord(p, kb, c.b);
                    const int nsub = min(min(c.kb_end - kb, KSUB), kc.left_in_segment);
                    if (!waited) {
                        grid_dependency_wait();
                        waited = true;
                    }
                    tok = tma_stage_step<false>(empty_bar(nstage), nphase ^ 1, full_bar(stage), 1,
                                                nsub * (p.a_box_bytes + boxes * (64 * kBlockK * 2)), full_bar(stage),
                                                &tmap_a, &tmap_b, sa, sa + L::kABytes, kc.k,
                                                c.m_tile * kBlockM, c.n_tile * BLOCK_N, kc.batch_a,
                                                kc.batch_b, boxes, nsub, L::kSubBytes);
                    kb += nsub - KSUB;                   // the loop adds KSUB
                    stage = nstage;
                    phase = nphase;
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
            uint32_t tok = 0;                            // answer of the probe of full[stage]
            for (int u = blockIdx.x; ok && u < p.num_units; u += gridDim.x) {
                const UnitCoord c = decode_unit(p, u);
                constexpr uint32_t idesc = make_idesc_bf16(kBlockM, BLOCK_N, 0, 1);
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1, abort_flag, p.wait_limit_ns)) {
                    report_timeout(p.status, kRoleMma, 0x40 + acc);
                    break;
                }
                const uint32_t d_tmem = tmem_base + acc * BLOCK_N;
                bool first_of_unit = true;
                for (int kb = c.kb_begin; kb < c.kb_end; kb += KSUB) {
                    if (!tok && !mbar_wait(full_bar(stage), phase, abort_flag, p.wait_limit_ns)) {
                        report_timeout(p.status, kRoleMma, stage);
                        ok = false;
                        break;
                    }
                    // probes the next stage, then issues this stage's MMAs (four per k-block) and
                    // the commit that frees the stage when they retire (one asm block).
                    // A: K-major, 8-row groups 1024 B apart (SBO); 16 K-elements = 32 B.
                    // B: MN-major, 64-column chunks 8192 B apart (LBO), 8-k groups
                    //    1024 B apart (SBO); 16 k = 2048 B.
                    const int nsub = min(min(c.kb_end - kb, KSUB), kblock_coord(p, kb, c.b).left_in_segment);
                    const int nstage = (stage + 1 == STAGES) ? 0 : stage + 1;
                    const uint32_t nphase = (stage + 1 == STAGES) ? phase ^ 1 : phase;
                    const uint32_t sa = smem_base + stage * L::kStageBytes;
                    tok = umma_stage_step<false>(full_bar(nstage), nphase, d_tmem, idesc,
                                                 first_of_unit ? 0u : 1u,
                                                 make_smem_desc_sw128(sa, 16, 1024),
                                                 make_smem_desc_sw128(sa + L::kABytes, 8192, 1024),
                                                 L::kSubBytes, nsub, empty_bar(stage), 0);
                    first_of_unit = false;
                    kb += nsub - KSUB;                   // the loop adds KSUB
                    stage = nstage;
                    phase = nphase;
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
        uint32_t sel = 0;                                // staging block of the next TMA store
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
            if (!epilogue_tile<BLOCK_N, OUT_BF16>(p, c, c.m_tile * kBlockM + epi_tid,
                                                  tmem_base + acc * BLOCK_N + (static_cast<uint32_t>(quad * 32) << 16),
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

}  // namespace cudallm
