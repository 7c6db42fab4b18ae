// Copying operands that TMA cannot address (base not 16-byte aligned, or a row pitch that
// is not a multiple of 16 bytes) into an aligned scratch buffer:
//  * PackJob     -- one operand to copy;
//  * row_copy_*  -- a warp copies up to 512 consecutive elements of one row from a 2-byte
//    aligned source to a 16-byte aligned destination with 16-byte loads and stores.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"

namespace cudallm {

// One operand to repack: dst[b][r][0..cols) = src[b][r][0..cols), columns up to the next
// multiple of 8 zero; dst is 16-byte aligned and its row pitch ld_dst and batch stride are
// multiples of 8 elements; src needs 2-byte alignment only.
struct PackJob {
    const uint16_t *src;
    uint16_t *dst;
    int rows, cols, batch;
    long long ld_src, ld_dst, stride_src, stride_dst;
    long long total_rows;                                // rows * batch (0 = nothing to do)
};

// ---------------------------------------------------------------------------
// Warp-wide copy of up to 64 consecutive 16-byte pieces (512 elements) of one row from a
// source that is only 2-byte aligned to a 16-byte aligned destination.
//   src / dst point at the first of those elements; cols_left (>= 1) is how many elements
//   the row still has from there: pieces beyond it are not written, the last one is
//   zero-padded to 8 elements.
// The source bytes are fetched as aligned 16-byte chunks of the window that starts at the
// 16-byte boundary at or below src: lane l takes chunks 2l and 2l + 1 (lane 31 also chunk
// 64), gets chunk 2l + 2 from its neighbour by shuffle, and extracts its two pieces with
// funnel shifts.  All lanes work on the same row, so the byte offset of the data inside the
// chunks is warp-uniform: a four-way uniform branch, no per-lane address arithmetic.  A
// chunk is only fetched if it holds at least one byte of the row from src on, so the loads
// touch the 16-byte granules that contain the first and the last element wanted but nothing
// beyond them.
struct RowCopy {
    uint4 c0, c1;               // chunks 2 * lane and 2 * lane + 1
    uint4 extra;                // lane 31: chunk 64
};
__device__ __forceinline__ void row_copy_load(RowCopy &rc, const uint16_t *src, int cols_left, int lane)
{
    const uintptr_t s = reinterpret_cast<uintptr_t>(src);
    const uintptr_t a = s & ~static_cast<uintptr_t>(15);
    const uintptr_t end = s + 2 * static_cast<uintptr_t>(min(cols_left, 512));   // one past the last byte wanted
    const uint4 zero = make_uint4(0, 0, 0, 0);
    const uintptr_t p0 = a + 32 * static_cast<uintptr_t>(lane);
    rc.c0 = p0 < end ? __ldg(reinterpret_cast<const uint4 *>(p0)) : zero;
    rc.c1 = p0 + 16 < end ? __ldg(reinterpret_cast<const uint4 *>(p0 + 16)) : zero;
    rc.extra = (lane == 31 && a + 1024 < end) ? __ldg(reinterpret_cast<const uint4 *>(a + 1024)) : zero;
}
// the 16 bytes that start `4 * wo + sh / 8` bytes into cur (continuing in nxt); wo and sh warp-uniform
__device__ __forceinline__ uint4 extract_piece(const uint4 &cur, const uint4 &nxt, uint32_t wo, uint32_t sh)
{
    uint4 o;
    switch (wo) {
    case 0:
        o.x = __funnelshift_r(cur.x, cur.y, sh); o.y = __funnelshift_r(cur.y, cur.z, sh);
        o.z = __funnelshift_r(cur.z, cur.w, sh); o.w = __funnelshift_r(cur.w, nxt.x, sh);
        break;
    case 1:
        o.x = __funnelshift_r(cur.y, cur.z, sh); o.y = __funnelshift_r(cur.z, cur.w, sh);
        o.z = __funnelshift_r(cur.w, nxt.x, sh); o.w = __funnelshift_r(nxt.x, nxt.y, sh);
        break;
    case 2:
        o.x = __funnelshift_r(cur.z, cur.w, sh); o.y = __funnelshift_r(cur.w, nxt.x, sh);
        o.z = __funnelshift_r(nxt.x, nxt.y, sh); o.w = __funnelshift_r(nxt.y, nxt.z, sh);
        break;
    default:
        o.x = __funnelshift_r(cur.w, nxt.x, sh); o.y = __funnelshift_r(nxt.x, nxt.y, sh);
        o.z = __funnelshift_r(nxt.y, nxt.z, sh); o.w = __funnelshift_r(nxt.z, nxt.w, sh);
        break;
    }
    return o;
}
// zero the elements from `nvalid` (< 8) on
__device__ __forceinline__ uint4 keep_elements(uint4 v, int nvalid)
{
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (2 * i >= nvalid) w[i] = 0;
        else if (2 * i + 1 >= nvalid) w[i] &= 0xFFFFu;
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}
__device__ __forceinline__ void row_copy_store(const RowCopy &rc, const uint16_t *src, uint16_t *dst, int cols_left,
                                               int lane)
{
    const uint32_t off = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(src) & 15);
    const uint32_t wo = off >> 2, sh = (off & 2) * 8;
    uint4 nxt;                                           // chunk 2 * lane + 2: the neighbour's first
    nxt.x = __shfl_down_sync(0xffffffffu, rc.c0.x, 1);
    nxt.y = __shfl_down_sync(0xffffffffu, rc.c0.y, 1);
    nxt.z = __shfl_down_sync(0xffffffffu, rc.c0.z, 1);
    nxt.w = __shfl_down_sync(0xffffffffu, rc.c0.w, 1);
    if (lane == 31) nxt = rc.extra;
    const int e0 = 16 * lane;                            // first element of this lane's two pieces
    if (e0 < cols_left) {
        uint4 o = extract_piece(rc.c0, rc.c1, wo, sh);
        if (cols_left - e0 < 8) o = keep_elements(o, cols_left - e0);
        *reinterpret_cast<uint4 *>(dst + e0) = o;
    }
    if (e0 + 8 < cols_left) {
        uint4 o = extract_piece(rc.c1, nxt, wo, sh);
        if (cols_left - e0 < 16) o = keep_elements(o, cols_left - e0 - 8);
        *reinterpret_cast<uint4 *>(dst + e0 + 8) = o;
    }
}

// The same copy for a unit with at least 514 elements left in its row (any unit that is not a
// row's last), with as few instructions as it takes: every lane reads, for each of its two
// pieces, the five 4-byte words that hold the piece (from the 4-byte boundary at or below it;
// the fifth word is only used when the source is 2 bytes past such a boundary, and lies inside
// the row either way) and shifts them into place.  No branch, no shuffle.
__device__ __forceinline__ void row_copy_interior(const uint16_t *src, uint16_t *dst, int lane)
{
    const uint32_t odd = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(src) >> 1) & 1u;
    const uint32_t *q = reinterpret_cast<const uint32_t *>(src - odd) + 4 * lane;
    const uint32_t sh = odd * 16;
    uint32_t w[2][5];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int i = 0; i < 5; ++i) w[h][i] = __ldg(q + 128 * h + i);
#pragma unroll
    for (int h = 0; h < 2; ++h)
        *reinterpret_cast<uint4 *>(dst + 8 * lane + 256 * h) =
            make_uint4(__funnelshift_r(w[h][0], w[h][1], sh), __funnelshift_r(w[h][1], w[h][2], sh),
                       __funnelshift_r(w[h][2], w[h][3], sh), __funnelshift_r(w[h][3], w[h][4], sh));
}

}  // namespace cudallm
