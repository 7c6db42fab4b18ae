// Fused multi-head self-attention for short sequences (the paper's Task 6):
//
//   head_i = softmax(Q_i K_i^T / sqrt(d_k)) V_i,   O = Concat(head_1 .. head_h)
//
// Q, K, V are N x d_model bf16, row-major; head i owns columns [i d_k, (i+1) d_k).
// One CTA computes 128 query rows of one head for d_k <= 32 (the paper's sizes go up
// to N = 512, d_model = 512, h = 16).  Up to 512 keys are handled in one pass, steps
// 1 to 5 below; longer sequences in blocks of 512 keys with a running maximum: a
// block's probabilities are taken relative to the maximum so far, the row's
// accumulated output and sum (registers) are scaled by exp(old max - new max) and the
// block's product is added (step 6).
//
//   1. all threads copy Q_i (128 x d_k), K_i (N x d_k) and V_i (N x d_k) into
//      shared memory, directly in the tensor core's unswizzled operand layouts
//      (8-row x 16-byte core matrices), zero-padding rows and d_k; the 16-byte
//      pieces of one row go to neighbouring lanes (a warp's load touches 8 rows,
//      not 32: the copy is bound by the number of 128-byte lines per
//      instruction), and the strides between d_k chunks carry 32 bytes of
//      padding so that those lanes' stores fall on distinct banks;
//   2. one thread issues S = Q_i K_i^T with tcgen05.mma into tensor memory: all
//      keys at once, 128 lanes x up to 512 fp32 columns -- the whole of TMEM;
//   3. two threads share one query row (one TMEM lane; warps w and w + 4 read
//      the same lanes), each taking half of the key chunks: two passes over
//      the row of S (maximum, exchanged through shared memory; then
//      p = exp2((s - max) * log2(e)/sqrt(d_k)), masked beyond N, summed, rounded
//      to bf16 and written to shared memory as the K-major A operand of the
//      second product);
//   4. one thread issues O = P [V_i | 1] (V_i is the MN-major B operand, with a
//      column of ones behind its d_k columns) into the TMEM columns that S no
//      longer needs: column d_k of O is the row sum of the rounded probabilities,
//      exactly what the product saw, at no cost to the softmax threads;
//   5. the row's two threads divide their halves of the row of O by the row sum;
//      the block goes through shared memory so that a warp's store covers whole
//      rows of the head's columns.
//
//   6. (N > 512) the next block of keys: K_i and V_i rows again (step 1), S (2), the
//      block's maximum joined with the running one, P relative to the new maximum (3),
//      the block's O and row sum (4) added to the scaled accumulators.
//
// The two waits on tensor-core completion per block are bounded like those of the
// GEMM kernels.
#pragma once
#include <cuda_bf16.h>

#include "ptx.cuh"

namespace cudallm {

constexpr int kMhsaRows = 128;        // queries per CTA
constexpr int kMhsaThreads = 256;     // two threads per query row
constexpr int kMhsaMaxKeys = 512;     // = TMEM columns
constexpr int kMhsaMaxDk = 32;

struct MhsaParams {
    const __nv_bfloat16 *Q, *K, *V;
    float *O;
    int N, h, dk;
    int keys_pad;           // keys per block: N rounded up to 32, or 512 when N > 512
    int dkp;                // d_k rounded up to 16 (K of the first product, N of the second)
    int tmem_cols;          // power of two >= max(keys_pad, 64): tensor-memory columns to allocate
    long long ldq, ldk, ldv, ldo;
    float scale_log2;       // log2(e) / sqrt(d_k)
    int *status;
};

// Unswizzled shared-memory matrix descriptor: start address, leading-dimension
// and stride-dimension byte offsets in 16-byte units, descriptor version 1.
__device__ __forceinline__ uint64_t make_smem_desc_plain(uint32_t smem_addr, uint32_t lbo_bytes,
                                                         uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFF) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    return d;
}

__device__ __forceinline__ void umma_bf16_1cta(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                               uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// 2^x by the special-function unit (relative error ~2^-22; inputs <= 0 here)
__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct MhsaSmem {
    // byte offsets inside the dynamic shared memory block (multiples of 32) and strides
    int q, k, v, p, bar, xch, total;
    int lbo_q, lbo_k;       // bytes between the d_k chunks (8 elements wide) of Q and of K
    int lbo_v, sbo_v;       // V: bytes between groups of 8 keys, and between d_k chunks inside a group
};
constexpr int kMhsaOutPitch = 36;     // floats per row of the output staging block (conflict-free 16-byte stores)
__host__ __device__ inline MhsaSmem mhsa_smem_layout(int keys_pad, int dkp)
{
    MhsaSmem s;
    const int kchunks = dkp / 8;
    s.lbo_q = kMhsaRows * 16 + 32;                    // [chunk][row][16 B] + padding
    s.lbo_k = keys_pad * 16 + 32;                     // [chunk][key][16 B] + padding
    s.sbo_v = 128 + 32;                               // [key group][chunk][key in group][16 B] + padding
    // one more chunk per key group: the column of ones.  (The second product has N = dkp + 16
    // columns, so it also reads the chunk after that one -- the next group's first chunk, or
    // the bytes behind V for the last group -- into output columns that nobody looks at.)
    s.lbo_v = (kchunks + 1) * s.sbo_v;
    s.q = 0;
    s.k = s.q + kchunks * s.lbo_q;
    s.v = s.k + kchunks * s.lbo_k;
    s.p = s.v + (keys_pad / 8) * s.lbo_v;             // (keys_pad/8) chunks x 16 row groups x 128 B
    s.p = (s.p + 127) & ~127;
    int p_bytes = (keys_pad / 8) * 2048;
    if (p_bytes < kMhsaRows * kMhsaOutPitch * 4) p_bytes = kMhsaRows * kMhsaOutPitch * 4;   // reused for the output block
    s.bar = s.p + p_bytes;
    s.xch = s.bar + 64;                               // row maxima and row sums of the two halves
    s.total = s.xch + 2 * kMhsaThreads * 4;
    return s;
}

// 32 scores of one row -> 32 probabilities exp2(s * c - max * c), rounded to bf16 and packed
// in pairs: one FMA and one ex2.approx per element.  MASKED: keys from `valid` on do not
// exist (the ragged last chunk) and get probability 0.
template <bool MASKED>
__device__ __forceinline__ void mhsa_exp_chunk(const uint32_t (&r)[32], float scale, float neg_max_scaled,
                                               int valid, uint32_t (&w)[16])
{
#pragma unroll
    for (int j = 0; j < 32; j += 2) {
        float e0 = fast_exp2(fmaf(__uint_as_float(r[j]), scale, neg_max_scaled));
        float e1 = fast_exp2(fmaf(__uint_as_float(r[j + 1]), scale, neg_max_scaled));
        if (MASKED) {
            if (j >= valid) e0 = 0.f;
            if (j + 1 >= valid) e1 = 0.f;
        }
        w[j >> 1] = pack_bf16x2(e0, e1);
    }
}

// MULTI: more than one block of keys (N > 512); the one-block instance keeps no accumulators.
template <bool MULTI>
__global__ void __launch_bounds__(kMhsaThreads, 1)
mhsa_kernel(const MhsaParams p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const MhsaSmem L = mhsa_smem_layout(p.keys_pad, p.dkp);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar = sbase + L.bar;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + L.bar + 16);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L.bar + 20);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int row_in = tid & (kMhsaRows - 1);         // query row of this thread inside the block
    const int half = tid >> 7;                        // which half of the key chunks it takes
    float *xch = reinterpret_cast<float *>(smem + L.xch);
    const int head = blockIdx.y;
    const int q0 = blockIdx.x * kMhsaRows;
    const int col0 = head * p.dk;
    const int kchunks = p.dkp / 8;                    // 16-byte chunks along d_k: 2 or 4

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar, 1);
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), p.tmem_cols);
        tmem_relinquish();
    }

    grid_launch_dependents();
    grid_dependency_wait();                           // (launched with programmatic stream serialisation)

    const uint32_t t_row_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const int kshift = kchunks == 4 ? 2 : 1;          // kchunks is 2 or 4
    const int nch = p.keys_pad / 32;
    const int ch_lo = half ? (nch + 1) / 2 : 0, ch_hi = half ? nch : (nch + 1) / 2;
    const int nblocks = MULTI ? (p.N + p.keys_pad - 1) / p.keys_pad : 1;
    constexpr int kInFlight = MULTI ? 2 : 4;          // 32-column loads of S per wait (the accumulators need registers too)
    // running maximum, sum and this thread's half of the row of O (blocks of keys: step 6)
    float m_run = -INFINITY, l_acc = 0.f;
    float o_acc[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) o_acc[k] = 0.f;
    uint32_t tmem = 0;
    bool ok = true;

#pragma unroll 1
    for (int kb = 0; kb < nblocks; ++kb) {
        const int key0 = kb * p.keys_pad;
        const int nvalid = min(p.keys_pad, p.N - key0);       // keys of this block that exist (>= 1)

        // ---- 1. operands -> shared memory, in core-matrix order -------------------
        // One list of 16-byte pieces: the rows of Q (first block only), then K's, then V's, the
        // d_k chunks of a row on neighbouring lanes (at N = 512 and d_k = 32, eighteen per thread).
        // Asynchronous 16-byte copies straight into shared memory (a piece outside the
        // operand -- a padding row or d_k chunk -- copies zero source bytes: it is zero-filled).
        const int first = kb == 0 ? 0 : kMhsaRows << kshift;
        const int total = (kMhsaRows + 2 * p.keys_pad) << kshift;
        for (int i = first + tid; i < total; i += kMhsaThreads) {
            const __nv_bfloat16 *src = p.Q;           // (any valid address: no byte of it is read)
            uint32_t bytes = 0;
            int dst;
            const int c = i & (kchunks - 1);
            int r = i >> kshift;
            const bool live = c * 8 < p.dk;
            if (r < kMhsaRows) {                      // Q: row within the block
                const int row = q0 + r;
                dst = L.q + c * L.lbo_q + r * 16;
                if (row < p.N && live) { src = p.Q + row * p.ldq + col0 + c * 8; bytes = 16; }
            } else if (r < kMhsaRows + p.keys_pad) {
                r -= kMhsaRows;                       // K: key of the block
                dst = L.k + c * L.lbo_k + r * 16;
                if (r < nvalid && live) { src = p.K + (key0 + r) * p.ldk + col0 + c * 8; bytes = 16; }
            } else {
                r -= kMhsaRows + p.keys_pad;          // V: key of the block
                dst = L.v + (r >> 3) * L.lbo_v + c * L.sbo_v + (r & 7) * 16;
                if (r < nvalid && live) { src = p.V + (key0 + r) * p.ldv + col0 + c * 8; bytes = 16; }
            }
            cp_async_16(sbase + dst, src, bytes);
        }
        cp_async_wait_all();
        // behind V's d_k chunks: a column of ones (bf16 1.0 in element 0 of the chunk)
        if (kb == 0)
            for (int j = tid; j < p.keys_pad; j += kMhsaThreads)
                *reinterpret_cast<uint4 *>(smem + L.v + (j >> 3) * L.lbo_v + kchunks * L.sbo_v + (j & 7) * 16) =
                    make_uint4(0x3F80u, 0, 0, 0);
        fence_proxy_async_smem();                     // make the writes visible to the tensor core
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        tmem = *tmem_slot;
        const uint32_t t_row = tmem + t_row_off;

        // ---- 2. S = Q K^T ---------------------------------------------------------
        const int n1 = p.keys_pad < 256 ? p.keys_pad : 256;
        const int n2 = p.keys_pad - n1;
        if (tid == 0 && ok) {
            for (int part = 0; part < 2; ++part) {
                const int n = part ? n2 : n1;
                if (n == 0) break;
                const uint32_t idesc = make_idesc_bf16(kMhsaRows, n, 0, 0);      // both operands K-major
                for (int ks = 0; ks < p.dkp / 16; ++ks) {
                    const uint64_t da = make_smem_desc_plain(sbase + L.q + ks * 2 * L.lbo_q, L.lbo_q, 128);
                    const uint64_t db = make_smem_desc_plain(sbase + L.k + ks * 2 * L.lbo_k + part * (256 / 8) * 128,
                                                             L.lbo_k, 128);
                    umma_bf16_1cta(tmem + part * 256, da, db, idesc, ks > 0 ? 1u : 0u);
                }
            }
            umma_commit(bar);
        }
        if (ok) ok = mbar_wait(bar, 0, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();

        // ---- 3. softmax: this thread's half of its row ------------------------------
        // Several 32-column loads are in flight per wait: a TMEM round trip costs far
        // more than the arithmetic on 32 values.
        float blk_max = -INFINITY;
        if (ok) {
#pragma unroll 1
            for (int ch0 = ch_lo; ch0 < ch_hi; ch0 += kInFlight) {
                uint32_t r[kInFlight][32];
#pragma unroll
                for (int u = 0; u < kInFlight; ++u)
                    if (ch0 + u < ch_hi) tmem_ld_32x32b_x32(t_row + (ch0 + u) * 32, r[u]);
                tmem_ld_wait();
#pragma unroll
                for (int u = 0; u < kInFlight; ++u) {
                    if (ch0 + u < ch_hi) {
                        if ((ch0 + u) * 32 + 32 <= nvalid) {                     // all 32 keys exist
#pragma unroll
                            for (int j = 0; j < 32; ++j) blk_max = fmaxf(blk_max, __uint_as_float(r[u][j]));
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if ((ch0 + u) * 32 + j < nvalid) blk_max = fmaxf(blk_max, __uint_as_float(r[u][j]));
                        }
                    }
                }
            }
        }
        xch[tid] = blk_max;
        __syncthreads();
        blk_max = fmaxf(xch[row_in], xch[row_in + kMhsaRows]);      // the first half always has a key that exists
        const float m_new = fmaxf(m_run, blk_max);
        // what the accumulators of the earlier blocks are worth relative to the new maximum
        const float alpha = (!MULTI || kb == 0) ? 0.f : fast_exp2((m_run - m_new) * p.scale_log2);
        m_run = m_new;
        const float neg_max_scaled = -m_new * p.scale_log2;
        if (ok) {
            const int r_off = (row_in >> 3) * 128 + (row_in & 7) * 16;           // this row inside a chunk of P
#pragma unroll 1
            for (int ch0 = ch_lo; ch0 < ch_hi; ch0 += kInFlight) {
                uint32_t r[kInFlight][32];
#pragma unroll
                for (int u = 0; u < kInFlight; ++u)
                    if (ch0 + u < ch_hi) tmem_ld_32x32b_x32(t_row + (ch0 + u) * 32, r[u]);
                tmem_ld_wait();
#pragma unroll
                for (int u = 0; u < kInFlight; ++u) {
                    const int ch = ch0 + u;
                    if (ch < ch_hi) {
                        uint32_t w[16];
                        if (ch * 32 + 32 <= nvalid) mhsa_exp_chunk<false>(r[u], p.scale_log2, neg_max_scaled, 32, w);
                        else                        mhsa_exp_chunk<true>(r[u], p.scale_log2, neg_max_scaled, nvalid - ch * 32, w);
#pragma unroll
                        for (int g = 0; g < 4; ++g)                              // 8 keys = one 16-byte chunk
                            *reinterpret_cast<uint4 *>(smem + L.p + (ch * 4 + g) * 2048 + r_off) =
                                make_uint4(w[4 * g], w[4 * g + 1], w[4 * g + 2], w[4 * g + 3]);
                    }
                }
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();                               // everyone is done reading S and writing P
        tc_fence_after();

        // ---- 4. O = P V -------------------------------------------------------------
        if (tid == 0 && ok) {
            const uint32_t idesc = make_idesc_bf16(kMhsaRows, p.dkp + 16, 0, 1); // [V | 1 | unused]: MN-major
            for (int ks = 0; ks < p.keys_pad / 16; ++ks) {
                const uint64_t da = make_smem_desc_plain(sbase + L.p + ks * 2 * 2048, 2048, 128);
                const uint64_t db = make_smem_desc_plain(sbase + L.v + ks * 2 * L.lbo_v, L.lbo_v, L.sbo_v);
                umma_bf16_1cta(tmem, da, db, idesc, ks > 0 ? 1u : 0u);
            }
            umma_commit(bar);
        }
        if (ok) {
            ok = mbar_wait(bar, 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
        }
        tc_fence_after();

        // ---- 6. the block's O and row sum join the accumulators ---------------------
        if (ok) {
            uint32_t r[32], r2[32];
            tmem_ld_32x32b_x32(t_row, r);              // d_k <= 32 columns of O ...
            if (p.dkp == 32) tmem_ld_32x32b_x32(t_row + 32, r2);             // ... and the row sum in column dkp
            tmem_ld_wait();
            if (MULTI) {
                l_acc = fmaf(l_acc, alpha, __uint_as_float(p.dkp == 32 ? r2[0] : r[16]));
#pragma unroll
                for (int k = 0; k < 16; ++k) o_acc[k] = fmaf(o_acc[k], alpha, __uint_as_float(half ? r[16 + k] : r[k]));
            } else {
                l_acc = __uint_as_float(p.dkp == 32 ? r2[0] : r[16]);
#pragma unroll
                for (int k = 0; k < 16; ++k) o_acc[k] = __uint_as_float(half ? r[16 + k] : r[k]);
            }
        }
        if (MULTI && kb + 1 < nblocks) {
            tc_fence_before();
            __syncthreads();                           // O has been read: the next block may overwrite S, K, V and P
            tc_fence_after();
        }
    }

    // ---- 5. normalise and store (each of the row's two threads: half of d_k) -----
    // P's shared memory is free now and takes the 128 x d_k block of O, rows 36 floats
    // apart; then every 16-byte store instruction of a warp covers whole rows of the
    // head's columns instead of 32 different rows.
    const bool vec_out = ((reinterpret_cast<uintptr_t>(p.O) & 15) == 0) && (p.ldo % 4 == 0);
    float *stage = reinterpret_cast<float *>(smem + L.p);
    if (ok) {
        const int row = q0 + row_in;
        const float inv = 1.f / l_acc;
        float o[16];                                   // this thread's half of the row
#pragma unroll
        for (int k = 0; k < 16; ++k) o[k] = o_acc[k] * inv;
        if (vec_out) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const int d = half * 16 + g * 4;
                if (d < p.dk)
                    *reinterpret_cast<float4 *>(stage + row_in * kMhsaOutPitch + d) =
                        make_float4(o[4 * g], o[4 * g + 1], o[4 * g + 2], o[4 * g + 3]);
            }
        } else if (row < p.N) {
            float *dst = p.O + row * p.ldo + col0 + half * 16;
#pragma unroll
            for (int k = 0; k < 16; ++k)
                if (half * 16 + k < p.dk) dst[k] = o[k];
        }
    } else if (tid == 0) {
        if (atomicCAS(p.status, 0, -9) == 0) p.status[1] = 0x600;
    }
    tc_fence_before();
    __syncthreads();
    if (ok && vec_out) {
        const int per_row = p.dk / 4;                  // 16-byte pieces per row: 2, 4, 6 or 8
        const int rows = min(kMhsaRows, p.N - q0);
        for (int i = tid; i < rows * per_row; i += kMhsaThreads) {
            const int r = i / per_row, c = i - r * per_row;
            *reinterpret_cast<float4 *>(p.O + (q0 + r) * p.ldo + col0 + c * 4) =
                *reinterpret_cast<const float4 *>(stage + r * kMhsaOutPitch + c * 4);
        }
    }
    if (warp == 0) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem, p.tmem_cols);
    }
}

}  // namespace cudallm
