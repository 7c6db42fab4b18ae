/*
 * cudallm_gemm.h -- C ABI of the B200 (sm_100a) bf16 GEMM library.
 *
 * The operation is the paper's benchmark Task 2, "Matrix Multiplication":
 * given A (M x K) and B (K x N) compute C = A x B (M x N), i.e.
 *
 *     C[i][j] = sum_{k=0}^{K-1} A[i][k] * B[k][j]
 *
 * with all three matrices stored row-major as flat arrays (the storage the
 * paper's task descriptions state for its matrix tasks).  Here A and B hold
 * bfloat16, products are accumulated in fp32 and C is written as fp32 or
 * bfloat16 (rounded once, to nearest even).  Old contents of C are never
 * read (beta = 0).
 *
 * The paper's programs own their buffers and transfers in host code and hand
 * raw device pointers to one kernel launch (Section 2, "CUDA program"); the
 * calls below keep that split: the caller owns every buffer, the library only
 * enqueues work on the caller's stream.
 *
 * General conventions
 *  - Unless a parameter says "host", pointers are DEVICE pointers.
 *  - Leading dimensions and batch strides are in ELEMENTS, not bytes.
 *  - Every call returns a status: 0 on success, a negative CUDALLM_ERR_* code
 *    otherwise.  Argument errors are detected before any CUDA call is made,
 *    and nothing is written in that case.
 *  - Calls enqueue on `stream` (a cudaStream_t passed as void*; NULL is the
 *    legacy default stream) and return without synchronising, except where
 *    stated.
 *  - Only element alignment is required (2 bytes for bf16, 4 for fp32
 *    output).  16-byte aligned bases with leading dimensions that are
 *    multiples of 8 elements take the direct TMA path; other operands are
 *    first repacked into the library workspace.
 *  - Degenerate sizes: M == 0 or N == 0 or batch == 0 -> success, nothing
 *    written.  K == 0 -> the M x N block of C is set to zero.
 *  - Padding columns of C (N <= j < ldc) are left untouched.
 *  - C must not overlap A or B.
 *  - The library is for compute capability 10.0 devices only and has no CPU
 *    fallback.
 *  - Calls that need the workspace (repacking, split-K) share one workspace
 *    per device; such calls must not run concurrently on different streams,
 *    unless each of those streams has a workspace of its own
 *    (cudallm_set_workspace_for_stream).
 *  - Split-K variants make some CTAs wait (with a time limit) for partial
 *    results of other CTAs of the same launch; they assume that the launch has
 *    the GPU to itself.  If another kernel holds SMs for seconds, such a wait
 *    can run out and is reported as CUDALLM_ERR_DEVICE_TIMEOUT.  On a stream
 *    with a workspace of its own the library's automatic choice therefore keeps
 *    to variants without such waits.
 */
#ifndef CUDALLM_GEMM_H
#define CUDALLM_GEMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* out_dtype */
#define CUDALLM_F32  0
#define CUDALLM_BF16 1

/* status codes */
#define CUDALLM_OK                      0
#define CUDALLM_ERR_INVALID_POINTER    -1  /* NULL operand with a non-empty problem            */
#define CUDALLM_ERR_INVALID_DIM        -2  /* negative size, or sizes beyond what is indexable  */
#define CUDALLM_ERR_INVALID_LD         -3  /* lda < K, ldb < N, ldc < N, or overlapping strides */
#define CUDALLM_ERR_INVALID_DTYPE      -4
#define CUDALLM_ERR_INVALID_VARIANT    -5
#define CUDALLM_ERR_UNSUPPORTED_SHAPE  -6  /* forced variant cannot run this problem            */
#define CUDALLM_ERR_UNSUPPORTED_DEVICE -7  /* current device is not compute capability 10.0     */
#define CUDALLM_ERR_CUDA               -8  /* a CUDA runtime/driver call failed                 */
#define CUDALLM_ERR_DEVICE_TIMEOUT     -9  /* a bounded wait inside a kernel ran out            */
#define CUDALLM_ERR_WORKSPACE         -10  /* workspace missing, too small or misaligned        */
#define CUDALLM_ERR_MISALIGNED        -11  /* pointer not aligned to its element size           */
#define CUDALLM_ERR_TOO_LARGE         -12  /* problem exceeds a built-in, fixed-size scratch    */

/* variant id meaning "let the library choose" */
#define CUDALLM_VARIANT_AUTO           -1

/*
 * C = A x B  (Task 2).
 *   A : bf16, M x K, row stride lda >= K      (read only)
 *   B : bf16, K x N, row stride ldb >= N      (read only)
 *   C : fp32 (out_dtype 0) or bf16 (out_dtype 1), M x N, row stride ldc >= N
 */
int cudallm_gemm_bf16(const void *A, const void *B, void *C,
                      int64_t M, int64_t N, int64_t K,
                      int64_t lda, int64_t ldb, int64_t ldc,
                      int out_dtype, void *stream);

/*
 * C = A x B with 32-bit floating point operands and result: the element type
 * the paper's Task 2 description gives for both factors and the product.
 *   A : fp32, M x K, row stride lda >= K      (read only)
 *   B : fp32, K x N, row stride ldb >= N      (read only)
 *   C : fp32, M x N, row stride ldc >= N
 * B200 has no fp32 tensor-core path, so each operand is first cut into three
 * bf16 pieces (x = x0 + x1 + x2, exact for normal numbers) in the workspace and
 * the six piece products of relative size >= 2^-16 are accumulated in fp32 by
 * the same tcgen05 kernels over a K range six times as long.  The result is
 * within 1e-5 * sum_k |a_ik||b_kj| of the exact product (what is dropped is of
 * relative size 2^-23; the fp32 accumulation contributes the rest); integer
 * cases whose partial sums stay below 2^24 are exact.  A non-finite input gives
 * a non-finite (possibly NaN) output in its row or column.  Pointers must be
 * 4-byte aligned; any leading dimensions are accepted.  Needs workspace:
 * 6 * (M*round_up(K,8) + K*round_up(N,8)) bytes plus what the chosen kernel
 * variant needs.  `variant` as in cudallm_gemm_bf16_variant (CUDALLM_VARIANT_AUTO
 * lets the library choose; the simt variant is not available here).
 */
int cudallm_gemm_f32(const void *A, const void *B, void *C,
                     int64_t M, int64_t N, int64_t K,
                     int64_t lda, int64_t ldb, int64_t ldc,
                     int variant, void *stream);

/*
 * The same product with the operands read by the tensor cores as they lie in
 * memory (tcgen05.mma kind::tf32: of every float32 operand the sign, the
 * exponent and the ten leading fraction bits are used; products are exact in
 * and accumulated in float32).  One pass over A and B, no conversion kernel, no
 * workspace beyond the header: about 3 times faster than cudallm_gemm_f32 on
 * the paper's Task 2 sizes, at about three decimal digits per product instead
 * of seven: every element within 2.5e-3 * sum_k |a_ik||b_kj| of the exact
 * product (2^-9 for two truncated operands plus the float32 accumulation);
 * operands whose values have at most 11 significant bits (e.g. integers below
 * 2048) are multiplied exactly.  Arguments as for cudallm_gemm_f32.  A and B must
 * be 16-byte aligned with lda and ldb multiples of 4 to be read in place; any
 * other alignment, and K == 0, are passed to cudallm_gemm_f32 (whose result is
 * the more accurate one).  C may have any 4-byte alignment and pitch.
 */
int cudallm_gemm_tf32(const void *A, const void *B, void *C,
                      int64_t M, int64_t N, int64_t K,
                      int64_t lda, int64_t ldb, int64_t ldc, void *stream);

/*
 * `batch` independent products of the same shape (Task 2 applied per item;
 * the paper's Task 6 score matrices Q_i K_i^T are products of this kind).
 * Item t uses A + t*strideA, B + t*strideB, C + t*strideC.  Items of C must
 * not overlap: strideC >= (M-1)*ldc + N when batch > 1.
 */
int cudallm_gemm_bf16_batched(const void *A, const void *B, void *C,
                              int64_t M, int64_t N, int64_t K,
                              int64_t lda, int64_t ldb, int64_t ldc,
                              int64_t strideA, int64_t strideB, int64_t strideC,
                              int64_t batch, int out_dtype, void *stream);

/*
 * As the batched call, but runs kernel variant `variant` instead of the
 * library's choice (CUDALLM_VARIANT_AUTO selects as the calls above do).
 * This is the hook for the search loop of the paper's Algorithm 1: candidates
 * are validated, timed and the fastest valid one kept.  Returns
 * CUDALLM_ERR_UNSUPPORTED_SHAPE when the variant cannot run the problem.
 */
int cudallm_gemm_bf16_variant(int variant,
                              const void *A, const void *B, void *C,
                              int64_t M, int64_t N, int64_t K,
                              int64_t lda, int64_t ldb, int64_t ldc,
                              int64_t strideA, int64_t strideB, int64_t strideC,
                              int64_t batch, int out_dtype, void *stream);

/*
 * The same product with HOST buffers (the paper's host-code pattern: copy the
 * operands in, launch, copy the result out).  A_host, B_host and C_host are
 * host pointers (pinned memory makes the copies asynchronous); `dev_buf` is a
 * caller-owned DEVICE staging buffer of `dev_bytes` bytes, at least
 * cudallm_host_staging_bytes(...) and 256-byte aligned.  The call copies
 * M*lda and K*ldb elements in, multiplies, copies M*ldc elements out, and
 * SYNCHRONISES `stream` before returning.  Internally B is copied first and A
 * in up to 4 row blocks on a second stream; each block is multiplied on
 * `stream` as soon as it has arrived and its rows of C return on a third
 * stream, so the two copy directions and the multiplication overlap.  The two
 * extra streams and their events are created on the first call per device.
 */
int cudallm_gemm_bf16_host(const void *A_host, const void *B_host, void *C_host,
                           int64_t M, int64_t N, int64_t K,
                           int64_t lda, int64_t ldb, int64_t ldc,
                           int out_dtype, void *dev_buf, size_t dev_bytes,
                           void *stream);
size_t cudallm_host_staging_bytes(int64_t M, int64_t N, int64_t K,
                                  int64_t lda, int64_t ldb, int64_t ldc,
                                  int out_dtype);

/*
 * Split-K product for callers that must not allocate.  (The paper has no
 * counterpart for this call: its programs allocate freely in host code.)
 *
 * Who needs it: a process whose device memory is entirely owned by someone
 * else's allocator (an inference server that reserved the whole GPU at start,
 * a framework plug-in that may only use the tensors it is handed), or code on
 * a path where a cudaMalloc -- which may synchronise the device or fail when
 * memory is exhausted -- is not acceptable.  The other entry points obtain
 * their split-K scratch from a workspace that the library allocates with
 * cudaMalloc on first need; this one calls no cudaMalloc, cudaFree or any
 * other allocating routine, ever.
 *
 * Its scratch is an array compiled into the library's device image
 * (CUDALLM_NOALLOC_SCRATCH_BYTES, 8 MiB, resident on every GPU that loads the
 * library until the process exits).  C is cut into tiles of 128 x 64 and each
 * tile's K range into `split_k` parts (2, 4, 8 or 16, at most ceil(K/64)) that
 * run as separate units; the units of a tile exchange their fp32 partial sums
 * through 32 KiB slots of that array, add them in fixed order and write C.
 *
 *  - A, B, C, sizes, leading dimensions and out_dtype as cudallm_gemm_bf16.
 *    A and B must take the direct TMA path: 16-byte aligned bases, lda and ldb
 *    multiples of 8 (else CUDALLM_ERR_UNSUPPORTED_SHAPE; repacking would need
 *    more scratch).
 *  - Limit: P = ceil(M/128) * ceil(N/64) * split_k slots of 32 KiB must fit
 *    behind the header: CUDALLM_NOALLOC_HEADER_BYTES + P * 32 KiB <=
 *    CUDALLM_NOALLOC_SCRATCH_BYTES, i.e. P <= 254; else the call returns
 *    CUDALLM_ERR_TOO_LARGE and nothing runs.
 *  - The call SYNCHRONISES `stream` before it returns (it reads the kernel's
 *    status word back) and reports a kernel whose bounded wait ran out as
 *    CUDALLM_ERR_DEVICE_TIMEOUT.  A synchronisation is not allowed on a stream
 *    that is being captured: never make this call, first or later, inside a
 *    stream capture.
 *  - The first call on each device also looks up the array's device address
 *    (and, like any first launch, lets the driver load the kernels).
 *  - All calls on a device share the one array, which keeps whatever the last
 *    call left in it; each call clears the words that must start at zero (the
 *    status word and the helper flags).  Two calls that overlap on the GPU
 *    (different streams, or different host threads) race on it: serialise them.
 */
#define CUDALLM_NOALLOC_SCRATCH_BYTES (8u << 20)
#define CUDALLM_NOALLOC_HEADER_BYTES  (64u << 10)   /* status word + helper flags */
int cudallm_gemm_bf16_splitk_noalloc(const void *A, const void *B, void *C,
                                     int64_t M, int64_t N, int64_t K,
                                     int64_t lda, int64_t ldb, int64_t ldc,
                                     int out_dtype, int split_k, void *stream);

/*
 * Multi-head self-attention: the paper's benchmark Task 6,
 *   O = Concat(head_1, ..., head_h),  head_i = softmax(Q_i K_i^T / sqrt(d_k)) V_i,
 * with d_k = d_model / h and Q_i, K_i, V_i the i-th head's partition (columns
 * [i d_k, (i+1) d_k)) of Q, K, V.  The softmax runs over the keys.
 *   Q, K, V : bf16, N x d_model, row strides ldq, ldk, ldv >= d_model (read only)
 *   O       : fp32, N x d_model, row stride ldo >= d_model; padding untouched
 * One fused kernel: scores in tensor memory, softmax in registers,
 * probabilities rounded to bf16 for the second product, fp32 accumulation.  Up
 * to 512 keys (the paper's sizes go up to N = 512, d_model = 512, h = 16) are
 * handled in one pass; longer sequences in blocks of 512 keys with a running
 * maximum, the accumulated row rescaled from block to block.
 * Limits: h divides d_model; d_k a multiple of 8, at most 32; Q, K, V 16-byte
 * aligned with ldq, ldk, ldv multiples of 8; O 4-byte aligned.  Shapes outside
 * these limits return CUDALLM_ERR_UNSUPPORTED_SHAPE.
 * N == 0 or d_model == 0 is a successful no-op.
 */
int cudallm_mhsa_bf16(const void *Q, const void *K, const void *V, void *O,
                      int64_t N, int64_t d_model, int64_t h,
                      int64_t ldq, int64_t ldk, int64_t ldv, int64_t ldo,
                      void *stream);

/*
 * Kernel variants (the candidate set of Algorithm 1's search).  A variant id is a number below
 * cudallm_num_variants().  Wherever a call takes a `variant`, it also takes a variant CODE: the
 * id plus two knobs that the search varies as well (cudallm_variant_code composes one):
 *   group_rows  0 = the library's rule, else a power of two <= 16384: the tiles are visited in
 *               raster groups of that many tile rows (what stays in L2 while B streams by);
 *   tail_parts  0 = the library's rule, else 2..7, for the tail-splitting ("_ts") variants only:
 *               the tiles of the ragged last wave are cut into up to that many parts along K.
 * cudallm_variant_code returns the code, or CUDALLM_ERR_INVALID_VARIANT.
 * cudallm_variant_name gives the variant's name for an id or a code (NULL if invalid).
 */
int cudallm_num_variants(void);
const char *cudallm_variant_name(int variant);
int cudallm_variant_code(int variant, int group_rows, int tail_parts);
/* 1 if `variant` can run the problem, 0 if not, negative status on bad args. */
int cudallm_variant_supports(int variant,
                             int64_t M, int64_t N, int64_t K,
                             int64_t lda, int64_t ldb, int64_t ldc,
                             int64_t batch, int out_dtype);
/* Variant the library would choose for this problem (host-side decision only;
 * no CUDA call; operand bases are assumed 16-byte aligned).  Returns a variant
 * id or a negative status. */
int cudallm_select_variant(int64_t M, int64_t N, int64_t K,
                           int64_t lda, int64_t ldb, int64_t ldc,
                           int64_t batch, int out_dtype);

/*
 * Dispatch table: the persisted outcome of the search (Algorithm 1's arg-min
 * over the valid candidates).  An entry says that `variant` (an id or a code) is
 * the fastest valid kernel for a shape (M, N, K, batch, out_dtype), or for a
 * shape CLASS: all shapes with the same ceil(M/128), ceil(N/64), ceil(K/64),
 * batch and out_dtype, on the same side of M <= 16 and M <= 64, whose operands
 * TMA can (tma_addressable != 0: 16-byte aligned bases, leading dimensions
 * multiples of 8) or cannot address -- every variant cuts all of them into the
 * same tiles and k-blocks.  cudallm_gemm_bf16, cudallm_gemm_bf16_batched,
 * cudallm_gemm_bf16_host and cudallm_select_variant look up the exact shape,
 * then its class, and use the entry if that variant can run the problem;
 * otherwise the cost model decides.
 * The tables are process-wide and hold at most 65536 entries each.  When the
 * library is first used the class table receives the winners of the search
 * recorded on a B200 and compiled into the library (the benchmark
 * configurations, the paper's Task 2 sizes and a grid of other shapes);
 * cudallm_dispatch_clear removes them too, cudallm_dispatch_load_packaged
 * enters them again.
 *   cudallm_dispatch_set / _set_class   add or replace an entry; variant == -1 removes it.
 *                           Errors: INVALID_DIM (a negative size), INVALID_DTYPE,
 *                           INVALID_VARIANT (not -1 and not a valid id or code),
 *                           TOO_LARGE (table full).
 *   cudallm_dispatch_get / _get_class   *variant = the entry's variant, or -1 if there is none.
 *                           Errors: as above, INVALID_POINTER (variant == NULL).
 *   cudallm_dispatch_clear  empties both tables; returns the number of entries they held.
 *   cudallm_dispatch_load_packaged      returns the number of entries entered.
 * Host-side only: no CUDA call.  Safe to call from several threads; a change is
 * seen by calls that start after it returns.
 */
int cudallm_dispatch_set(int64_t M, int64_t N, int64_t K, int64_t batch, int out_dtype, int variant);
int cudallm_dispatch_get(int64_t M, int64_t N, int64_t K, int64_t batch, int out_dtype, int *variant);
int cudallm_dispatch_set_class(int64_t M, int64_t N, int64_t K, int64_t batch, int out_dtype,
                               int tma_addressable, int variant);
int cudallm_dispatch_get_class(int64_t M, int64_t N, int64_t K, int64_t batch, int out_dtype,
                               int tma_addressable, int *variant);
int cudallm_dispatch_clear(void);
int cudallm_dispatch_load_packaged(void);

/*
 * Workspace.  Upper bound of the scratch bytes any variant may need for the
 * problem (repacked operands, split-K partial tiles and their flags).  Without
 * cudallm_set_workspace the library allocates (and grows) one workspace per
 * device with cudaMalloc on demand.  A caller-provided workspace must be
 * 256-byte aligned, zero-filled once before first use, and stay valid until
 * replaced; pass (NULL, 0) to return to the internal one.  It applies to the
 * device that is current at the time of the call.
 */
size_t cudallm_workspace_bytes(int64_t M, int64_t N, int64_t K,
                               int64_t lda, int64_t ldb, int64_t ldc,
                               int64_t batch, int out_dtype);
int cudallm_set_workspace(void *dev_ptr, size_t bytes);

/*
 * A workspace of its own for the calls made on `stream` (current device), so
 * that calls which need scratch (repacking, split-K, LayerNorm, the fp32
 * product) can run on several streams at once: flags, partial sums, repacked
 * operands and the status word of that stream's calls then live in `dev_ptr`.
 * Same requirements as cudallm_set_workspace: 256-byte aligned, at least
 * cudallm_workspace_bytes(...) for the products to come, zero-filled once,
 * valid until replaced or removed with (stream, NULL, 0); it may not overlap
 * another stream's workspace (CUDALLM_ERR_WORKSPACE).  A call whose needs
 * exceed it returns CUDALLM_ERR_WORKSPACE; it is never grown.
 * cudallm_device_status(stream, ...) reads this workspace's status word.
 * Attaching a workspace to a stream also tells the library that launches may
 * share the GPU: cudallm_gemm_bf16 / _batched on that stream choose only among
 * variants whose CTAs do not wait for one another (a forced split variant still
 * runs, with the caveat stated at the top of this file).
 */
int cudallm_set_workspace_for_stream(void *stream, void *dev_ptr, size_t bytes);

/*
 * Sizes the library's own workspace of the current device to at least `bytes`
 * now (cudaMalloc; synchronises the device if an older, smaller one has to be
 * replaced), so that later calls up to that need allocate nothing.  Returns
 * CUDALLM_ERR_WORKSPACE while a caller-provided workspace is set.
 */
int cudallm_reserve_workspace(size_t bytes);

/*
 * Releases what the library holds on every device: its own workspaces, the
 * streams and events of cudallm_gemm_bf16_host, and the stream-workspace table
 * (caller-provided buffers are only forgotten).  Synchronises those devices.
 * The library can be used again afterwards.
 */
int cudallm_shutdown(void);

/*
 * Test hooks for the bounded waits inside the kernels (host side; they change
 * how later launches are parameterised, nothing that has been enqueued).
 *   CUDALLM_DEBUG_WAIT_LIMIT_NS          value = the wall-clock limit of every
 *       in-kernel wait in nanoseconds (0 restores the default of 2 s).
 *   CUDALLM_DEBUG_MISS_NEXT_SPLIT_FLAGS  value != 0: the next launch that splits
 *       tiles along K (or the next one-pass cudallm_layernorm_f32 launch,
 *       whichever comes first) raises its hand-over flags to a value that
 *       nobody waits for, so every such wait runs out after the limit; the
 *       kernel then returns normally, its output is unspecified, and
 *       cudallm_device_status reports CUDALLM_ERR_DEVICE_TIMEOUT.  One launch only.
 *   CUDALLM_DEBUG_LAYERNORM_PATH         value = 0: cudallm_layernorm_f32 picks its
 *       kernel by size; 1: always the two-kernel path; 2: the one-pass kernel
 *       whenever the samples fit in shared memory, however small.
 * Returns CUDALLM_ERR_INVALID_VARIANT for an unknown `what` or value.
 */
#define CUDALLM_DEBUG_WAIT_LIMIT_NS          1
#define CUDALLM_DEBUG_MISS_NEXT_SPLIT_FLAGS  2
#define CUDALLM_DEBUG_LAYERNORM_PATH         3
int cudallm_debug_set(int what, unsigned long long value);

/*
 * Synchronises `stream`, then reads and clears the device status word that
 * kernels set when one of their bounded waits ran out.  *code is CUDALLM_OK or
 * CUDALLM_ERR_DEVICE_TIMEOUT, *detail identifies the wait (role and barrier).
 * Returns *code (or CUDALLM_ERR_CUDA if the synchronisation failed).
 */
int cudallm_device_status(void *stream, int *code, int *detail);

/* Text for a status code; for CUDALLM_ERR_CUDA includes the last CUDA error
 * text seen by the calling thread.  Never NULL. */
const char *cudallm_strerror(int status);

/* major*10000 + minor*100 + patch */
int cudallm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CUDALLM_GEMM_H */
