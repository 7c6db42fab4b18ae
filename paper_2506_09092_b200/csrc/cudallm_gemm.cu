// C ABI of the bf16 GEMM library: argument validation, variant table and
// selection, workspace, tensor-map encoding and kernel launches.
// See include/cudallm_gemm.h for the contract of every entry point.
#include "../../include/cudallm_gemm.h"
#include "../../include/cudallm_tasks.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <algorithm>
#include <cstring>
#include <atomic>
#include <mutex>
#include <unordered_map>

#include "aux_kernels.cuh"
#include "umma_gemm.cuh"
#include "umma_gemm_2cta.cuh"
#include "umma_tf32.cuh"
#include "mhsa.cuh"
#include "hbm_tasks.cuh"

using namespace cudallm;

namespace {

// ------------------------------------------------------------------ errors --
thread_local char g_cuda_err[256] = "";

int cuda_fail(cudaError_t e, const char *where)
{
    snprintf(g_cuda_err, sizeof g_cuda_err, "%s: %s", where, cudaGetErrorString(e));
    return CUDALLM_ERR_CUDA;
}
#define CUDA_TRY(expr)                                          \
    do {                                                        \
        cudaError_t e__ = (expr);                               \
        if (e__ != cudaSuccess) return cuda_fail(e__, #expr);   \
    } while (0)

// ----------------------------------------------------------------- problem --
struct Problem {
    const void *A, *B;
    void *C;
    int64_t M, N, K, lda, ldb, ldc, sA, sB, sC, batch;
    int out_dtype;
};

constexpr int64_t kMaxDim = (int64_t(1) << 31) - 1024;   // kernels index tiles with int
constexpr int64_t kMaxElems = int64_t(1) << 46;          // per operand, keeps byte offsets < 2^48

int validate(const Problem &p)
{
    if (p.out_dtype != CUDALLM_F32 && p.out_dtype != CUDALLM_BF16) return CUDALLM_ERR_INVALID_DTYPE;
    if (p.M < 0 || p.N < 0 || p.K < 0 || p.batch < 0) return CUDALLM_ERR_INVALID_DIM;
    if (p.M > kMaxDim || p.N > kMaxDim || p.K > kMaxDim || p.batch > kMaxDim)
        return CUDALLM_ERR_INVALID_DIM;
    if (p.M == 0 || p.N == 0 || p.batch == 0) return CUDALLM_OK;   // nothing to do
    if (p.lda < p.K || p.ldb < p.N || p.ldc < p.N) return CUDALLM_ERR_INVALID_LD;
    if (p.lda > kMaxElems || p.ldb > kMaxElems || p.ldc > kMaxElems) return CUDALLM_ERR_INVALID_DIM;
    if (p.batch > 1) {
        if (p.sA < 0 || p.sB < 0 || p.sC < 0) return CUDALLM_ERR_INVALID_LD;
        if (p.sC < (p.M - 1) * p.ldc + p.N) return CUDALLM_ERR_INVALID_LD;   // items of C overlap
    }
    // extents must stay indexable
    const long double extA = (long double)(p.batch - 1) * p.sA + (long double)(p.M - 1) * p.lda + p.K;
    const long double extB = (long double)(p.batch - 1) * p.sB + (long double)(p.K > 0 ? p.K - 1 : 0) * p.ldb + p.N;
    const long double extC = (long double)(p.batch - 1) * p.sC + (long double)(p.M - 1) * p.ldc + p.N;
    if (extA > (long double)kMaxElems || extB > (long double)kMaxElems || extC > (long double)kMaxElems)
        return CUDALLM_ERR_INVALID_DIM;
    if ((long double)p.M * p.N * p.batch > (long double)kMaxElems) return CUDALLM_ERR_INVALID_DIM;
    if (!p.C) return CUDALLM_ERR_INVALID_POINTER;
    if (p.K > 0 && (!p.A || !p.B)) return CUDALLM_ERR_INVALID_POINTER;
    if (p.K > 0 && ((reinterpret_cast<uintptr_t>(p.A) & 1) || (reinterpret_cast<uintptr_t>(p.B) & 1)))
        return CUDALLM_ERR_MISALIGNED;
    const uintptr_t cmask = (p.out_dtype == CUDALLM_F32) ? 3 : 1;
    if (reinterpret_cast<uintptr_t>(p.C) & cmask) return CUDALLM_ERR_MISALIGNED;
    return CUDALLM_OK;
}

inline bool is_empty(const Problem &p) { return p.M == 0 || p.N == 0 || p.batch == 0; }

// ---------------------------------------------------------------- variants --
enum Family { kSimt = 0, kUmma = 1, kUmmaPair = 2 };
constexpr int kTailSplit = 0;          // Variant::split_k value: split only the tiles of the ragged last wave
struct Variant {
    char name[32];
    Family family;
    int block_n;
    int split_k;                       // 1 = none, 2..16 = every tile along K, kTailSplit = see above
    int per_sm;                        // CTAs per SM: 1, or 2 for the two-stage kernels for short K
    int alt_ring;                      // 1: the other arrangement of the shared-memory ring (see build_variants)
};
constexpr int kBlockNs[3] = {64, 128, 256};
constexpr int kSplits[6] = {1, 2, 4, 8, 16, kTailSplit};
constexpr int kNumVariants = 1 + 3 * 6 + 6 + 2 + 6;
Variant g_variants[kNumVariants];

// A variant code as the entry points take it: the variant id in the low 8 bits; above it two
// knobs that the search varies and the dispatch table records, 0 meaning "the library's rule":
//   bits 8..11  raster group height: g > 0 asks for groups of 2^(g-1) tile rows
//   bits 12..14 tail split: t >= 2 cuts the tiles of the ragged last wave into up to t parts
//               (at least 4 k-blocks each) instead of up to 4 parts of at least 8
inline int code_base(int code) { return code & 0xFF; }
inline int code_group(int code) { return (code >> 8) & 0xF; }
inline int code_tail(int code) { return (code >> 12) & 0x7; }
inline bool code_valid(int code)
{
    return code >= 0 && (code >> 15) == 0 && code_base(code) < kNumVariants && code_tail(code) != 1;
}
std::once_flag g_variants_once;

void name_variant(Variant &v, const char *stem, int bn, int sk)
{
    if (sk == 1) snprintf(v.name, sizeof v.name, "%s_n%d", stem, bn);
    else if (sk == kTailSplit) snprintf(v.name, sizeof v.name, "%s_n%d_ts", stem, bn);
    else snprintf(v.name, sizeof v.name, "%s_n%d_sk%d", stem, bn, sk);
}

int load_packaged_entries();
std::once_flag g_packaged_once;
void build_variants()
{
    std::call_once(g_variants_once, [] {
        snprintf(g_variants[0].name, sizeof g_variants[0].name, "simt");
        g_variants[0].family = kSimt;
        g_variants[0].block_n = 0;
        g_variants[0].split_k = 1;
        int v = 1;
        for (int bn : kBlockNs)
            for (int sk : kSplits) {
                name_variant(g_variants[v], "umma", bn, sk);
                g_variants[v].family = kUmma;
                g_variants[v].block_n = bn;
                g_variants[v].split_k = sk;
                ++v;
            }
        // CTA pairs (cta_group::2), 256 x 256 tile per pair
        for (int sk : kSplits) {
            name_variant(g_variants[v], "umma2", 256, sk);
            g_variants[v].family = kUmmaPair;
            g_variants[v].block_n = 256;
            g_variants[v].split_k = sk;
            ++v;
        }
        // Two CTAs per SM, each with a two-stage ring and half of tensor memory: for
        // batches of products with one or two k-blocks, where a CTA's time goes into the
        // first load's latency and the epilogue, and a second CTA fills those gaps.
        for (int bn : {64, 128}) {
            snprintf(g_variants[v].name, sizeof g_variants[v].name, "umma_n%d_x2", bn);
            g_variants[v].family = kUmma;
            g_variants[v].block_n = bn;
            g_variants[v].split_k = 1;
            g_variants[v].per_sm = 2;
            ++v;
        }
        // The other arrangement of the same shared memory: one barrier round trip per two
        // k-blocks where the standard kernel has one per k-block (256-column tiles), or per
        // k-block where it has one per two (128-column tiles, CTA pairs).  Which one is faster
        // depends on whether the MMA thread or the load latency bounds the shape: the search decides.
        for (int bn : {128, 256})
            for (int sk : {1, kTailSplit}) {
                snprintf(g_variants[v].name, sizeof g_variants[v].name, "umma_n%d_%s%s", bn, bn == 256 ? "k2" : "k1",
                         sk == kTailSplit ? "_ts" : "");
                g_variants[v].family = kUmma;
                g_variants[v].block_n = bn;
                g_variants[v].split_k = sk;
                g_variants[v].alt_ring = 1;
                ++v;
            }
        for (int sk : {1, kTailSplit}) {
            snprintf(g_variants[v].name, sizeof g_variants[v].name, "umma2_n256_k1%s", sk == kTailSplit ? "_ts" : "");
            g_variants[v].family = kUmmaPair;
            g_variants[v].block_n = 256;
            g_variants[v].split_k = sk;
            g_variants[v].alt_ring = 1;
            ++v;
        }
        for (int i = 0; i < kNumVariants; ++i)
            if (g_variants[i].per_sm == 0) g_variants[i].per_sm = 1;
    });
    // the dispatch table starts out with the packaged winners of the search
    std::call_once(g_packaged_once, [] { load_packaged_entries(); });
}

constexpr int kNumSMs = 148;
constexpr int64_t kMaxPartialBytes = int64_t(1) << 30;   // split-K scratch a variant may ask for
constexpr int64_t kMaxHelperTiles = 65536;               // helper partial tiles per launch (4 flags each)

inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int64_t round_up(int64_t a, int64_t b) { return cdiv(a, b) * b; }

// How a variant cuts a problem into units.
struct Tiling {
    int64_t tiles_m, tiles_n, tiles, kblocks;
    int64_t dp_tiles;        // leading tiles that are one unit each
    int split;               // K parts per remaining tile
    int64_t units;           // dp_tiles + (tiles - dp_tiles) * split
    int64_t helper_tiles;    // partial tiles in the workspace: (tiles - dp_tiles) * split * CTAs per tile
    int64_t partial_bytes;
};

// `slots` = units that run at once (CTAs, or CTA pairs, of the persistent grid); `tail` = the
// tail-split knob of the variant code (0 = the default rule).
Tiling tiling_for(const Variant &v, const Problem &p, int slots, int tail = 0)
{
    const bool pair = v.family == kUmmaPair;
    Tiling t{};
    if (v.family == kSimt) return t;                  // no tiles, no scratch
    t.tiles_m = cdiv(p.M, pair ? kPairM : kBlockM);
    t.tiles_n = cdiv(p.N, v.block_n);
    t.tiles = t.tiles_m * t.tiles_n * p.batch;
    t.kblocks = cdiv(p.K, kBlockK);
    t.split = 1;
    t.dp_tiles = t.tiles;
    if (v.split_k == kTailSplit) {
        // Split the tiles of the ragged last wave along K so that they fill the
        // grid about once: up to 4 parts, each at least 8 k-blocks deep.
        const int64_t left = t.tiles % slots;
        int64_t parts = left > 0 ? slots / left : 1;
        const int64_t max_parts = tail >= 2 ? tail : 4, min_depth = tail >= 2 ? 4 : 8;
        if (parts > max_parts) parts = max_parts;
        while (parts > 1 && t.kblocks / parts < min_depth) --parts;
        if (parts > 1) {
            t.split = (int)parts;
            t.dp_tiles = t.tiles - left;
        }
    } else if (v.split_k > 1) {
        t.split = v.split_k;
        t.dp_tiles = 0;
    }
    t.units = t.dp_tiles + (t.tiles - t.dp_tiles) * t.split;
    t.helper_tiles = t.split > 1 ? (t.tiles - t.dp_tiles) * t.split * (pair ? 2 : 1) : 0;
    t.partial_bytes = t.helper_tiles * int64_t(kBlockM) * v.block_n * 4;
    return t;
}
inline int default_slots(const Variant &v)
{
    return v.family == kUmmaPair ? kNumSMs / 2 : kNumSMs * (v.per_sm == 2 ? 2 : 1);
}

bool variant_supports(const Variant &v, const Problem &p)
{
    if (is_empty(p)) return true;
    if (v.family == kSimt) return true;
    if (p.K == 0) return false;                       // the zero-fill case runs on the simt kernel
    const Tiling t = tiling_for(v, p, default_slots(v));
    if (t.units > kMaxDim) return false;
    if (v.split_k > 1 && v.split_k > t.kblocks) return false;
    // bounds that must hold for any grid size the device may give
    // (tail-split variants have at most one grid's worth of helper tiles)
    if (v.split_k > 1 && (t.helper_tiles > kMaxHelperTiles || t.partial_bytes > kMaxPartialBytes))
        return false;
    return true;
}

constexpr double kPairClocksPerKBlock = 455.0;       // 256 x 256 x 64 on a CTA pair (measured: 0.89 x a lone CTA's 128 x 256 x 64)

// Cost model (SM clocks) behind the automatic choice: the larger of
//  compute: rounds of units x k-blocks per unit x clocks per k-block (measured
//      on 4096^3: about 300 + 0.83 * BLOCK_N for a lone CTA, 540 for a pair),
//      plus one exposed epilogue; a split tile's owner also reads its helpers'
//      partial tiles from L2;
//  memory: A and B read once, C written once (partial tiles stay in L2), over
//      the bandwidth the active SMs can draw (about 40 B/clock each), capped
//      by HBM.
double variant_cost(const Variant &v, const Problem &p)
{
    const bool pair = v.family == kUmmaPair;
    const int slots = default_slots(v);
    const Tiling t = tiling_for(v, p, slots);
    // (the two-stage ring of the two-per-SM kernels cannot hide load latency: measured 2x on C5a)
    const double per_kb = pair ? kPairClocksPerKBlock : (300.0 + 0.83 * v.block_n) * (v.per_sm == 2 ? 2.2 : 1.0);
    const double rows = p.M < kBlockM ? (double)p.M : (double)kBlockM;
    const double out_b = (p.out_dtype == CUDALLM_F32) ? 4.0 : 2.0;
    const double epi = rows * v.block_n * out_b / 32.0 + 1500.0;
    const double full_main = (double)t.kblocks * per_kb;
    const double dp_rounds = (double)cdiv(t.dp_tiles, slots);
    double compute = dp_rounds * (full_main > epi ? full_main : epi);
    if (t.split > 1) {
        const double split_units = (double)(t.tiles - t.dp_tiles) * t.split;
        const double rounds = (double)cdiv((int64_t)split_units, slots);
        const double part_main = (double)cdiv(t.kblocks, t.split) * per_kb;
        // exchange of partial chunks between the units of a tile: each unit writes
        // and reads (S-1)/S of a tile through L2; measured ~2.4 us for two units of a
        // 128 x 128 tile, growing with the number of partners and the size of the tile
        const double fix = 2000.0 + (t.split - 1) * (1500.0 + rows * v.block_n * 4.0 / 64.0);
        compute += rounds * (part_main + fix);
    }
    compute += epi;
    const double hbm = 3500.0;                         // bytes per clock: ~6.5 TB/s at ~1.9 GHz
    const double active = (pair ? 2.0 : 1.0) * (t.units < slots ? (double)t.units : (double)slots);
    const double bw = active * 40.0 < hbm ? active * 40.0 : hbm;
    const double bytes = (double)p.batch * (2.0 * p.M * p.K + 2.0 * p.K * p.N + out_b * p.M * p.N);
    const double memory = bytes / bw;
    return (compute > memory ? compute : memory) + 4000.0;
}

// Dispatch table: what a search recorded (cudallm_dispatch_set / _set_class).  Two levels: an
// entry for the exact shape, and an entry for the shape's class -- all shapes that every
// variant cuts into the same tiles and k-blocks (same ceil(M / 128), ceil(N / 64), ceil(K / 64),
// batch and output type, same side of the short-A limits M <= 16 and M <= 64, operands
// addressable by TMA or not): the kernels do the same work on all of them.
struct DispatchKey {
    int64_t M, N, K, batch;
    int out_dtype;
    bool operator==(const DispatchKey &o) const
    {
        return M == o.M && N == o.N && K == o.K && batch == o.batch && out_dtype == o.out_dtype;
    }
};
struct DispatchHash {
    size_t operator()(const DispatchKey &k) const
    {
        uint64_t h = 0x9E3779B97F4A7C15ull;
        for (uint64_t x : {(uint64_t)k.M, (uint64_t)k.N, (uint64_t)k.K, (uint64_t)k.batch, (uint64_t)k.out_dtype})
            h = (h ^ x) * 0x100000001B3ull + (h >> 29);
        return (size_t)h;
    }
};
// The class of a shape, written as a key of the same type: tile counts in place of sizes; the
// short-A bucket and the alignment flag are folded into the M and out_dtype fields.
DispatchKey class_key(int64_t M, int64_t N, int64_t K, int64_t batch, int out_dtype, bool aligned)
{
    const int64_t mt = (M + 127) / 128;
    const int64_t bucket = M <= 16 ? 0 : M <= 64 ? 1 : 2;
    return DispatchKey{mt * 4 + (mt == 1 ? bucket : 3), (N + 63) / 64, (K + 63) / 64, batch,
                       out_dtype + (aligned ? 0 : 2)};
}
constexpr size_t kMaxDispatchEntries = 65536;
std::unordered_map<DispatchKey, int, DispatchHash> g_dispatch, g_dispatch_class;
std::mutex g_dispatch_mutex;
std::atomic<uint64_t> g_dispatch_generation{0};      // bumped by every change of the tables

inline bool a_operand_aligned(const Problem &p);
inline bool b_operand_aligned(const Problem &p);

// `no_waits`: only variants whose CTAs never wait for one another (no split tiles), for
// calls that may share the GPU with other launches of this library.  Returns a variant code.
int select_variant_uncached(const Problem &p, bool no_waits)
{
    build_variants();
    if (is_empty(p) || p.K == 0) return 0;
    {
        std::lock_guard<std::mutex> lock(g_dispatch_mutex);
        auto usable = [&](int code) {
            const Variant &v = g_variants[code_base(code)];
            return variant_supports(v, p) && !(no_waits && v.split_k != 1);
        };
        const auto it = g_dispatch.find(DispatchKey{p.M, p.N, p.K, p.batch, p.out_dtype});
        if (it != g_dispatch.end() && usable(it->second)) return it->second;
        if (!g_dispatch_class.empty()) {
            const bool aligned = a_operand_aligned(p) && b_operand_aligned(p);
            const auto ic = g_dispatch_class.find(class_key(p.M, p.N, p.K, p.batch, p.out_dtype, aligned));
            if (ic != g_dispatch_class.end() && usable(ic->second)) return ic->second;
        }
    }
    int best = -1;
    double best_cost = 0;
    for (int v = 1; v < kNumVariants; ++v) {
        if (g_variants[v].alt_ring) continue;          // the model does not tell the rings apart: the search does
        if (no_waits && g_variants[v].split_k != 1) continue;
        if (!variant_supports(g_variants[v], p)) continue;
        const double c = variant_cost(g_variants[v], p);
        if (best < 0 || c < best_cost) { best = v; best_cost = c; }
    }
    return best < 0 ? 0 : best;
}

// The choice depends only on the shape, the operands' alignment class and the dispatch
// tables; repeated calls with the same shape (the common case) reuse the previous answer.
int select_variant(const Problem &p, bool no_waits = false)
{
    struct Last { int64_t M, N, K, batch; int out_dtype, variant; uint64_t generation; bool no_waits, aligned; };
    static thread_local Last last = {-1, -1, -1, -1, -1, 0, 0, false, false};
    const uint64_t gen = g_dispatch_generation.load(std::memory_order_acquire);
    const bool aligned = a_operand_aligned(p) && b_operand_aligned(p);
    if (last.M == p.M && last.N == p.N && last.K == p.K && last.batch == p.batch
        && last.out_dtype == p.out_dtype && last.generation == gen && last.no_waits == no_waits
        && last.aligned == aligned)
        return last.variant;
    const int v = select_variant_uncached(p, no_waits);
    last = Last{p.M, p.N, p.K, p.batch, p.out_dtype, v, gen, no_waits, aligned};
    return v;
}

// --------------------------------------------------------------- workspace --
// Layout: [status 256 B][split-K flags][LayerNorm entries][split-K partial tiles][packed A][packed B]
// The two areas of the header are kept apart because of what their words may hold: a flag word
// is zero or the epoch of some launch, and a kernel takes it for raised when it equals ITS
// epoch; an entry word is a 32-bit payload (any bits) under a 32-bit epoch tag.  A payload
// left behind in a flag word could one day equal the epoch of a later launch.
constexpr size_t kFlagBytes = kMaxHelperTiles * 4 * sizeof(int);
constexpr size_t kEntryBytes = size_t(1) << 20;      // the persistent LayerNorm kernel's exchange area
constexpr size_t kEntryOffset = 256 + kFlagBytes;
constexpr size_t kHeaderBytes = kEntryOffset + kEntryBytes;   // zeroed when a workspace is created
constexpr int kMaxDevices = 64;

// A workspace: the device's default one (allocated and grown by the library unless the
// caller set one) or one that the caller attached to a stream.
struct Workspace {
    void *ptr = nullptr;         // active buffer
    size_t bytes = 0;
    bool external = false;       // the caller's: never grown or freed here
    void *internal = nullptr;    // owned allocation (kept while an external one is set)
    size_t internal_bytes = 0;
};

struct DeviceState {
    bool probed = false;
    bool supported = false;
    int sm_count = 0;
    Workspace ws;                // the device's default workspace
    std::unordered_map<cudaStream_t, Workspace> stream_ws;   // cudallm_set_workspace_for_stream
    bool smem_attr_set[40] = {};
    bool layernorm_attr_set = false;
    bool tf32_attr_set = false;
    int max_pairs = 0;           // co-resident 2-CTA clusters of the pair kernel (0 = not asked yet)
    int epoch = 0;               // last split-K flag value used on this device
};
DeviceState g_dev[kMaxDevices];
std::mutex g_mutex;

// Host-side knobs of the kernels' bounded waits (cudallm_debug_set): the limit itself, and a
// one-shot request to raise the split-K flags of the next split launch to a value nobody
// waits for, so that every such wait runs out (the self-test of the timeout path).
std::atomic<unsigned long long> g_wait_limit_ns{kWaitLimitNs};
std::atomic<int> g_skew_next_flags{0};
std::atomic<int> g_layernorm_path{0};      // 0 = by size, 1 = always the two-kernel path, 2 = one-pass whenever it fits

// The workspace calls on `stream` use: the one attached to the stream, else the device's.
Workspace &workspace_for(DeviceState &d, cudaStream_t stream)
{
    if (!d.stream_ws.empty()) {
        const auto it = d.stream_ws.find(stream);
        if (it != d.stream_ws.end()) return it->second;
    }
    return d.ws;
}
bool stream_has_workspace(DeviceState &d, cudaStream_t stream)
{
    return !d.stream_ws.empty() && d.stream_ws.find(stream) != d.stream_ws.end();
}

// Streams and events of the host-buffer entry point (created on first use).
constexpr int kHostPipeChunks = 4;
struct HostPipe {
    bool ready = false;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t arrived[kHostPipeChunks] = {}, computed[kHostPipeChunks] = {};
    cudaEvent_t start = nullptr, done = nullptr;
};
HostPipe g_host_pipe[kMaxDevices];

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int probe_device(int dev)
{
    DeviceState &d = g_dev[dev];
    if (d.probed) return d.supported ? CUDALLM_OK : CUDALLM_ERR_UNSUPPORTED_DEVICE;
    int major = 0, minor = 0, sms = 0;
    CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    CUDA_TRY(cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev));
    CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    d.supported = (major == 10 && minor == 0);
    d.sm_count = sms;
    if (!d.supported) {
        d.probed = true;
        return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    }
    if (!g_encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        if (qres != cudaDriverEntryPointSuccess || !fn) {
            snprintf(g_cuda_err, sizeof g_cuda_err, "cuTensorMapEncodeTiled not available");
            return CUDALLM_ERR_CUDA;
        }
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    d.probed = true;                 // only now: a failed look-up above is retried by the next call
    return CUDALLM_OK;
}

// Make sure workspace `w` holds `bytes`; allocates or grows an internal one (never a
// caller-provided one).  `exact`: allocate just `bytes` (cudallm_reserve_workspace).
int ensure_workspace(Workspace &w, size_t bytes, cudaStream_t stream, bool exact = false)
{
    if (w.ptr && w.bytes >= bytes) return CUDALLM_OK;
    if (w.external) return CUDALLM_ERR_WORKSPACE;
    size_t want = exact ? bytes : (bytes < (size_t(8) << 20) ? (size_t(8) << 20) : bytes + bytes / 4);
    if (want < kHeaderBytes) want = kHeaderBytes;
    if (w.internal) {
        CUDA_TRY(cudaDeviceSynchronize());            // earlier launches may still use it
        CUDA_TRY(cudaFree(w.internal));
        w.internal = nullptr;
        w.internal_bytes = 0;
        w.ptr = nullptr;
        w.bytes = 0;
    }
    void *ptr = nullptr;
    CUDA_TRY(cudaMalloc(&ptr, want));
    CUDA_TRY(cudaMemsetAsync(ptr, 0, kHeaderBytes, stream));
    // later launches on other streams must see the cleared header
    CUDA_TRY(cudaStreamSynchronize(stream));
    w.internal = ptr;
    w.internal_bytes = want;
    w.ptr = ptr;
    w.bytes = want;
    return CUDALLM_OK;
}

struct Plan {
    bool pack_a, pack_b;
    int64_t ldap, ldbp, sAp, sBp;      // packed leading dimensions / strides (elements)
    size_t off_partials, off_pack_a, off_pack_b, total;
};

inline bool a_operand_aligned(const Problem &p)
{
    return (reinterpret_cast<uintptr_t>(p.A) % 16 == 0) && (p.lda % 8 == 0)
        && (p.batch == 1 || p.sA % 8 == 0);
}
inline bool b_operand_aligned(const Problem &p)
{
    return (reinterpret_cast<uintptr_t>(p.B) % 16 == 0) && (p.ldb % 8 == 0)
        && (p.batch == 1 || p.sB % 8 == 0);
}

Plan make_plan(const Tiling &t, const Problem &p, bool pack_a, bool pack_b)
{
    Plan pl{};
    pl.pack_a = pack_a;
    pl.pack_b = pack_b;
    size_t off = kHeaderBytes;
    pl.off_partials = off;
    off += (size_t)t.partial_bytes;
    off = (size_t)round_up((int64_t)off, 256);
    pl.off_pack_a = off;
    pl.ldap = round_up(p.K, 8);
    pl.sAp = p.M * pl.ldap;
    if (pack_a) off += (size_t)(p.batch * pl.sAp * 2);
    off = (size_t)round_up((int64_t)off, 256);
    pl.off_pack_b = off;
    pl.ldbp = round_up(p.N, 8);
    pl.sBp = p.K * pl.ldbp;
    if (pack_b) off += (size_t)(p.batch * pl.sBp * 2);
    pl.total = (size_t)round_up((int64_t)off, 256);
    return pl;
}

// ------------------------------------------------------------- tensor maps --
// Encoding a tensor map costs about a microsecond on the host, which is a large
// share of a small GEMM; the last few are kept and reused when the same operand
// (same base, extents, strides and box) comes back.  Called with g_mutex held.
struct MapKey {
    const void *base;
    int64_t inner, rows, batch, ld, stride;
    int box_inner, box_rows;
    int kind;                              // 0 = bf16 operand, 1 = fp32 C, 2 = bf16 C
    bool operator==(const MapKey &o) const
    {
        return base == o.base && inner == o.inner && rows == o.rows && batch == o.batch && ld == o.ld
            && stride == o.stride && box_inner == o.box_inner && box_rows == o.box_rows && kind == o.kind;
    }
};
constexpr int kMapCacheSize = 16;
struct MapCache {
    MapKey key[kMapCacheSize] = {};
    CUtensorMap map[kMapCacheSize];
    bool used[kMapCacheSize] = {};
    int next = 0;
};
MapCache g_map_cache[kMaxDevices];

// kind 0: a bf16 operand read in 128-byte-swizzled boxes; kind 1 / 2: fp32 / bf16
// C written in boxes of 32 columns x 32 rows (128- / 64-byte swizzle).
int encode_map(int dev, CUtensorMap *tm, const void *base, int64_t inner, int64_t rows, int64_t batch,
               int64_t ld, int64_t stride, int box_inner, int box_rows, int kind)
{
    MapCache &mc = g_map_cache[dev];
    const MapKey k{base, inner, rows, batch, ld, batch > 1 ? stride : 0, box_inner, box_rows, kind};
    for (int i = 0; i < kMapCacheSize; ++i)
        if (mc.used[i] && mc.key[i] == k) {
            *tm = mc.map[i];
            return CUDALLM_OK;
        }
    const cuuint64_t es = (kind == 1 || kind == 3) ? 4 : 2;      // kinds: 0 bf16, 1 fp32, 2 bf16 with a 64-byte swizzle,
                                                                 // 3 fp32 with the 128-byte swizzle on 32-byte units
    cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)batch};
    cuuint64_t item_stride = (batch > 1) ? (cuuint64_t)stride * es : (cuuint64_t)rows * ld * es;
    cuuint64_t strides[2] = {(cuuint64_t)ld * es, item_stride};
    cuuint32_t box[3] = {(cuuint32_t)box_inner, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(tm, (kind == 1 || kind == 3) ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                          const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          kind == 2 ? CU_TENSOR_MAP_SWIZZLE_64B
                                    : kind == 3 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                          kind == 0 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_cuda_err, sizeof g_cuda_err, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return CUDALLM_ERR_CUDA;
    }
    const int slot = mc.next;
    mc.next = (mc.next + 1) % kMapCacheSize;
    mc.key[slot] = k;
    mc.map[slot] = *tm;
    mc.used[slot] = true;
    return CUDALLM_OK;
}
int encode_operand_map(int dev, CUtensorMap *tm, const void *base, int64_t inner, int64_t rows,
                       int64_t batch, int64_t ld, int64_t stride, int box_inner, int box_rows)
{
    return encode_map(dev, tm, base, inner, rows, batch, ld, stride, box_inner, box_rows, 0);
}
// Tensor map of C for the epilogue's stores; all zero (and unused) when C's
// alignment does not allow TMA.
int encode_c_map(int dev, CUtensorMap *tm, const Problem &p, bool c_tma)
{
    if (!c_tma) {
        memset(tm, 0, sizeof *tm);
        return CUDALLM_OK;
    }
    return encode_map(dev, tm, p.C, p.N, p.M, p.batch, p.ldc, p.sC, 32, 32, p.out_dtype == CUDALLM_F32 ? 1 : 2);
}

// ---------------------------------------------------------------- launches --
// Launch of a plain kernel with programmatic stream serialisation (the kernel calls
// griddepcontrol.wait before it touches global memory): its launch latency hides behind the
// previous kernel of the stream.
template <typename... KArgs, typename... Args>
int launch_serialised(void (*kernel)(KArgs...), unsigned grid, unsigned block, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
    return CUDALLM_OK;
}

// The same for a kernel with a two-dimensional grid and dynamic shared memory.
template <typename... KArgs, typename... Args>
int launch_serialised_smem(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem_bytes, cudaStream_t stream,
                           Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
    return CUDALLM_OK;
}

// Launch with programmatic stream serialisation: the kernel may begin while the
// previous kernel of the stream drains; it waits (griddepcontrol.wait) before it
// touches global memory.
template <typename Kernel>
int launch_overlapped(Kernel kernel, int grid, int smem_bytes, cudaStream_t stream, const CUtensorMap &ta,
                      const CUtensorMap &tb, const CUtensorMap &tc, const GemmParams &gp)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kNumThreads);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, ta, tb, tc, gp));
    return CUDALLM_OK;
}

template <int BLOCK_N, int STAGES, int KSUB, bool OUT_BF16, int A_ROWS = kBlockM>
int launch_umma(int dev, int slot, const CUtensorMap &ta, const CUtensorMap &tb, const CUtensorMap &tc,
                const GemmParams &gp,
                cudaStream_t stream)
{
    using L = SmemLayout<BLOCK_N, STAGES, KSUB, A_ROWS>;
    static_assert(L::kDynamicBytes <= 232448, "shared memory budget");
    // Either more than half of an SM's shared memory, so two CTAs (and their tensor
    // memory allocations) can never share an SM, or small enough that exactly two fit,
    // each with at most half of tensor memory.
    constexpr bool kTwoPerSm = L::kDynamicBytes <= 112 * 1024;
    static_assert(L::kDynamicBytes > 120 * 1024 || (kTwoPerSm && 3 * L::kDynamicBytes > 233472 && BLOCK_N <= 128),
                  "one or exactly two CTAs per SM");
    auto kernel = umma_gemm_kernel<BLOCK_N, STAGES, KSUB, OUT_BF16, A_ROWS>;
    DeviceState &d = g_dev[dev];
    if (!d.smem_attr_set[slot]) {
        CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      L::kDynamicBytes));
        d.smem_attr_set[slot] = true;
    }
    const int cap = kTwoPerSm ? 2 * d.sm_count : d.sm_count;
    int grid = gp.num_units < cap ? gp.num_units : cap;
    return launch_overlapped(kernel, grid, L::kDynamicBytes, stream, ta, tb, tc, gp);
}

// Sets the pair kernel's shared-memory attribute and asks how many CTA pairs
// the device can hold at once (the persistent grid of the pair kernels).
template <int STAGES, int KSUB, bool OUT_BF16>
int prepare_umma_pair(int dev, int slot)
{
    using L = PairSmemLayout<STAGES, KSUB>;
    static_assert(L::kDynamicBytes <= 232448, "shared memory budget");
    static_assert(L::kDynamicBytes > 120 * 1024, "one CTA per SM");
    auto kernel = umma_gemm_2cta_kernel<STAGES, KSUB, OUT_BF16>;
    DeviceState &d = g_dev[dev];
    if (!d.smem_attr_set[slot]) {
        CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      L::kDynamicBytes));
        d.smem_attr_set[slot] = true;
    }
    if (d.max_pairs == 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * (d.sm_count / 2));
        cfg.blockDim = dim3(kNumThreads);
        cfg.dynamicSmemBytes = L::kDynamicBytes;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, kernel, &cfg));
        d.max_pairs = n > 0 ? n : 1;
        if (d.max_pairs > d.sm_count / 2) d.max_pairs = d.sm_count / 2;
    }
    return CUDALLM_OK;
}

template <int STAGES, int KSUB, bool OUT_BF16>
int launch_umma_pair(int dev, const CUtensorMap &ta, const CUtensorMap &tb, const CUtensorMap &tc,
                const GemmParams &gp,
                     cudaStream_t stream)
{
    using L = PairSmemLayout<STAGES, KSUB>;
    auto kernel = umma_gemm_2cta_kernel<STAGES, KSUB, OUT_BF16>;
    DeviceState &d = g_dev[dev];
    const int pairs = gp.num_units < d.max_pairs ? gp.num_units : d.max_pairs;
    return launch_overlapped(kernel, 2 * pairs, L::kDynamicBytes, stream, ta, tb, tc, gp);
}

int launch_simt(const Problem &p, cudaStream_t stream)
{
    dim3 block(256);
    int64_t gy = cdiv(p.M, 16), gz = p.batch;
    dim3 grid((unsigned)cdiv(p.N, 16), (unsigned)(gy > 65535 ? 65535 : gy), (unsigned)(gz > 65535 ? 65535 : gz));
    const __nv_bfloat16 *A = static_cast<const __nv_bfloat16 *>(p.A);
    const __nv_bfloat16 *B = static_cast<const __nv_bfloat16 *>(p.B);
    if (p.out_dtype == CUDALLM_BF16)
        simt_gemm_kernel<true><<<grid, block, 0, stream>>>(A, B, p.C, (int)p.M, (int)p.N, (int)p.K, p.lda,
                                                           p.ldb, p.ldc, p.sA, p.sB, p.sC, (int)p.batch);
    else
        simt_gemm_kernel<false><<<grid, block, 0, stream>>>(A, B, p.C, (int)p.M, (int)p.N, (int)p.K, p.lda,
                                                            p.ldb, p.ldc, p.sA, p.sB, p.sC, (int)p.batch);
    CUDA_TRY(cudaGetLastError());
    return CUDALLM_OK;
}

PackJob pack_job(const void *src, void *dst, int64_t rows, int64_t cols, int64_t ld_src, int64_t ld_dst,
                 int64_t s_src, int64_t s_dst, int64_t batch)
{
    PackJob j{};
    j.src = static_cast<const uint16_t *>(src);
    j.dst = static_cast<uint16_t *>(dst);
    j.rows = (int)rows; j.cols = (int)cols; j.batch = (int)batch;
    j.ld_src = ld_src; j.ld_dst = ld_dst; j.stride_src = s_src; j.stride_dst = s_dst;
    j.total_rows = rows * batch;
    return j;
}

// One launch repacks both jobs (either may be empty: total_rows == 0).
int launch_pack(const PackJob &a, const PackJob &b, cudaStream_t stream)
{
    const int64_t units = a.total_rows * cdiv(a.cols, 512) + b.total_rows * cdiv(b.cols, 512);
    if (units == 0) return CUDALLM_OK;
    int64_t blocks = cdiv(units, kPackThreads / 32);     // one warp per 512 elements of a row, grid-stride
    if (blocks > kNumSMs * 8) blocks = kNumSMs * 8;
    return launch_serialised(pack_rows_kernel, (unsigned)blocks, kPackThreads, stream, a, b);
}

// Launches the tcgen05 kernel of variant `v` (lone CTAs or CTA pairs).
int launch_variant(int dev, const Variant &v, bool bf, const CUtensorMap &ta, const CUtensorMap &tb,
                   const CUtensorMap &tc, const GemmParams &gp, cudaStream_t stream)
{
    if (v.family == kUmmaPair) {
        if (v.alt_ring)
            return bf ? launch_umma_pair<6, 1, true>(dev, ta, tb, tc, gp, stream)
                      : launch_umma_pair<6, 1, false>(dev, ta, tb, tc, gp, stream);
        return bf ? launch_umma_pair<3, 2, true>(dev, ta, tb, tc, gp, stream)
                  : launch_umma_pair<3, 2, false>(dev, ta, tb, tc, gp, stream);
    }
    if (v.per_sm == 2) {
        if (v.block_n == 64)
            return bf ? launch_umma<64, 2, 1, true>(dev, 11, ta, tb, tc, gp, stream)
                      : launch_umma<64, 2, 1, false>(dev, 12, ta, tb, tc, gp, stream);
        return bf ? launch_umma<128, 2, 1, true>(dev, 13, ta, tb, tc, gp, stream)
                  : launch_umma<128, 2, 1, false>(dev, 14, ta, tb, tc, gp, stream);
    }
    if (v.alt_ring) {
        if (v.block_n == 128)
            return bf ? launch_umma<128, 6, 1, true>(dev, 24, ta, tb, tc, gp, stream)
                      : launch_umma<128, 6, 1, false>(dev, 25, ta, tb, tc, gp, stream);
        return bf ? launch_umma<256, 2, 2, true>(dev, 26, ta, tb, tc, gp, stream)
                  : launch_umma<256, 2, 2, false>(dev, 27, ta, tb, tc, gp, stream);
    }
    switch (v.block_n) {
    case 64:  return bf ? launch_umma<64, 4, 2, true>(dev, 0, ta, tb, tc, gp, stream)
                        : launch_umma<64, 4, 2, false>(dev, 1, ta, tb, tc, gp, stream);
    case 128:
        // short A (M <= 16 / M <= 64): its rows take 2 / 8 KiB of a k-block's shared memory
        // instead of 16, and the ring holds 10 / 8 k-blocks instead of 6
        if (gp.M <= 16)
            return bf ? launch_umma<128, 5, 2, true, 16>(dev, 16, ta, tb, tc, gp, stream)
                      : launch_umma<128, 5, 2, false, 16>(dev, 17, ta, tb, tc, gp, stream);
        if (gp.M <= 64)
            return bf ? launch_umma<128, 4, 2, true, 64>(dev, 18, ta, tb, tc, gp, stream)
                      : launch_umma<128, 4, 2, false, 64>(dev, 19, ta, tb, tc, gp, stream);
        return bf ? launch_umma<128, 3, 2, true>(dev, 2, ta, tb, tc, gp, stream)
                  : launch_umma<128, 3, 2, false>(dev, 3, ta, tb, tc, gp, stream);
    default:  return bf ? launch_umma<256, 4, 1, true>(dev, 4, ta, tb, tc, gp, stream)
                        : launch_umma<256, 4, 1, false>(dev, 5, ta, tb, tc, gp, stream);
    }
}
int prepare_pair(int dev, const Variant &v, bool bf)
{
    if (v.alt_ring) return bf ? prepare_umma_pair<6, 1, true>(dev, 28) : prepare_umma_pair<6, 1, false>(dev, 29);
    return bf ? prepare_umma_pair<3, 2, true>(dev, 6) : prepare_umma_pair<3, 2, false>(dev, 7);
}

// Fills the kernel parameters that depend only on the problem and the tiling.  `group` = the
// raster-group knob of the variant code (0 = the rule below).
GemmParams make_params(const Problem &p, const Tiling &t, int a_box_rows, int group_knob = 0)
{
    GemmParams gp{};
    gp.C = p.C;
    gp.ldc = p.ldc;
    gp.strideC = p.batch > 1 ? p.sC : 0;
    gp.M = (int)p.M; gp.N = (int)p.N; gp.K = (int)p.K; gp.batch = (int)p.batch;
    gp.tiles_m = (int)t.tiles_m; gp.tiles_n = (int)t.tiles_n;
    // raster groups: as many tile rows as keep the group's slice of A within about 32 MB
    // (half of what one L2 partition holds), so that it stays resident while B streams by
    const int64_t tile_rows = cdiv(p.M, t.tiles_m);
    int64_t group = (int64_t(32) << 20) / (tile_rows * p.K * 2 + 1);
    if (group_knob > 0) group = int64_t(1) << (group_knob - 1);
    if (group < 1) group = 1;
    if (group > t.tiles_m) group = t.tiles_m;
    gp.group_m = (int)group;
    gp.kblocks = (int)t.kblocks;
    gp.dp_tiles = (int)t.dp_tiles;
    gp.split_k = t.split;
    gp.num_units = (int)t.units;
    const int64_t vec = (p.out_dtype == CUDALLM_F32) ? 4 : 8;
    gp.c_tma = (reinterpret_cast<uintptr_t>(p.C) % 16 == 0) && (p.ldc % vec == 0)
               && (p.batch == 1 || p.sC % vec == 0);
    gp.n_edge_tma = (p.N % vec == 0);
    gp.a_box_bytes = a_box_rows * 128;
    gp.div_split = make_fast_div((uint32_t)gp.split_k);
    gp.div_item = make_fast_div((uint32_t)(gp.tiles_m * gp.tiles_n));
    gp.div_group = make_fast_div((uint32_t)(gp.group_m * gp.tiles_n));
    gp.div_gm = make_fast_div((uint32_t)gp.group_m);
    const int last_gm = gp.tiles_m % gp.group_m;
    gp.div_gm_last = make_fast_div((uint32_t)(last_gm ? last_gm : gp.group_m));
    gp.wait_limit_ns = g_wait_limit_ns.load(std::memory_order_relaxed);
    return gp;
}

// The launch's flag value for split tiles (0 when nothing is split); normally the units also
// raise their flags to it.
void set_split_epoch(GemmParams &gp, DeviceState &d, bool split);

int next_epoch(DeviceState &d)
{
    d.epoch = (d.epoch == 0x7fffffff) ? 1 : d.epoch + 1;
    return d.epoch;
}
void set_split_epoch(GemmParams &gp, DeviceState &d, bool split)
{
    gp.epoch = split ? next_epoch(d) : 0;
    gp.flag_post = gp.epoch;
    if (split && g_skew_next_flags.exchange(0)) gp.flag_post = gp.epoch ^ 0x40000000;
}

int run_umma(int dev, int code, const Problem &p, cudaStream_t stream)
{
    DeviceState &d = g_dev[dev];
    const Variant &v = g_variants[code_base(code)];
    const bool pair = v.family == kUmmaPair;
    const bool bf = p.out_dtype == CUDALLM_BF16;
    int st;
    if (pair) {
        st = prepare_pair(dev, v, bf);
        if (st != CUDALLM_OK) return st;
    }
    const int slots = pair ? d.max_pairs : d.sm_count * (v.per_sm == 2 ? 2 : 1);
    const Tiling t = tiling_for(v, p, slots, code_tail(code));
    if (t.helper_tiles > kMaxHelperTiles || t.partial_bytes > kMaxPartialBytes)
        return CUDALLM_ERR_UNSUPPORTED_SHAPE;

    const bool pack_a = !a_operand_aligned(p);
    const bool pack_b = !b_operand_aligned(p);
    const Plan pl = make_plan(t, p, pack_a, pack_b);
    Workspace &w = workspace_for(d, stream);
    st = ensure_workspace(w, pl.total, stream);
    if (st != CUDALLM_OK) return st;
    uint8_t *ws = static_cast<uint8_t *>(w.ptr);

    const void *A = p.A, *B = p.B;
    int64_t lda = p.lda, ldb = p.ldb, sA = p.sA, sB = p.sB;
    PackJob ja{}, jb{};
    if (pack_a) {
        ja = pack_job(p.A, ws + pl.off_pack_a, p.M, p.K, p.lda, pl.ldap, p.sA, pl.sAp, p.batch);
        A = ws + pl.off_pack_a; lda = pl.ldap; sA = pl.sAp;
    }
    if (pack_b) {
        jb = pack_job(p.B, ws + pl.off_pack_b, p.K, p.N, p.ldb, pl.ldbp, p.sB, pl.sBp, p.batch);
        B = ws + pl.off_pack_b; ldb = pl.ldbp; sB = pl.sBp;
    }
    st = launch_pack(ja, jb, stream);
    if (st != CUDALLM_OK) return st;

    CUtensorMap ta, tb;
    // Rows of A beyond M only feed rows of C that are never stored, so the box
    // need not cover (and zero-fill) them.  (CTA pairs always use full boxes.)
    const int a_box_rows = (p.M >= kBlockM || pair) ? kBlockM : (int)round_up(p.M, 8);
    st = encode_operand_map(dev, &ta, A, p.K, p.M, p.batch, lda, sA, kBlockK, a_box_rows);
    if (st != CUDALLM_OK) return st;
    st = encode_operand_map(dev, &tb, B, p.N, p.K, p.batch, ldb, sB, 64, kBlockK);
    if (st != CUDALLM_OK) return st;

    GemmParams gp = make_params(p, t, a_box_rows, code_group(code));
    CUtensorMap tc;
    st = encode_c_map(dev, &tc, p, gp.c_tma != 0);
    if (st != CUDALLM_OK) return st;
    set_split_epoch(gp, d, t.split > 1);
    gp.partials = reinterpret_cast<float *>(ws + pl.off_partials);
    gp.flags = reinterpret_cast<int *>(ws + 256);
    gp.status = reinterpret_cast<int *>(ws);
    return launch_variant(dev, v, bf, ta, tb, tc, gp, stream);
}

int run(int variant, const Problem &p, void *stream_v)
{
    build_variants();
    int st = validate(p);
    if (st != CUDALLM_OK) return st;
    if (variant != CUDALLM_VARIANT_AUTO && !code_valid(variant)) return CUDALLM_ERR_INVALID_VARIANT;
    if (is_empty(p)) return CUDALLM_OK;
    if (variant != CUDALLM_VARIANT_AUTO && !variant_supports(g_variants[code_base(variant)], p))
        return CUDALLM_ERR_UNSUPPORTED_SHAPE;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> lock(g_mutex);
    st = probe_device(dev);
    if (st != CUDALLM_OK) return st;
    // A stream with a workspace of its own declares that other launches may share the GPU:
    // the automatic choice then keeps to variants whose CTAs never wait for one another.
    if (variant == CUDALLM_VARIANT_AUTO) variant = select_variant(p, stream_has_workspace(g_dev[dev], stream));
    const Variant &v = g_variants[code_base(variant)];
    if (!variant_supports(v, p)) return CUDALLM_ERR_UNSUPPORTED_SHAPE;
    if (v.family == kSimt) return launch_simt(p, stream);
    return run_umma(dev, variant, p, stream);  // both tcgen05 families
}

Problem make_problem(const void *A, const void *B, void *C, int64_t M, int64_t N, int64_t K, int64_t lda,
                     int64_t ldb, int64_t ldc, int64_t sA, int64_t sB, int64_t sC, int64_t batch,
                     int out_dtype)
{
    Problem p;
    p.A = A; p.B = B; p.C = C;
    p.M = M; p.N = N; p.K = K;
    p.lda = lda; p.ldb = ldb; p.ldc = ldc;
    p.sA = sA; p.sB = sB; p.sC = sC;
    p.batch = batch;
    p.out_dtype = out_dtype;
    return p;
}

// Shape-only problem for the query functions: aligned dummy pointers.
Problem shape_problem(int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb, int64_t ldc,
                      int64_t batch, int out_dtype)
{
    void *dummy = reinterpret_cast<void *>(uintptr_t(256));
    return make_problem(dummy, dummy, dummy, M, N, K, lda, ldb, ldc, M * lda, K * ldb, M * ldc, batch,
                        out_dtype);
}

}  // namespace

// ================================================================= C ABI ====
extern "C" {

int cudallm_gemm_bf16(const void *A, const void *B, void *C, int64_t M, int64_t N, int64_t K,
                      int64_t lda, int64_t ldb, int64_t ldc, int out_dtype, void *stream)
{
    return run(CUDALLM_VARIANT_AUTO,
               make_problem(A, B, C, M, N, K, lda, ldb, ldc, 0, 0, 0, 1, out_dtype), stream);
}

int cudallm_gemm_bf16_batched(const void *A, const void *B, void *C, int64_t M, int64_t N, int64_t K,
                              int64_t lda, int64_t ldb, int64_t ldc, int64_t strideA, int64_t strideB,
                              int64_t strideC, int64_t batch, int out_dtype, void *stream)
{
    return run(CUDALLM_VARIANT_AUTO,
               make_problem(A, B, C, M, N, K, lda, ldb, ldc, strideA, strideB, strideC, batch, out_dtype),
               stream);
}

int cudallm_gemm_bf16_variant(int variant, const void *A, const void *B, void *C, int64_t M, int64_t N,
                              int64_t K, int64_t lda, int64_t ldb, int64_t ldc, int64_t strideA,
                              int64_t strideB, int64_t strideC, int64_t batch, int out_dtype, void *stream)
{
    return run(variant,
               make_problem(A, B, C, M, N, K, lda, ldb, ldc, strideA, strideB, strideC, batch, out_dtype),
               stream);
}

int cudallm_gemm_f32(const void *A, const void *B, void *C, int64_t M, int64_t N, int64_t K, int64_t lda,
                     int64_t ldb, int64_t ldc, int variant, void *stream_v)
{
    build_variants();
    // validate as a product with fp32 output; the operand pointers need 4-byte alignment
    const Problem p = make_problem(A, B, C, M, N, K, lda, ldb, ldc, 0, 0, 0, 1, CUDALLM_F32);
    int st = validate(p);
    if (st != CUDALLM_OK) return st;
    if (variant != CUDALLM_VARIANT_AUTO && (!code_valid(variant) || code_base(variant) < 1))
        return CUDALLM_ERR_INVALID_VARIANT;
    if (is_empty(p)) return CUDALLM_OK;
    if (K > 0 && ((reinterpret_cast<uintptr_t>(A) & 3) || (reinterpret_cast<uintptr_t>(B) & 3)))
        return CUDALLM_ERR_MISALIGNED;
    if (K > kMaxDim / 6) return CUDALLM_ERR_INVALID_DIM;

    // the tcgen05 kernels see a bf16 product over a K range six times as long
    Problem q = p;
    q.K = 6 * round_up(K > 0 ? K : 1, kBlockK);
    q.lda = q.K;
    if (variant == CUDALLM_VARIANT_AUTO) variant = select_variant(q);
    const Variant &v = g_variants[code_base(variant)];
    if (v.family == kSimt || !variant_supports(v, q)) return CUDALLM_ERR_UNSUPPORTED_SHAPE;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> lock(g_mutex);
    st = probe_device(dev);
    if (st != CUDALLM_OK) return st;
    DeviceState &d = g_dev[dev];
    const bool pair = v.family == kUmmaPair;
    if (pair) {
        st = prepare_pair(dev, v, false);
        if (st != CUDALLM_OK) return st;
    }
    if (K == 0) {
        // empty sum: C := 0 (the CUDA-core kernel writes zeros without reading A or B)
        Problem z = p;
        z.A = z.B = C;
        return launch_simt(z, stream);
    }
    const Tiling t = tiling_for(v, q, pair ? d.max_pairs : d.sm_count * (v.per_sm == 2 ? 2 : 1), code_tail(variant));
    if (t.helper_tiles > kMaxHelperTiles || t.partial_bytes > kMaxPartialBytes)
        return CUDALLM_ERR_UNSUPPORTED_SHAPE;

    // workspace: [header][partial tiles][A pieces 3 x M x ldap][B pieces 3 x K x ldbp]
    const int64_t ldap = round_up(K, 8), ldbp = round_up(N, 8);
    size_t off = kHeaderBytes;
    const size_t off_partials = off;
    off = (size_t)round_up((int64_t)(off + t.partial_bytes), 256);
    const size_t off_a = off;
    off = (size_t)round_up((int64_t)off + 3 * M * ldap * 2, 256);
    const size_t off_b = off;
    off = (size_t)round_up((int64_t)off + 3 * K * ldbp * 2, 256);
    Workspace &w = workspace_for(d, stream);
    st = ensure_workspace(w, off, stream);
    if (st != CUDALLM_OK) return st;
    uint8_t *ws = static_cast<uint8_t *>(w.ptr);

    auto split = [&](const void *src, void *dst, int64_t rows, int64_t cols, int64_t ld_src, int64_t ld_dst) {
        const int64_t total = rows * cdiv(cols, 8);
        int64_t blocks = cdiv(total, 256);
        if (blocks > kNumSMs * 16) blocks = kNumSMs * 16;
        return launch_serialised(split3_rows_kernel, (unsigned)blocks, 256, stream, static_cast<const float *>(src),
                                 static_cast<uint16_t *>(dst), (int)rows, (int)cols, (long long)ld_src,
                                 (long long)ld_dst, (long long)(rows * ld_dst));
    };
    st = split(A, ws + off_a, M, K, lda, ldap);
    if (st != CUDALLM_OK) return st;
    st = split(B, ws + off_b, K, N, ldb, ldbp);
    if (st != CUDALLM_OK) return st;
    CUDA_TRY(cudaGetLastError());

    CUtensorMap ta, tb;
    const int a_box_rows = (M >= kBlockM || pair) ? kBlockM : (int)round_up(M, 8);
    st = encode_operand_map(dev, &ta, ws + off_a, K, M, 3, ldap, M * ldap, kBlockK, a_box_rows);
    if (st != CUDALLM_OK) return st;
    st = encode_operand_map(dev, &tb, ws + off_b, N, K, 3, ldbp, K * ldbp, 64, kBlockK);
    if (st != CUDALLM_OK) return st;

    GemmParams gp = make_params(p, t, a_box_rows, code_group(variant));
    CUtensorMap tc;
    st = encode_c_map(dev, &tc, p, gp.c_tma != 0);
    if (st != CUDALLM_OK) return st;
    gp.K = (int)q.K;
    gp.piece_kblocks = (int)cdiv(K, kBlockK);
    set_split_epoch(gp, d, t.split > 1);
    gp.partials = reinterpret_cast<float *>(ws + off_partials);
    gp.flags = reinterpret_cast<int *>(ws + 256);
    gp.status = reinterpret_cast<int *>(ws);
    return launch_variant(dev, v, false, ta, tb, tc, gp, stream);
}

int cudallm_gemm_tf32(const void *A, const void *B, void *C, int64_t M, int64_t N, int64_t K, int64_t lda,
                      int64_t ldb, int64_t ldc, void *stream_v)
{
    build_variants();
    const Problem p = make_problem(A, B, C, M, N, K, lda, ldb, ldc, 0, 0, 0, 1, CUDALLM_F32);
    int st = validate(p);
    if (st != CUDALLM_OK) return st;
    if (is_empty(p)) return CUDALLM_OK;
    if (K > 0 && ((reinterpret_cast<uintptr_t>(A) & 3) || (reinterpret_cast<uintptr_t>(B) & 3)))
        return CUDALLM_ERR_MISALIGNED;
    // TMA reads the operands where they lie: bases on 16 bytes, pitches multiples of 16 bytes.
    // Anything else (and the empty sum) goes the way of cudallm_gemm_f32, which copies its
    // operands anyway and is the more accurate of the two.
    const bool direct = K > 0 && ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B)) & 15) == 0
                     && lda % 4 == 0 && ldb % 4 == 0;
    if (!direct) return cudallm_gemm_f32(A, B, C, M, N, K, lda, ldb, ldc, CUDALLM_VARIANT_AUTO, stream_v);

    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> lock(g_mutex);
    st = probe_device(dev);
    if (st != CUDALLM_OK) return st;
    DeviceState &d = g_dev[dev];

    // CTA pairs (256 x 256 tiles) from two tile rows up; lone CTAs (128 x 256) for one
    const bool pair = M > kBlockM;
    if (pair && d.max_pairs == 0) {
        st = prepare_umma_pair<3, 2, false>(dev, 7);           // asks how many pairs the device holds at once
        if (st != CUDALLM_OK) return st;
    }
    // Tiles as for the bf16 kernels of the same shape (a k-block is 128 bytes of a row of A in
    // both), the tiles of a ragged last wave split along K.
    Variant tv{};
    tv.family = pair ? kUmmaPair : kUmma;
    tv.block_n = kTf32BlockN;
    tv.split_k = kTailSplit;
    tv.per_sm = 1;
    Problem q = p;
    q.K = 2 * K;                                               // in 2-byte elements
    const Tiling t = tiling_for(tv, q, pair ? d.max_pairs : d.sm_count);
    if (t.units > kMaxDim || t.helper_tiles > kMaxHelperTiles || t.partial_bytes > kMaxPartialBytes)
        return CUDALLM_ERR_UNSUPPORTED_SHAPE;

    Workspace &w = workspace_for(d, stream);
    st = ensure_workspace(w, kHeaderBytes + (size_t)t.partial_bytes, stream);
    if (st != CUDALLM_OK) return st;
    uint8_t *ws = static_cast<uint8_t *>(w.ptr);

    CUtensorMap ta, tb, tc;
    st = encode_map(dev, &ta, A, K, M, 1, lda, 0, kTf32BlockK, kBlockM, 1);
    if (st != CUDALLM_OK) return st;
    st = encode_map(dev, &tb, B, N, K, 1, ldb, 0, 32, kTf32BlockK, 3);
    if (st != CUDALLM_OK) return st;
    // raster groups as for bf16, but A's elements are four bytes: as many tile rows as keep the
    // group's slice of A within about 32 MB, rounded down to a power of two (the knob's unit)
    int64_t group = (int64_t(32) << 20) / (cdiv(M, t.tiles_m) * K * 4 + 1);
    int knob = 1;
    while (knob < 15 && (int64_t(2) << (knob - 1)) <= group) ++knob;
    GemmParams gp = make_params(p, t, kBlockM, knob);
    st = encode_c_map(dev, &tc, p, gp.c_tma != 0);
    if (st != CUDALLM_OK) return st;
    set_split_epoch(gp, d, t.split > 1);
    gp.partials = reinterpret_cast<float *>(ws + kHeaderBytes);
    gp.flags = reinterpret_cast<int *>(ws + 256);
    gp.status = reinterpret_cast<int *>(ws);
    if (!d.tf32_attr_set) {
        CUDA_TRY(cudaFuncSetAttribute(umma_tf32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      Tf32Smem::kDynamicBytes));
        CUDA_TRY(cudaFuncSetAttribute(umma_tf32_2cta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      Tf32PairSmem::kDynamicBytes));
        d.tf32_attr_set = true;
    }
    if (pair) {
        const int pairs = (int)std::min<int64_t>(t.units, d.max_pairs);
        return launch_overlapped(umma_tf32_2cta_kernel, 2 * pairs, Tf32PairSmem::kDynamicBytes, stream, ta, tb, tc, gp);
    }
    const int grid = (int)std::min<int64_t>(t.units, d.sm_count);
    return launch_overlapped(umma_tf32_kernel, grid, Tf32Smem::kDynamicBytes, stream, ta, tb, tc, gp);
}

int cudallm_mhsa_bf16(const void *Q, const void *K, const void *V, void *O, int64_t N, int64_t d_model,
                      int64_t h, int64_t ldq, int64_t ldk, int64_t ldv, int64_t ldo, void *stream_v)
{
    if (N < 0 || d_model < 0 || h < 0) return CUDALLM_ERR_INVALID_DIM;
    if (N == 0 || d_model == 0) return CUDALLM_OK;
    if (h == 0 || d_model % h) return CUDALLM_ERR_INVALID_DIM;
    if (ldq < d_model || ldk < d_model || ldv < d_model || ldo < d_model) return CUDALLM_ERR_INVALID_LD;
    if (!Q || !K || !V || !O) return CUDALLM_ERR_INVALID_POINTER;
    if (reinterpret_cast<uintptr_t>(O) & 3) return CUDALLM_ERR_MISALIGNED;
    if ((reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V)) & 1)
        return CUDALLM_ERR_MISALIGNED;
    const int64_t dk = d_model / h;
    if (N > kMaxDim) return CUDALLM_ERR_INVALID_DIM;
    if (dk > kMhsaMaxDk || dk % 8 || h > 65535) return CUDALLM_ERR_UNSUPPORTED_SHAPE;
    if (((reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V)) & 15)
        || ldq % 8 || ldk % 8 || ldv % 8)
        return CUDALLM_ERR_UNSUPPORTED_SHAPE;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> lock(g_mutex);
    int st = probe_device(dev);
    if (st != CUDALLM_OK) return st;
    DeviceState &d = g_dev[dev];
    Workspace &w = workspace_for(d, stream);
    st = ensure_workspace(w, kHeaderBytes, stream);            // for the status word
    if (st != CUDALLM_OK) return st;

    MhsaParams mp{};
    mp.Q = static_cast<const __nv_bfloat16 *>(Q);
    mp.K = static_cast<const __nv_bfloat16 *>(K);
    mp.V = static_cast<const __nv_bfloat16 *>(V);
    mp.O = static_cast<float *>(O);
    mp.N = (int)N; mp.h = (int)h; mp.dk = (int)dk;
    mp.keys_pad = N <= kMhsaMaxKeys ? (int)round_up(N, 32) : kMhsaMaxKeys;   // keys per block
    mp.dkp = (int)round_up(dk, 16);
    mp.tmem_cols = 64;                                  // the second product writes dkp + 16 <= 48 columns
    while (mp.tmem_cols < mp.keys_pad) mp.tmem_cols *= 2;
    mp.ldq = ldq; mp.ldk = ldk; mp.ldv = ldv; mp.ldo = ldo;
    mp.scale_log2 = 1.4426950408889634f / sqrtf((float)dk);
    mp.status = static_cast<int *>(w.ptr);
    const MhsaSmem L = mhsa_smem_layout(mp.keys_pad, mp.dkp);
    if (!d.smem_attr_set[8]) {
        CUDA_TRY(cudaFuncSetAttribute(mhsa_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        CUDA_TRY(cudaFuncSetAttribute(mhsa_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        d.smem_attr_set[8] = true;
    }
    dim3 grid((unsigned)cdiv(N, kMhsaRows), (unsigned)h);
    if (N > kMhsaMaxKeys)
        return launch_serialised_smem(mhsa_kernel<true>, grid, dim3(kMhsaThreads), (size_t)L.total, stream, mp);
    return launch_serialised_smem(mhsa_kernel<false>, grid, dim3(kMhsaThreads), (size_t)L.total, stream, mp);
}

size_t cudallm_host_staging_bytes(int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb, int64_t ldc,
                                  int out_dtype)
{
    if (M < 0 || N < 0 || K < 0 || lda < K || ldb < N || ldc < N) return 0;
    const int64_t esz = out_dtype == CUDALLM_F32 ? 4 : 2;
    return (size_t)(round_up(M * lda * 2, 256) + round_up(K * ldb * 2, 256) + round_up(M * ldc * esz, 256));
}

int cudallm_gemm_bf16_host(const void *A_host, const void *B_host, void *C_host, int64_t M, int64_t N,
                           int64_t K, int64_t lda, int64_t ldb, int64_t ldc, int out_dtype, void *dev_buf,
                           size_t dev_bytes, void *stream_v)
{
    // Validate with stand-in device pointers first (nothing is touched on error).
    void *dummy = reinterpret_cast<void *>(uintptr_t(256));
    Problem p = make_problem(A_host ? dummy : nullptr, B_host ? dummy : nullptr, C_host ? dummy : nullptr,
                             M, N, K, lda, ldb, ldc, 0, 0, 0, 1, out_dtype);
    int st = validate(p);
    if (st != CUDALLM_OK) return st;
    if (is_empty(p)) return CUDALLM_OK;
    const size_t need = cudallm_host_staging_bytes(M, N, K, lda, ldb, ldc, out_dtype);
    if (!dev_buf || dev_bytes < need || (reinterpret_cast<uintptr_t>(dev_buf) % 256))
        return CUDALLM_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int64_t esz = out_dtype == CUDALLM_F32 ? 4 : 2;
    uint8_t *dA = static_cast<uint8_t *>(dev_buf);
    uint8_t *dB = dA + round_up(M * lda * 2, 256);
    uint8_t *dC = dB + round_up(K * ldb * 2, 256);

    // Copy engines and tensor cores overlap: B goes in first, then A in row
    // blocks; block i is multiplied as soon as it has arrived while block i+1
    // is still on the bus, and its rows of C travel back on a third stream.
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    HostPipe &hp = g_host_pipe[dev];
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!hp.ready) {
            CUDA_TRY(cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking));
            CUDA_TRY(cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking));
            for (int i = 0; i < kHostPipeChunks; ++i) {
                CUDA_TRY(cudaEventCreateWithFlags(&hp.arrived[i], cudaEventDisableTiming));
                CUDA_TRY(cudaEventCreateWithFlags(&hp.computed[i], cudaEventDisableTiming));
            }
            CUDA_TRY(cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming));
            CUDA_TRY(cudaEventCreateWithFlags(&hp.done, cudaEventDisableTiming));
            hp.ready = true;
        }
    }
    int64_t rows_per_chunk = round_up(cdiv(M, kHostPipeChunks), 256);
    if (rows_per_chunk < 512) rows_per_chunk = 512;
    const int n_chunks = (int)cdiv(M, rows_per_chunk);

    // the staging buffer may still be in use by earlier work on the caller's stream
    CUDA_TRY(cudaEventRecord(hp.start, stream));
    CUDA_TRY(cudaStreamWaitEvent(hp.in, hp.start, 0));
    if (K > 0)
        CUDA_TRY(cudaMemcpyAsync(dB, B_host, (size_t)(((K - 1) * ldb + N) * 2), cudaMemcpyHostToDevice, hp.in));
    for (int i = 0; i < n_chunks; ++i) {
        const int64_t r0 = i * rows_per_chunk;
        const int64_t rows = (M - r0) < rows_per_chunk ? (M - r0) : rows_per_chunk;
        if (K > 0)
            CUDA_TRY(cudaMemcpyAsync(dA + r0 * lda * 2, static_cast<const uint8_t *>(A_host) + r0 * lda * 2,
                                     (size_t)(((rows - 1) * lda + K) * 2), cudaMemcpyHostToDevice, hp.in));
        CUDA_TRY(cudaEventRecord(hp.arrived[i], hp.in));
        CUDA_TRY(cudaStreamWaitEvent(stream, hp.arrived[i], 0));
        st = cudallm_gemm_bf16(dA + r0 * lda * 2, dB, dC + r0 * ldc * esz, rows, N, K, lda, ldb, ldc,
                               out_dtype, stream_v);
        if (st != CUDALLM_OK) return st;
        CUDA_TRY(cudaEventRecord(hp.computed[i], stream));
        CUDA_TRY(cudaStreamWaitEvent(hp.out, hp.computed[i], 0));
        uint8_t *hc = static_cast<uint8_t *>(C_host) + r0 * ldc * esz;
        if (ldc == N) {
            CUDA_TRY(cudaMemcpyAsync(hc, dC + r0 * ldc * esz, (size_t)(rows * N * esz), cudaMemcpyDeviceToHost,
                                     hp.out));
        } else {
            // keep the caller's padding columns untouched
            CUDA_TRY(cudaMemcpy2DAsync(hc, (size_t)(ldc * esz), dC + r0 * ldc * esz, (size_t)(ldc * esz),
                                       (size_t)(N * esz), (size_t)rows, cudaMemcpyDeviceToHost, hp.out));
        }
    }
    CUDA_TRY(cudaEventRecord(hp.done, hp.out));
    CUDA_TRY(cudaStreamWaitEvent(stream, hp.done, 0));
    CUDA_TRY(cudaStreamSynchronize(stream));
    return CUDALLM_OK;
}

// ---------------------------------------------------------------------------
// Split-K without any allocation: the scratch is part of the device image.
// `g_noalloc_scratch` names the array for device code; on the host the same
// name is only a handle for cudaGetSymbolAddress, never a device address.
// Layout: [status word, 256 B][helper flags, 64 KiB][helper partial tiles].
static __device__ __align__(256) unsigned char g_noalloc_scratch[CUDALLM_NOALLOC_SCRATCH_BYTES];
static void *g_noalloc_scratch_addr[kMaxDevices] = {};   // per device, filled on first use
static int g_noalloc_epoch[kMaxDevices] = {};
constexpr size_t kNoallocHeaderBytes = CUDALLM_NOALLOC_HEADER_BYTES;   // status + flags
constexpr int64_t kNoallocMaxHelperTiles = (kNoallocHeaderBytes - 256) / 16;

int cudallm_gemm_bf16_splitk_noalloc(const void *A, const void *B, void *C, int64_t M, int64_t N,
                                     int64_t K, int64_t lda, int64_t ldb, int64_t ldc, int out_dtype,
                                     int split_k, void *stream_v)
{
    build_variants();
    const Problem p = make_problem(A, B, C, M, N, K, lda, ldb, ldc, 0, 0, 0, 1, out_dtype);
    int st = validate(p);
    if (st != CUDALLM_OK) return st;
    if (split_k != 2 && split_k != 4 && split_k != 8 && split_k != 16) return CUDALLM_ERR_INVALID_VARIANT;
    if (is_empty(p)) return CUDALLM_OK;
    if (cdiv(K, kBlockK) < split_k) return CUDALLM_ERR_UNSUPPORTED_SHAPE;   // also covers K == 0
    if (!a_operand_aligned(p) || !b_operand_aligned(p)) return CUDALLM_ERR_UNSUPPORTED_SHAPE;

    // always 128 x 64 tiles, every tile split: split_k slots of 32 KiB per tile
    Variant v{};
    v.family = kUmma;
    v.block_n = 64;
    v.split_k = split_k;
    const Tiling t = tiling_for(v, p, kNumSMs);
    if (t.units > kMaxDim || t.helper_tiles > kNoallocMaxHelperTiles
        || (long double)t.partial_bytes + (long double)kNoallocHeaderBytes
               > (long double)CUDALLM_NOALLOC_SCRATCH_BYTES)
        return CUDALLM_ERR_TOO_LARGE;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    std::unique_lock<std::mutex> lock(g_mutex);
    st = probe_device(dev);
    if (st != CUDALLM_OK) return st;
    if (!g_noalloc_scratch_addr[dev]) {
        // once per device, with that device current
        void *addr = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&addr, g_noalloc_scratch));
        g_noalloc_scratch_addr[dev] = addr;
    }
    uint8_t *scratch = static_cast<uint8_t *>(g_noalloc_scratch_addr[dev]);

    CUtensorMap ta, tb;
    const int a_box_rows = p.M >= kBlockM ? kBlockM : (int)round_up(p.M, 8);
    st = encode_operand_map(dev, &ta, A, p.K, p.M, 1, lda, 0, kBlockK, a_box_rows);
    if (st != CUDALLM_OK) return st;
    st = encode_operand_map(dev, &tb, B, p.N, p.K, 1, ldb, 0, 64, kBlockK);
    if (st != CUDALLM_OK) return st;

    GemmParams gp = make_params(p, t, a_box_rows);
    CUtensorMap tc;
    st = encode_c_map(dev, &tc, p, gp.c_tma != 0);
    if (st != CUDALLM_OK) return st;
    g_noalloc_epoch[dev] = (g_noalloc_epoch[dev] == 0x7fffffff) ? 1 : g_noalloc_epoch[dev] + 1;
    gp.epoch = g_noalloc_epoch[dev];
    gp.flag_post = gp.epoch;
    gp.status = reinterpret_cast<int *>(scratch);
    gp.flags = reinterpret_cast<int *>(scratch + 256);
    gp.partials = reinterpret_cast<float *>(scratch + kNoallocHeaderBytes);

    // The array keeps the last call's contents.  The status word and the flags
    // must start at zero; partial tiles are written before they are read.
    CUDA_TRY(cudaMemsetAsync(scratch, 0, kNoallocHeaderBytes, stream));
    st = (p.out_dtype == CUDALLM_BF16) ? launch_umma<64, 4, 2, true>(dev, 0, ta, tb, tc, gp, stream)
                                       : launch_umma<64, 4, 2, false>(dev, 1, ta, tb, tc, gp, stream);
    if (st != CUDALLM_OK) return st;
    lock.unlock();                   // other library calls need not wait for this kernel
    int host_status[2] = {0, 0};
    CUDA_TRY(cudaMemcpyAsync(host_status, scratch, sizeof host_status, cudaMemcpyDeviceToHost, stream));
    CUDA_TRY(cudaStreamSynchronize(stream));
    return host_status[0] == 0 ? CUDALLM_OK : CUDALLM_ERR_DEVICE_TIMEOUT;
}

int cudallm_num_variants(void)
{
    return kNumVariants;
}

const char *cudallm_variant_name(int variant)
{
    build_variants();
    if (!code_valid(variant)) return nullptr;
    return g_variants[code_base(variant)].name;
}

static int compose_code(int variant, int group_rows, int tail_parts)
{
    if (variant < 0 || variant >= kNumVariants) return CUDALLM_ERR_INVALID_VARIANT;
    int g = 0;
    if (group_rows != 0) {
        if (group_rows < 0 || group_rows > 16384 || (group_rows & (group_rows - 1))) return CUDALLM_ERR_INVALID_VARIANT;
        while ((1 << g) < group_rows) ++g;
        ++g;
    }
    if (tail_parts != 0 && (tail_parts < 2 || tail_parts > 7)) return CUDALLM_ERR_INVALID_VARIANT;
    if (tail_parts != 0 && g_variants[variant].split_k != kTailSplit) return CUDALLM_ERR_INVALID_VARIANT;
    return variant | (g << 8) | (tail_parts << 12);
}

int cudallm_variant_code(int variant, int group_rows, int tail_parts)
{
    build_variants();
    return compose_code(variant, group_rows, tail_parts);
}

int cudallm_variant_supports(int variant, int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb,
                             int64_t ldc, int64_t batch, int out_dtype)
{
    build_variants();
    if (!code_valid(variant)) return CUDALLM_ERR_INVALID_VARIANT;
    Problem p = shape_problem(M, N, K, lda, ldb, ldc, batch, out_dtype);
    int st = validate(p);
    if (st != CUDALLM_OK) return st;
    return variant_supports(g_variants[code_base(variant)], p) ? 1 : 0;
}

int cudallm_select_variant(int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb, int64_t ldc,
                           int64_t batch, int out_dtype)
{
    Problem p = shape_problem(M, N, K, lda, ldb, ldc, batch, out_dtype);
    int st = validate(p);
    if (st != CUDALLM_OK) return st;
    return select_variant(p);
}

static int dispatch_key_status(int64_t M, int64_t N, int64_t K, int64_t batch, int out_dtype)
{
    if (M < 0 || N < 0 || K < 0 || batch < 0) return CUDALLM_ERR_INVALID_DIM;
    if (out_dtype != CUDALLM_F32 && out_dtype != CUDALLM_BF16) return CUDALLM_ERR_INVALID_DTYPE;
    return CUDALLM_OK;
}

static int dispatch_store(std::unordered_map<DispatchKey, int, DispatchHash> &table, const DispatchKey &key, int variant)
{
    if (variant != -1 && !code_valid(variant)) return CUDALLM_ERR_INVALID_VARIANT;
    std::lock_guard<std::mutex> lock(g_dispatch_mutex);
    if (variant < 0) {
        table.erase(key);
    } else {
        if (table.size() >= kMaxDispatchEntries && table.find(key) == table.end()) return CUDALLM_ERR_TOO_LARGE;
        table[key] = variant;
    }
    g_dispatch_generation.fetch_add(1, std::memory_order_release);
    return CUDALLM_OK;
}

int cudallm_dispatch_set(int64_t M, int64_t N, int64_t K, int64_t batch, int out_dtype, int variant)
{
    build_variants();
    const int st = dispatch_key_status(M, N, K, batch, out_dtype);
    if (st != CUDALLM_OK) return st;
    return dispatch_store(g_dispatch, DispatchKey{M, N, K, batch, out_dtype}, variant);
}

int cudallm_dispatch_set_class(int64_t M, int64_t N, int64_t K, int64_t batch, int out_dtype, int tma_addressable,
                               int variant)
{
    build_variants();
    const int st = dispatch_key_status(M, N, K, batch, out_dtype);
    if (st != CUDALLM_OK) return st;
    return dispatch_store(g_dispatch_class, class_key(M, N, K, batch, out_dtype, tma_addressable != 0), variant);
}

int cudallm_dispatch_get(int64_t M, int64_t N, int64_t K, int64_t batch, int out_dtype, int *variant)
{
    const int st = dispatch_key_status(M, N, K, batch, out_dtype);
    if (st != CUDALLM_OK) return st;
    if (!variant) return CUDALLM_ERR_INVALID_POINTER;
    std::lock_guard<std::mutex> lock(g_dispatch_mutex);
    const auto it = g_dispatch.find(DispatchKey{M, N, K, batch, out_dtype});
    *variant = it == g_dispatch.end() ? -1 : it->second;
    return CUDALLM_OK;
}

int cudallm_dispatch_get_class(int64_t M, int64_t N, int64_t K, int64_t batch, int out_dtype, int tma_addressable,
                               int *variant)
{
    const int st = dispatch_key_status(M, N, K, batch, out_dtype);
    if (st != CUDALLM_OK) return st;
    if (!variant) return CUDALLM_ERR_INVALID_POINTER;
    std::lock_guard<std::mutex> lock(g_dispatch_mutex);
    const auto it = g_dispatch_class.find(class_key(M, N, K, batch, out_dtype, tma_addressable != 0));
    *variant = it == g_dispatch_class.end() ? -1 : it->second;
    return CUDALLM_OK;
}

int cudallm_dispatch_clear(void)
{
    build_variants();                  // (the packaged entries are entered on first use: before, not after, this)
    std::lock_guard<std::mutex> lock(g_dispatch_mutex);
    const int n = (int)(g_dispatch.size() + g_dispatch_class.size());
    g_dispatch.clear();
    g_dispatch_class.clear();
    g_dispatch_generation.fetch_add(1, std::memory_order_release);
    return n;
}

// The winners of the search as recorded on a B200 (generated from the package's table file
// when the library is built): entered as class entries when the library is first used.
struct PackagedEntry {
    long long M, N, K, batch;
    int out_dtype, tma_addressable;
    const char *variant;
    int group_rows, tail_parts;
};
static const PackagedEntry kPackaged[] = {
#include "tuned_table.inc"
    {0, 0, 0, 0, 0, 0, nullptr, 0, 0}
};

}  // extern "C"
namespace {
int load_packaged_entries()
{
    int n = 0;
    for (const PackagedEntry *e = kPackaged; e->variant; ++e) {
        int base = -1;
        for (int v = 0; v < kNumVariants; ++v)
            if (!strcmp(g_variants[v].name, e->variant)) base = v;
        const int code = compose_code(base, e->group_rows, e->tail_parts);
        if (code < 0 || dispatch_key_status(e->M, e->N, e->K, e->batch, e->out_dtype) != CUDALLM_OK) continue;
        if (dispatch_store(g_dispatch_class, class_key(e->M, e->N, e->K, e->batch, e->out_dtype, e->tma_addressable != 0),
                           code) == CUDALLM_OK)
            ++n;
    }
    return n;
}
}  // namespace
extern "C" {

int cudallm_dispatch_load_packaged(void)
{
    build_variants();
    return load_packaged_entries();
}

size_t cudallm_workspace_bytes(int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb, int64_t ldc,
                               int64_t batch, int out_dtype)
{
    build_variants();
    Problem p = shape_problem(M, N, K, lda, ldb, ldc, batch, out_dtype);
    if (validate(p) != CUDALLM_OK || is_empty(p)) return kHeaderBytes;
    size_t best = kHeaderBytes;
    for (int v = 0; v < kNumVariants; ++v) {
        if (!variant_supports(g_variants[v], p)) continue;
        // worst case: both operands repacked
        const Plan pl = make_plan(tiling_for(g_variants[v], p, default_slots(g_variants[v])), p, true, true);
        if (pl.total > best) best = pl.total;
    }
    return best;
}

int cudallm_set_workspace(void *dev_ptr, size_t bytes)
{
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> lock(g_mutex);
    Workspace &w = g_dev[dev].ws;
    if (!dev_ptr) {
        w.ptr = w.internal;
        w.bytes = w.internal_bytes;
        w.external = false;
        return CUDALLM_OK;
    }
    if (bytes < kHeaderBytes || (reinterpret_cast<uintptr_t>(dev_ptr) % 256)) return CUDALLM_ERR_WORKSPACE;
    w.ptr = dev_ptr;
    w.bytes = bytes;
    w.external = true;
    return CUDALLM_OK;
}

int cudallm_set_workspace_for_stream(void *stream_v, void *dev_ptr, size_t bytes)
{
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState &d = g_dev[dev];
    if (!dev_ptr) {
        d.stream_ws.erase(stream);
        return CUDALLM_OK;
    }
    if (bytes < kHeaderBytes || (reinterpret_cast<uintptr_t>(dev_ptr) % 256)) return CUDALLM_ERR_WORKSPACE;
    for (const auto &kv : d.stream_ws)           // two streams must not share scratch
        if (kv.first != stream) {
            const uint8_t *a = static_cast<const uint8_t *>(kv.second.ptr), *b = static_cast<const uint8_t *>(dev_ptr);
            if (a < b + bytes && b < a + kv.second.bytes) return CUDALLM_ERR_WORKSPACE;
        }
    Workspace w;
    w.ptr = dev_ptr;
    w.bytes = bytes;
    w.external = true;
    d.stream_ws[stream] = w;
    return CUDALLM_OK;
}

int cudallm_reserve_workspace(size_t bytes)
{
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> lock(g_mutex);
    Workspace &w = g_dev[dev].ws;
    if (w.external) return CUDALLM_ERR_WORKSPACE;
    return ensure_workspace(w, bytes < kHeaderBytes ? kHeaderBytes : bytes, nullptr, true);
}

int cudallm_shutdown(void)
{
    int cur = 0;
    const bool have_dev = cudaGetDevice(&cur) == cudaSuccess;
    std::lock_guard<std::mutex> lock(g_mutex);
    int first_error = CUDALLM_OK;
    for (int dev = 0; dev < kMaxDevices; ++dev) {
        DeviceState &d = g_dev[dev];
        HostPipe &hp = g_host_pipe[dev];
        if (!d.ws.internal && !hp.ready) {
            d.stream_ws.clear();
            continue;
        }
        if (cudaSetDevice(dev) != cudaSuccess) continue;
        cudaError_t e = cudaDeviceSynchronize();
        if (d.ws.internal) {
            if (e == cudaSuccess) e = cudaFree(d.ws.internal);
            if (!d.ws.external) { d.ws.ptr = nullptr; d.ws.bytes = 0; }
            d.ws.internal = nullptr;
            d.ws.internal_bytes = 0;
        }
        if (hp.ready) {
            cudaStreamDestroy(hp.in);
            cudaStreamDestroy(hp.out);
            for (int i = 0; i < kHostPipeChunks; ++i) {
                cudaEventDestroy(hp.arrived[i]);
                cudaEventDestroy(hp.computed[i]);
            }
            cudaEventDestroy(hp.start);
            cudaEventDestroy(hp.done);
            hp = HostPipe{};
        }
        d.stream_ws.clear();
        if (e != cudaSuccess && first_error == CUDALLM_OK) first_error = cuda_fail(e, "cudallm_shutdown");
    }
    if (have_dev) cudaSetDevice(cur);
    return first_error;
}

int cudallm_debug_set(int what, unsigned long long value)
{
    switch (what) {
    case CUDALLM_DEBUG_WAIT_LIMIT_NS:
        g_wait_limit_ns.store(value ? value : kWaitLimitNs);
        return CUDALLM_OK;
    case CUDALLM_DEBUG_MISS_NEXT_SPLIT_FLAGS:
        g_skew_next_flags.store(value ? 1 : 0);
        return CUDALLM_OK;
    case CUDALLM_DEBUG_LAYERNORM_PATH:
        if (value > 2) return CUDALLM_ERR_INVALID_VARIANT;
        g_layernorm_path.store((int)value);
        return CUDALLM_OK;
    default:
        return CUDALLM_ERR_INVALID_VARIANT;
    }
}

int cudallm_device_status(void *stream_v, int *code, int *detail)
{
    if (code) *code = CUDALLM_OK;
    if (detail) *detail = 0;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CUDALLM_ERR_UNSUPPORTED_DEVICE;
    CUDA_TRY(cudaStreamSynchronize(stream));
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState &d = g_dev[dev];
    Workspace &w = workspace_for(d, stream);
    if (!w.ptr) return CUDALLM_OK;                     // no kernel of ours has run yet
    int host[2] = {0, 0};
    CUDA_TRY(cudaMemcpy(host, w.ptr, sizeof host, cudaMemcpyDeviceToHost));
    if (host[0] != 0) {
        // a kernel gave up: flags and counters may be stale; clear the whole header
        CUDA_TRY(cudaMemset(w.ptr, 0, kHeaderBytes));
    }
    if (code) *code = host[0];
    if (detail) *detail = host[1];
    return host[0];
}

const char *cudallm_strerror(int status)
{
    switch (status) {
    case CUDALLM_OK: return "success";
    case CUDALLM_ERR_INVALID_POINTER: return "null operand pointer for a non-empty problem";
    case CUDALLM_ERR_INVALID_DIM: return "negative or too large dimension";
    case CUDALLM_ERR_INVALID_LD: return "leading dimension smaller than the row length, or overlapping batch items of C";
    case CUDALLM_ERR_INVALID_DTYPE: return "out_dtype must be 0 (fp32) or 1 (bf16)";
    case CUDALLM_ERR_INVALID_VARIANT: return "variant id out of range";
    case CUDALLM_ERR_UNSUPPORTED_SHAPE: return "the requested variant cannot run this problem";
    case CUDALLM_ERR_UNSUPPORTED_DEVICE: return "the current device is not compute capability 10.0";
    case CUDALLM_ERR_CUDA: return g_cuda_err[0] ? g_cuda_err : "CUDA call failed";
    case CUDALLM_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case CUDALLM_ERR_WORKSPACE: return "workspace missing, too small or misaligned";
    case CUDALLM_ERR_MISALIGNED: return "pointer not aligned to its element size";
    case CUDALLM_ERR_TOO_LARGE: return "problem exceeds the fixed-size built-in scratch of this entry point";
    default: return "unknown status";
    }
}

int cudallm_version(void)
{
    return 100;   // 0.1.0
}

}  // extern "C"

#include "hbm_tasks_host.cuh"
