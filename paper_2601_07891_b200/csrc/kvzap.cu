// Host side of the C ABI declared in include/kvzap.h: context, weight
// repacking, TMA descriptors, argument checks and kernel launches.
#include "../../include/kvzap.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <algorithm>
#include <vector>

#include "attn_kernel.cuh"
#include "decode_kernels.cuh"
#include "prune_kernels.cuh"
#include "prune_onepass_kernel.cuh"
#include "score_kernel.cuh"
#include "score_linear_split_kernel.cuh"
#include "score_split_kernel.cuh"
#include "select_kernels.cuh"

namespace kvzap {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);


static char g_create_error[512] = "";

// Mask slices used in rotation.  A scoring kernel may start while the compaction of the call before it
// is still running (see launch_score); that compaction reads the previous slice, never the current one.
constexpr int kMaskRing = 4;

}  // namespace kvzap

struct kvzap_ctx {
    kvzap_config cfg;
    int sm_count = 0;
    int w1_rows = 0;                 // rows of the stored first-layer matrix (Linear: padded to 16)
    bool lin_split_ok = false;       // KVzap-Linear: the four-CTAs-per-tile kernel for short inputs can be used
    // scoring schedules (see ScoreParams): [0] one CTA per tile, [1] CTA pairs (MLP only)
    struct Schedule {
        int group_w = 0, n_groups = 0, chunk_n = 0, n_chunks = 0, n_stages = 0, acc_bufs = 0, acc_stride = 0,
            tmem_cols = 0;
        uint32_t smem = 0;
        CUtensorMap tmap_w;          // box = the W1 rows one CTA stages per MMA chunk
    } sched[2];
    int pair_clusters = 0;           // CTA pairs that can be resident at once; 0 = pairs unavailable
    // few-token scoring (decode): clusters of split_n CTAs share a tile, each takes hidden / split_n units
    int split_n = 0, split_k = 1, split_stages = 0, split_tmem_cols = 0;   // cluster = split_n * split_k CTAs
    uint32_t split_smem = 0;
    CUtensorMap split_tmap_w;
    CUtensorMap split_tmap_w8;           // the 8-bit copy of the weights, same slices (set by kvzap_set_weights_fp8)
    bool split8_ok = false;
    // the same kernel with eight CTAs per tile (4 slices x 2 halves of K) for launches of even fewer tiles
    // (a short prompt or a chunk of one): set when the shape allows it
    int wide_n = 0, wide_k = 1, wide_stages = 0, wide_tmem_cols = 0;
    uint32_t wide_smem = 0;
    CUtensorMap wide_tmap_w;
    uint32_t *wide_arrive = nullptr;     // its own arrival counts (the count per tile is taken modulo the slices)
    // weights of all layers, stacked so that one tensor map / one base pointer serves any layer range
    void *w1_all = nullptr;          // bf16 [L * w1_rows, d_model]
    float *b1_all = nullptr;         // [L][w1_rows]
    float *w2t_all = nullptr;        // [L][hidden][8] fp32 (MLP)
    float *b2_all = nullptr;         // [L][8] (MLP)
    std::vector<char> layer_set;
    // layers whose first layer was given as E4M3 bytes (kvzap_set_weights_fp8): K-blocked copy with 128 elements
    // per block, one scale per output row; allocated when the first such layer arrives
    void *w1_fp8_all = nullptr;      // [d_model / 128][L * w1_rows][128] bytes
    float *w1_scale_all = nullptr;   // [L][w1_rows]
    std::vector<char> layer_fp8;
    CUtensorMap tmap_w8[2];          // boxes as sched[].tmap_w
    kvzap::EncodeTiledFn encode = nullptr;
    // scratch
    int64_t max_blocks = 0, max_words = 0;
    uint32_t *maskbits = nullptr;    // [kMaskRing][H][max_words]: consecutive calls use different slices
    uint64_t mask_turn = 0;
    int32_t *tile_counters = nullptr;    // [kMaskRing] work-tile counters of the scoring launches, used in rotation
    uint32_t *select_hist = nullptr;     // fixed-budget selection: [4 passes][max_seqs][H][256] histograms
    float *select_tau = nullptr;         //                         [max_seqs][H] cut values when the caller wants none
    float *plan_scores = nullptr;        // kvzap_prefill_plan without scores_out: [max_tokens][H] (allocated on first use)
    int64_t *batch_map = nullptr;        // kvzap_prefill_to_cache_batch: first list of each sequence of the call [max_seqs]
    float *split_part = nullptr;         // few-token kernel: [sm_count tiles][4 slices][128][8] partial scores
    uint32_t *split_arrive = nullptr;    //                   [sm_count] arrival counts per tile
    uint64_t score_turn = 0;
    bool last_score_early = false;       // the last scoring launch was allowed to start early
    const void *last_scores = nullptr;   // scores buffer of the previous scoring launch, and its size
    size_t last_scores_bytes = 0;
    int32_t *list_page0 = nullptr;   // [max_seqs * H] first page of each list (paged output)
    int32_t *list_base = nullptr;    // [max_seqs * H] appending to lists: rows each list held before
    int32_t *status_dev = nullptr;
    int32_t *status_host = nullptr;  // pinned
    int64_t launches = 0;
    // tensor maps of recently used hidden-state buffers (encoding one costs about as much as a launch)
    struct TmapEntry { const void *base; int64_t rows; int32_t slabs; CUtensorMap map; };
    std::vector<TmapEntry> tmap_cache;
    size_t tmap_next = 0;
    // optional per-kernel timing (kvzap_set_profiling)
    bool profiling = false;
    struct ProfRec { int kind; cudaEvent_t start, stop; };
    std::vector<ProfRec> prof;
    // device staging for the host-buffer entry point (allocated on first use)
    // two sets, used by alternate layers: layer l + 1 is copied in while layer l is computed and copied out
    struct HostStage {
        void *x = nullptr, *k = nullptr, *v = nullptr, *ko = nullptr, *vo = nullptr;
        float *scores = nullptr;
        int32_t *lengths = nullptr, *table = nullptr, *used = nullptr;   // device
        int32_t *lengths_pinned = nullptr;                               // host, lengths followed by the page count
        size_t out_bytes = 0, table_ints = 0;
        cudaEvent_t copied_in = nullptr, computed = nullptr;
    } stage[2];
    int32_t *stage_cu = nullptr;
    cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
    // kvzap_config.flags & KVZAP_FLAG_TRUSTED_PRODUCERS: kernels may read caller data before the work ahead of
    // them in the stream has completed
    bool trusted = false;
    int64_t wait_limit = KVZAP_WAIT_LIMIT_CYCLES;   // bound of the waits on flags in global memory
    // Every public call that enqueues work takes the next number.  A fused decode step may start before the
    // kernel ahead of it has finished only when that kernel is the fused step of the call just before, on
    // the same cache: those two order their cache accesses through the step counters, nothing else does.
    uint64_t op_seq = 0, fused_seq = 0;
    const kvzap_cache *fused_cache = nullptr;
    std::vector<kvzap_cache *> caches;              // caches created on this context (their step counters are
                                                    // cleared when a timeout has been polled)
    // one-launch pruning (kvzap_prune_prefill and its paged / fixed-budget forms): kOpRing scratch sets in rotation
    int op_capacity = 0;                 // CTAs of prune_onepass_kernel the device holds at once
    uint32_t *op_mask = nullptr;         // [kOpRing][H][max_words]
    uint64_t *op_counts = nullptr;       // [kOpRing][op_capacity][8]
    int32_t *op_len_acc = nullptr;       // [kOpRing][max_seqs * H], zero between calls
    uint32_t *op_arrive = nullptr;       // [kOpRing]
    int32_t *op_scan_flag = nullptr;     // [kOpRing]
    int32_t *op_page0 = nullptr;         // [kOpRing][max_seqs * H]
    uint64_t *lin_counts = nullptr;      // [kOpRing][kLinMaxTiles][8]: tile counts of the scoring launch that also compacts
    uint64_t op_turn = 0;
    int32_t op_epoch = 0;
    int op_chain = 0;                    // launches of that kernel in a row that did not wait for the work ahead
    uint64_t op_last_seq = 0;            // number (op_seq) of the last call that launched it
    // Caller memory read or written by the launches of that kernel since the last one that waited for all
    // work ahead of it: these launches may still be running.  Another one is started without such a wait
    // only directly behind them and only if it conflicts with none of these ranges; the scoring kernels
    // consult the list before they write a scores buffer early.
    struct Range { const char *p; size_t n; bool w; };
    std::vector<Range> pending;
    char err[512] = "";
};

namespace kvzap {

static kvzap_status fail(kvzap_ctx *ctx, kvzap_status st, const char *fmt, ...)
{
    char *dst = ctx ? ctx->err : g_create_error;
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(dst, 512, fmt, ap);
    va_end(ap);
    return st;
}

#define KVZAP_CUDA(ctx, call)                                                                        \
    do {                                                                                             \
        cudaError_t e_ = (call);                                                                     \
        if (e_ != cudaSuccess)                                                                       \
            return kvzap::fail(ctx, KVZAP_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); \
    } while (0)

// Numbers a public call (see kvzap_ctx::op_seq).
static inline void begin_op(kvzap_ctx *ctx) { ctx->op_seq += 1; }

// ---- what the kernels in flight may still touch (see kvzap_ctx::pending)
constexpr size_t kMaxPending = 96;
static inline void note_range(kvzap_ctx *ctx, const void *p, size_t n, bool write)
{
    if (p != nullptr && n > 0) ctx->pending.push_back({static_cast<const char *>(p), n, write});
}
// true if [p, p + n) overlaps a pending range in a conflicting way (a write on either side)
static inline bool hazard(const kvzap_ctx *ctx, const void *p, size_t n, bool write)
{
    if (p == nullptr || n == 0) return false;
    if (ctx->pending.size() > kMaxPending) return true;
    const char *a = static_cast<const char *>(p);
    for (const auto &r : ctx->pending)
        if ((write || r.w) && a < r.p + r.n && r.p < a + n) return true;
    return false;
}
// everything enqueued so far is complete before whatever is enqueued next starts
static inline void serial_point(kvzap_ctx *ctx) { ctx->pending.clear(); ctx->op_chain = 0; }

// Clears the fused decode step's counters (device and host view) of every cache of the context.
static void reset_step_counters(kvzap_ctx *ctx, cudaStream_t stream);

static int next_pow2(int v)
{
    int p = 32;
    while (p < v) p <<= 1;
    return p;
}

// bf16 tensor map over `slabs` matrices of `rows` x `cols` (row-major, slabs contiguous); box = one slab,
// `box_rows` rows, 64 elements; 128-byte swizzle.  slabs == 0 makes a 2-D map.
static kvzap_status make_tmap(kvzap_ctx *ctx, CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols,
                              uint32_t box_rows, uint64_t slabs = 0)
{
    const cuuint64_t dims[3] = {cols, rows, slabs ? slabs : 1};
    const cuuint64_t strides[2] = {cols * 2, cols * 2 * rows};
    const cuuint32_t box[3] = {static_cast<cuuint32_t>(kBlockK), box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = ctx->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, slabs ? 3 : 2, const_cast<void *>(base), dims,
                                   strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(ctx, KVZAP_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d (rows=%llu cols=%llu box_rows=%u)",
                    static_cast<int>(r), static_cast<unsigned long long>(rows), static_cast<unsigned long long>(cols),
                    box_rows);
    return KVZAP_OK;
}

// 8-bit tensor map over `slabs` matrices of `rows` x `cols` bytes; box = box_rows rows x 128 bytes, 128-byte swizzle.
// inner_blocked: the matrix is stored K block by K block, [cols / 128][rows][128] (the weights' copy).
static kvzap_status make_tmap8(kvzap_ctx *ctx, CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                               uint64_t slabs, bool inner_blocked)
{
    cuuint64_t dims[3], strides[2];
    if (inner_blocked) {
        dims[0] = 128; dims[1] = rows; dims[2] = cols / 128;
        strides[0] = 128; strides[1] = 128 * rows;
    } else {
        dims[0] = cols; dims[1] = rows; dims[2] = slabs ? slabs : 1;
        strides[0] = cols; strides[1] = cols * rows;
    }
    const cuuint32_t box[3] = {128, box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = ctx->encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(base), dims, strides, box, estr,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(ctx, KVZAP_ERR_CUDA, "cuTensorMapEncodeTiled (8-bit) failed with code %d (rows=%llu cols=%llu box_rows=%u)",
                    static_cast<int>(r), static_cast<unsigned long long>(rows), static_cast<unsigned long long>(cols), box_rows);
    return KVZAP_OK;
}

// Tensor map over `rows` rows of `row_bytes` bytes each, seen as tiles of box_rows whole rows: a tile is one
// contiguous, 128-byte aligned piece of memory (box_rows * row_bytes is a multiple of 128), fetched as that many
// full 128-byte lines and laid out in shared memory as it lies in memory (no swizzle).  Coordinates (0, 0, tile).
static kvzap_status make_tmap_rows(kvzap_ctx *ctx, CUtensorMap *map, const void *base, uint64_t rows, uint32_t row_bytes,
                                   uint32_t box_rows)
{
    const uint32_t lines = box_rows * row_bytes / 128;
    const cuuint64_t dims[3] = {128, lines, rows / box_rows};
    const cuuint64_t strides[2] = {128, static_cast<cuuint64_t>(lines) * 128};
    const cuuint32_t box[3] = {128, lines, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = ctx->encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(base), dims, strides, box, estr,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(ctx, KVZAP_ERR_CUDA, "cuTensorMapEncodeTiled (rows) failed with code %d (rows=%llu row_bytes=%u box_rows=%u)",
                    static_cast<int>(r), static_cast<unsigned long long>(rows), row_bytes, box_rows);
    return KVZAP_OK;
}

// Tensor map over the context's copy of the first-layer weights, stored K block by K block:
// [k_blocks][rows_total][64] bf16, so that the `box_rows` x 64 tile a CTA stages per K step is one
// contiguous piece of memory (a decode step reads every weight byte from HBM exactly once; contiguous
// tiles keep those reads inside open DRAM pages).  Box = box_rows rows of one K block, 128-byte swizzle.
static kvzap_status make_tmap_w(kvzap_ctx *ctx, CUtensorMap *map, const void *base, uint64_t rows_total,
                                uint64_t k_blocks, uint32_t box_rows)
{
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(kBlockK), rows_total, k_blocks};
    const cuuint64_t strides[2] = {kBlockK * 2, kBlockK * 2 * rows_total};
    const cuuint32_t box[3] = {static_cast<cuuint32_t>(kBlockK), box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = ctx->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box,
                                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(ctx, KVZAP_ERR_CUDA, "cuTensorMapEncodeTiled (weights) failed with code %d (rows=%llu box_rows=%u)",
                    static_cast<int>(r), static_cast<unsigned long long>(rows_total), box_rows);
    return KVZAP_OK;
}

// W1 [rows, d_model] bf16 (row-major) -> rows row0 .. row0+rows-1 of the K-blocked copy
// dst [d_model / 64][rows_total][64]; one thread moves 8 elements (16 bytes).
__global__ void pack_w1_kernel(const uint4 *__restrict__ W1, int rows, int d_model, int64_t rows_total, int64_t row0,
                               uint4 *__restrict__ dst)
{
    const int units_per_row = d_model / 8;
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= static_cast<int64_t>(rows) * units_per_row) return;
    const int r = static_cast<int>(idx / units_per_row), u = static_cast<int>(idx % units_per_row);
    const int kb = u / (kBlockK / 8), xu = u % (kBlockK / 8);
    dst[(static_cast<int64_t>(kb) * rows_total + row0 + r) * (kBlockK / 8) + xu] = W1[idx];
}

// The same for E4M3 bytes: 128 elements per K block, one thread moves 16 of them (16 bytes).
__global__ void pack_w1_fp8_kernel(const uint4 *__restrict__ W1, int rows, int d_model, int64_t rows_total, int64_t row0,
                                   uint4 *__restrict__ dst)
{
    const int units_per_row = d_model / 16;
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= static_cast<int64_t>(rows) * units_per_row) return;
    const int r = static_cast<int>(idx / units_per_row), u = static_cast<int>(idx % units_per_row);
    const int kb = u / 8, xu = u % 8;
    dst[(static_cast<int64_t>(kb) * rows_total + row0 + r) * 8 + xu] = W1[idx];
}

__global__ void add_int_kernel(int32_t *x, int n, int32_t delta)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) x[i] += delta;
}

// out[i] = src ? src[i] : 1 for i < n, 1 (unused rows) up to n_pad
__global__ void fill_scale_kernel(const float *__restrict__ src, int n, int n_pad, float *__restrict__ out)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_pad) out[i] = (src != nullptr && i < n) ? src[i] : 1.0f;
}

// W2 [H, hidden] bf16 -> w2t [hidden][8] fp32 (zero for heads >= H); b2 -> [8] fp32.
__global__ void pack_w2_kernel(const uint16_t *__restrict__ W2, const float *__restrict__ b2, int n_heads, int hidden,
                               float *__restrict__ w2t, float *__restrict__ b2p)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < hidden * kMaxHeads) {
        const int j = idx / kMaxHeads, h = idx % kMaxHeads;
        float v = 0.0f;
        if (h < n_heads) v = __uint_as_float(static_cast<uint32_t>(W2[static_cast<int64_t>(h) * hidden + j]) << 16);
        w2t[idx] = v;
    }
    if (idx < kMaxHeads) b2p[idx] = (b2 != nullptr && idx < n_heads) ? b2[idx] : 0.0f;
}

// NVTX range around a public call, for timelines; off unless the environment has KVZAP_NVTX=1 when the
// library is first used (the header-only NVTX does nothing without a tool attached).
static bool nvtx_enabled()
{
    static const bool on = [] { const char *v = getenv("KVZAP_NVTX"); return v != nullptr && v[0] == '1'; }();
    return on;
}
struct NvtxRange {
    bool on;
    explicit NvtxRange(const char *name) : on(nvtx_enabled()) { if (on) nvtxRangePushA(name); }
    ~NvtxRange() { if (on) nvtxRangePop(); }
};

// Brackets one kernel launch with events when profiling is on.
struct ProfScope {
    kvzap_ctx *ctx;
    cudaStream_t stream;
    cudaEvent_t stop = nullptr;
    ProfScope(kvzap_ctx *c, int kind, cudaStream_t s) : ctx(c), stream(s)
    {
        if (!ctx->profiling) return;
        cudaEvent_t start = nullptr;
        if (cudaEventCreate(&start) != cudaSuccess || cudaEventCreate(&stop) != cudaSuccess) { stop = nullptr; return; }
        cudaEventRecord(start, stream);
        ctx->prof.push_back({kind, start, stop});
    }
    ~ProfScope()
    {
        if (stop) cudaEventRecord(stop, stream);
    }
};

struct DeviceGuard {
    int prev = -1;
    bool ok = true, changed = false;
    explicit DeviceGuard(int dev)
    {
        ok = cudaGetDevice(&prev) == cudaSuccess;
        if (ok && prev != dev) {           // the usual case (already current) costs one query
            ok = cudaSetDevice(dev) == cudaSuccess;
            changed = true;
        }
    }
    ~DeviceGuard()
    {
        if (changed && prev >= 0) cudaSetDevice(prev);
    }
};

static void free_all(kvzap_ctx *ctx)
{
    cudaFree(ctx->w1_all);
    cudaFree(ctx->b1_all);
    cudaFree(ctx->w2t_all);
    cudaFree(ctx->b2_all);
    cudaFree(ctx->w1_fp8_all);
    cudaFree(ctx->w1_scale_all);
    cudaFree(ctx->maskbits);
    cudaFree(ctx->tile_counters);
    cudaFree(ctx->split_part);
    cudaFree(ctx->plan_scores);
    cudaFree(ctx->batch_map);
    cudaFree(ctx->select_hist);
    cudaFree(ctx->select_tau);
    cudaFree(ctx->split_arrive);
    cudaFree(ctx->wide_arrive);
    cudaFree(ctx->list_page0);
    cudaFree(ctx->list_base);
    cudaFree(ctx->op_mask); cudaFree(ctx->op_counts); cudaFree(ctx->op_len_acc);
    cudaFree(ctx->op_arrive); cudaFree(ctx->op_scan_flag); cudaFree(ctx->op_page0); cudaFree(ctx->lin_counts);
    cudaFree(ctx->status_dev);
    if (ctx->status_host) cudaFreeHost(ctx->status_host);
    for (auto &r : ctx->prof) { cudaEventDestroy(r.start); cudaEventDestroy(r.stop); }
    ctx->prof.clear();
    for (auto &g : ctx->stage) {
        cudaFree(g.x); cudaFree(g.k); cudaFree(g.v); cudaFree(g.ko); cudaFree(g.vo); cudaFree(g.scores);
        cudaFree(g.lengths); cudaFree(g.table); cudaFree(g.used);
        if (g.lengths_pinned) cudaFreeHost(g.lengths_pinned);
        if (g.copied_in) cudaEventDestroy(g.copied_in);
        if (g.computed) cudaEventDestroy(g.computed);
    }
    cudaFree(ctx->stage_cu);
    if (ctx->h2d_stream) cudaStreamDestroy(ctx->h2d_stream);
    if (ctx->d2h_stream) cudaStreamDestroy(ctx->d2h_stream);
}

static kvzap_status check_common(kvzap_ctx *ctx, int64_t n_tokens, int32_t n_seqs, const int32_t *cu_seqlens)
{
    if (n_tokens < 0) return fail(ctx, KVZAP_ERR_INVALID_ARG, "n_tokens is negative");
    if (n_tokens > ctx->cfg.max_tokens)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "n_tokens %lld exceeds the context's max_tokens %lld",
                    static_cast<long long>(n_tokens), static_cast<long long>(ctx->cfg.max_tokens));
    if (n_seqs < 1 || n_seqs > ctx->cfg.max_seqs)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "n_seqs %d outside 1..max_seqs (%d)", n_seqs, ctx->cfg.max_seqs);
    if (cu_seqlens == nullptr && n_seqs != 1)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "cu_seqlens is NULL but n_seqs is %d", n_seqs);
    return KVZAP_OK;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Tensor map of hidden states [slabs][rows][d_model] (box 128 x 64), from a small cache keyed by the
// buffer's address and shape.
static kvzap_status hidden_tmap(kvzap_ctx *ctx, CUtensorMap *out, const void *base, int64_t rows, int32_t slabs)
{
    for (const auto &e : ctx->tmap_cache)
        if (e.base == base && e.rows == rows && e.slabs == slabs) { *out = e.map; return KVZAP_OK; }
    kvzap_ctx::TmapEntry e;
    e.base = base; e.rows = rows; e.slabs = slabs;
    kvzap_status st = make_tmap(ctx, &e.map, base, static_cast<uint64_t>(rows), static_cast<uint64_t>(ctx->cfg.d_model),
                                kTileM, static_cast<uint64_t>(slabs));
    if (st != KVZAP_OK) return st;
    constexpr size_t kEntries = 128;
    if (ctx->tmap_cache.size() < kEntries) ctx->tmap_cache.push_back(e);
    else { ctx->tmap_cache[ctx->tmap_next] = e; ctx->tmap_next = (ctx->tmap_next + 1) % kEntries; }
    *out = e.map;
    return KVZAP_OK;
}

static uint32_t *next_mask_slice(kvzap_ctx *ctx)
{
    uint32_t *m = ctx->maskbits + (ctx->mask_turn % kMaskRing) * ctx->max_words * ctx->cfg.n_kv_heads;
    ctx->mask_turn += 1;
    return m;
}

// Fills a launch configuration; `early` adds the attribute that lets the kernel start before the
// kernel ahead of it in the stream has finished (programmatic dependent launch), `cluster` > 1 the
// cluster dimension.  `attrs` must have room for two attributes.
static void make_launch(cudaLaunchConfig_t *cfg, cudaLaunchAttribute *attrs, dim3 grid, dim3 block, size_t smem,
                        cudaStream_t stream, bool early, int cluster)
{
    memset(cfg, 0, sizeof *cfg);
    cfg->gridDim = grid;
    cfg->blockDim = block;
    cfg->dynamicSmemBytes = smem;
    cfg->stream = stream;
    int n = 0;
    if (cluster > 1) {
        attrs[n].id = cudaLaunchAttributeClusterDimension;
        attrs[n].val.clusterDim.x = static_cast<unsigned>(cluster);
        attrs[n].val.clusterDim.y = 1;
        attrs[n].val.clusterDim.z = 1;
        ++n;
    }
    if (early) {
        attrs[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attrs[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg->attrs = attrs;
    cfg->numAttrs = static_cast<unsigned>(n);
}

// What the compaction of a fused call works on; given to launch_score so that a launch which can do the
// compaction itself (KVzap-Linear, a short single sequence) does it.
struct CompactArgs {
    const void *K, *V;
    void *K_out, *V_out;
    int32_t *lengths;
    bool tok_major;
};

// Launches the scoring kernel over layers [layer, layer + n_layers); hidden is [n_layers][n_tokens][d_model],
// scores [n_layers][n_tokens][H]; maskbits != nullptr fuses the threshold/window test.
static kvzap_status launch_score(kvzap_ctx *ctx, int32_t layer, int32_t n_layers, const void *hidden, int64_t n_tokens,
                                 float *scores, uint32_t *maskbits, const int32_t *cu_seqlens, int32_t n_seqs,
                                 float tau, int32_t w, cudaStream_t stream, int32_t window_keep = 1,
                                 const DecodeFuse *fuse = nullptr, bool *fused = nullptr, bool fuse_chain = false,
                                 const CompactArgs *compact = nullptr, bool *compacted = nullptr,
                                 bool fp8 = false, const float *x_scale = nullptr)
{
    if (fused) *fused = false;
    if (compacted) *compacted = false;
    // Early start.  When the grid fills the machine (one CTA per SM), this kernel is allowed to start
    // while the kernels ahead of it in the stream -- the previous call's scoring kernel finishing its
    // last tiles, and its compaction -- are still running: its CTAs take the SMs as they become free.
    // That is safe because (a) it reads only hidden states and weights, which none of this library's
    // kernels write, (b) every scoring CTA waits for the kernel ahead of it before it exits, so a
    // free SM implies that everything two launches back has completed, and the mask slice written
    // here was last read at least kMaskRing launches back, (c) the scores buffer is checked below.
    // A smaller grid (or a scores buffer shared with the previous call) is started early as well, but
    // its epilogue waits for the kernel ahead before its first store (wait_before_write): loads and
    // MMAs of several small calls then overlap, and nothing is written while an earlier call may
    // still use it.
    const kvzap_config &c = ctx->cfg;
    const int64_t blocks_per_layer = (n_tokens + kTileM - 1) / kTileM;
    // the scores buffer may still be in use by a kernel of an earlier call that has not completed
    const bool scores_busy = scores != nullptr &&
                             hazard(ctx, scores, sizeof(float) * static_cast<size_t>(n_layers) * n_tokens * c.n_kv_heads, true);
    // Few tiles (a decode step: one tile per layer): split every tile's hidden units (and K range) over
    // several CTAs, so that the launch fills the machine and every CTA reads only its own part of W1.
    // ... and with the K split left out (two CTAs per tile, each a slice of the hidden units over the whole K
    // range) the same kernel serves launches of up to half as many tiles as there are SMs, where CTA pairs
    // would leave most SMs idle.
    const bool slices_only = ctx->split_n == 2 && ctx->split_k == 2 && fuse == nullptr && !fp8 &&
                             blocks_per_layer * n_layers * 4 > ctx->sm_count && blocks_per_layer * n_layers * 2 <= ctx->sm_count;
    if (fp8 && !(ctx->split8_ok && blocks_per_layer * n_layers * ctx->split_n * ctx->split_k <= ctx->sm_count))
        return fail(ctx, KVZAP_ERR_UNSUPPORTED, "8-bit few-token scoring: this shape has no four-CTA layout");
    if (ctx->split_n > 0 && (slices_only || blocks_per_layer * n_layers * ctx->split_n * ctx->split_k <= ctx->sm_count)) {
        // eight CTAs per tile when even those fit (not for the fused decode step, which is laid out for four)
        const bool wide = ctx->wide_n > 0 && fuse == nullptr && !fp8 &&
                          blocks_per_layer * n_layers * ctx->wide_n * ctx->wide_k <= ctx->sm_count;
        const int split_n = wide ? ctx->wide_n : ctx->split_n, split_k = wide ? ctx->wide_k : (slices_only ? 1 : ctx->split_k);
        CUtensorMap tmap_x;
        kvzap_status st = fp8 ? make_tmap8(ctx, &tmap_x, hidden, static_cast<uint64_t>(n_tokens), static_cast<uint64_t>(c.d_model),
                                           kTileM, static_cast<uint64_t>(n_layers), false)
                              : hidden_tmap(ctx, &tmap_x, hidden, n_tokens, n_layers);
        if (st != KVZAP_OK) return st;
        ScoreParams p;
        memset(&p, 0, sizeof p);
        p.x_scale = x_scale;
        p.w1_scale = ctx->w1_scale_all;
        p.n_tokens = n_tokens;
        p.n_tiles = static_cast<int32_t>(blocks_per_layer * n_layers);
        p.tiles_per_layer = static_cast<int32_t>(blocks_per_layer);
        p.blocks_per_layer = static_cast<int32_t>(blocks_per_layer);
        p.n_layers_call = n_layers;
        p.layer0 = layer;
        p.w_rows = ctx->w1_rows;
        p.d_model = c.d_model;
        p.group_w = p.chunk_n = c.hidden / split_n;
        p.n_groups = p.n_chunks = 1;
        p.n_stages = wide ? ctx->wide_stages : ctx->split_stages;
        p.acc_bufs = 1;
        p.tmem_cols = wide ? ctx->wide_tmem_cols : ctx->split_tmem_cols;
        p.n_hidden = c.hidden;
        p.n_heads = c.n_kv_heads;
        p.b1 = ctx->b1_all;
        p.w2t = ctx->w2t_all;
        p.b2 = ctx->b2_all;
        p.scores = scores;
        p.maskbits = maskbits;
        p.n_words = blocks_per_layer * 4;
        p.cu_seqlens = cu_seqlens;
        p.n_seqs = n_seqs;
        p.window = w;
        p.window_keep = window_keep;
        p.tau = tau;
        p.status = ctx->status_dev;
        p.split_part = ctx->split_part;
        p.split_arrive = wide ? ctx->wide_arrive : ctx->split_arrive;
        // Early start (consecutive decode steps): this kernel reads only hidden states and weights; the one
        // thing it may not do is write a scores buffer that the kernels of the previous call still read.
        const size_t sbytes = scores ? sizeof(float) * static_cast<size_t>(n_layers) * n_tokens * c.n_kv_heads : 0;
        bool clash = scores_busy;
        if (scores && ctx->last_scores) {
            const char *a0 = reinterpret_cast<const char *>(scores), *b0 = static_cast<const char *>(ctx->last_scores);
            clash = clash || (a0 < b0 + ctx->last_scores_bytes && b0 < a0 + sbytes);
        }
        ctx->last_scores = scores;
        ctx->last_scores_bytes = sbytes;
        const int n_ctas = split_n * split_k;
        DecodeFuse f;
        memset(&f, 0, sizeof f);
        const bool fuse_ok = fuse != nullptr && !ctx->profiling && n_ctas == 4;
        if (fuse_ok) {
            f = *fuse;
            f.enabled = 1;
            if (fused) *fused = true;
        }
        // The fused decode step touches the cache (counters, page allocator, rows) before it has waited for
        // the kernel ahead; its clusters order themselves through `done`, which covers earlier fused steps
        // only.  So it is started early only directly behind the fused step of the previous call on the
        // same cache (fuse_chain) -- never behind a prompt chunk's page assignment, a release or an export,
        // whose kernels it would race with -- and with a grid of at least half the SMs and its own scores
        // buffer.  Without the fused part the kernel reads nothing but hidden states and weights until
        // every thread has waited, and writes only after: it may always start early.
        const bool early = !ctx->profiling &&
                           (fuse_ok ? (fuse_chain && !clash && p.n_tiles * n_ctas * 2 >= ctx->sm_count) : true);
        p.wait_before_load = ctx->trusted ? 0 : 1;
        ctx->last_score_early = early;
        {
            ProfScope prof(ctx, KVZAP_KERNEL_SCORE, stream);
            cudaLaunchConfig_t cfg;
            cudaLaunchAttribute attrs[2];
            make_launch(&cfg, attrs, dim3(static_cast<unsigned>(p.n_tiles * n_ctas)), dim3(kScoreThreads),
                        wide ? ctx->wide_smem : ctx->split_smem, stream, early, split_k);
            if (fp8)
                KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, score_split_kernel<true>, tmap_x, ctx->split_tmap_w8, p, split_n, split_k, f));
            else
                KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, score_split_kernel<false>, tmap_x, wide ? ctx->wide_tmap_w : ctx->split_tmap_w, p,
                                                   split_n, split_k, f));
        }
        ctx->launches += 1;
        return KVZAP_OK;
    }
    // KVzap-Linear on few tiles (a short prompt, or a decode step): four CTAs share a tile, each a quarter
    // of the K range.  The kernel writes only after it has waited for the kernel ahead, so it may always
    // be placed early.
    // (with the compaction in the same launch the CTAs are small enough for several per SM: up to kLinMaxTiles tiles)
    const bool lin_one_launch = compact != nullptr && n_layers == 1 && n_seqs == 1 && maskbits != nullptr && window_keep == 1 &&
                                blocks_per_layer <= kLinMaxTiles && c.head_dim * 2 <= 2048;
    if (c.hidden == 0 && ctx->lin_split_ok &&
        (blocks_per_layer * n_layers * kLinSplit <= ctx->sm_count ||
         (lin_one_launch && blocks_per_layer * kLinSplit <= 2 * static_cast<int64_t>(ctx->sm_count)))) {
        CUtensorMap tmap_x;
        kvzap_status st = hidden_tmap(ctx, &tmap_x, hidden, n_tokens, n_layers);
        if (st != KVZAP_OK) return st;
        ScoreParams p;
        memset(&p, 0, sizeof p);
        p.n_tokens = n_tokens;
        p.n_tiles = static_cast<int32_t>(blocks_per_layer * n_layers);
        p.tiles_per_layer = static_cast<int32_t>(blocks_per_layer);
        p.blocks_per_layer = static_cast<int32_t>(blocks_per_layer);
        p.n_layers_call = n_layers;
        p.layer0 = layer;
        p.w_rows = ctx->w1_rows;
        p.d_model = c.d_model;
        p.n_heads = c.n_kv_heads;
        p.b1 = ctx->b1_all;
        p.scores = scores;
        p.maskbits = maskbits;
        p.n_words = blocks_per_layer * 4;
        p.cu_seqlens = cu_seqlens;
        p.n_seqs = n_seqs;
        p.window = w;
        p.window_keep = window_keep;
        p.tau = tau;
        p.status = ctx->status_dev;
        p.wait_before_load = ctx->trusted ? 0 : 1;
        const bool early = !ctx->profiling;
        // Writing before the kernel ahead has completed is safe only if (a) the scores buffer is not the
        // previous call's, and (b) the launch takes more than half of the SMs (one CTA each): then its
        // CTAs find room only as CTAs of the previous scoring launch exit, which they do after the
        // compaction two launches back has completed -- so the mask slice written here, last read
        // kMaskRing launches back, is free.
        const size_t sbytes = scores ? sizeof(float) * static_cast<size_t>(n_layers) * n_tokens * c.n_kv_heads : 0;
        bool clash = scores_busy;
        if (scores && ctx->last_scores) {
            const char *a0 = reinterpret_cast<const char *>(scores), *b0 = static_cast<const char *>(ctx->last_scores);
            clash = clash || (a0 < b0 + ctx->last_scores_bytes && b0 < a0 + sbytes);
        }
        p.wait_before_write = (clash || p.n_tiles * kLinSplit * 2 <= ctx->sm_count) ? 1 : 0;
        ctx->last_score_early = early;
        ctx->last_scores = scores;
        ctx->last_scores_bytes = sbytes;
        // Scoring and compaction in one launch: one layer, one sequence, the window kept, few enough tiles.
        LinCompact fc;
        memset(&fc, 0, sizeof fc);
        uint32_t smem = kLinSmemBytes;
        if (lin_one_launch) {
            const size_t kv_bytes = static_cast<size_t>(c.n_kv_heads) * n_tokens * c.head_dim * 2;
            const int set = static_cast<int>(ctx->op_turn % kOpRing);
            ctx->op_turn += 1;
            ctx->op_epoch = ctx->op_epoch == 0x7fffffff ? 1 : ctx->op_epoch + 1;
            // the same rule as for the one-launch pruning kernel: rows and counts are written before the work
            // ahead has completed only directly behind launches whose memory is on the pending list and does
            // not conflict
            bool wait_first = !ctx->trusted || ctx->profiling || ctx->op_last_seq + 1 != ctx->op_seq || ctx->op_chain >= kOpRing - 2 ||
                              clash;
            if (!wait_first)
                wait_first = hazard(ctx, hidden, static_cast<size_t>(n_tokens) * c.d_model * 2, false) ||
                             hazard(ctx, compact->K, kv_bytes, false) || hazard(ctx, compact->V, kv_bytes, false) ||
                             hazard(ctx, compact->K_out, kv_bytes, true) || hazard(ctx, compact->V_out, kv_bytes, true) ||
                             hazard(ctx, compact->lengths, sizeof(int32_t) * c.n_kv_heads, true);
            if (wait_first) serial_point(ctx);
            else ctx->op_chain += 1;
            ctx->op_last_seq = ctx->op_seq;
            note_range(ctx, hidden, static_cast<size_t>(n_tokens) * c.d_model * 2, false);
            note_range(ctx, scores, sbytes, true);
            note_range(ctx, compact->K, kv_bytes, false);
            note_range(ctx, compact->V, kv_bytes, false);
            note_range(ctx, compact->K_out, kv_bytes, true);
            note_range(ctx, compact->V_out, kv_bytes, true);
            note_range(ctx, compact->lengths, sizeof(int32_t) * c.n_kv_heads, true);
            fc.enabled = 1;
            fc.row_bytes = c.head_dim * 2;
            fc.K = static_cast<const char *>(compact->K);
            fc.V = static_cast<const char *>(compact->V);
            fc.K_out = static_cast<char *>(compact->K_out);
            fc.V_out = static_cast<char *>(compact->V_out);
            fc.in_stride_h = compact->tok_major ? 1 : n_tokens;
            fc.in_stride_t = compact->tok_major ? c.n_kv_heads : 1;
            fc.lengths = compact->lengths;
            fc.tile_counts = ctx->lin_counts + static_cast<size_t>(set) * kLinMaxTiles * kMaxHeads;
            fc.epoch = ctx->op_epoch;
            fc.n_stages = kLinStagesCompact;
            fc.wait_limit = ctx->wait_limit;
            p.wait_before_write = wait_first ? 1 : 0;
            p.maskbits = nullptr;
            smem = lin_smem_bytes(kLinStagesCompact);
            if (compacted) *compacted = true;
        }
        {
            ProfScope prof(ctx, KVZAP_KERNEL_SCORE, stream);
            cudaLaunchConfig_t cfg;
            cudaLaunchAttribute attrs[2];
            make_launch(&cfg, attrs, dim3(static_cast<unsigned>(p.n_tiles * kLinSplit)), dim3(kLinThreads), smem,
                        stream, early, kLinSplit);
            KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, score_linear_split_kernel, tmap_x, ctx->sched[0].tmap_w, p, fc));
        }
        ctx->launches += 1;
        return KVZAP_OK;
    }
    // CTA pairs pay off once a layer has at least two 128-token blocks; a pair's work tile is 256 tokens
    const bool pair = c.hidden > 0 && ctx->pair_clusters > 0 && blocks_per_layer >= 2;
    const kvzap_ctx::Schedule &sc = ctx->sched[pair ? 1 : 0];
    const int64_t tiles_per_layer = pair ? (blocks_per_layer + 1) / 2 : blocks_per_layer;
    const int64_t n_tiles = tiles_per_layer * n_layers;
    CUtensorMap tmap_x;
    kvzap_status st = hidden_tmap(ctx, &tmap_x, hidden, n_tokens, n_layers);
    if (st != KVZAP_OK) return st;
    ScoreParams p;
    memset(&p, 0, sizeof p);
    p.n_tokens = n_tokens;
    p.n_tiles = static_cast<int32_t>(n_tiles);
    p.tiles_per_layer = static_cast<int32_t>(tiles_per_layer);
    p.blocks_per_layer = static_cast<int32_t>(blocks_per_layer);
    p.n_layers_call = n_layers;
    p.layer0 = layer;
    p.w_rows = ctx->w1_rows;
    p.d_model = c.d_model;
    p.group_w = sc.group_w;
    p.n_groups = sc.n_groups;
    p.chunk_n = sc.chunk_n;
    p.n_chunks = sc.n_chunks;
    p.n_stages = sc.n_stages;
    p.acc_bufs = sc.acc_bufs;
    p.acc_stride = sc.acc_stride;
    p.tmem_cols = sc.tmem_cols;
    p.n_hidden = c.hidden;
    p.n_heads = c.n_kv_heads;
    p.b1 = ctx->b1_all;
    p.w2t = ctx->w2t_all;
    p.b2 = ctx->b2_all;
    p.scores = scores;
    p.maskbits = maskbits;
    p.n_words = blocks_per_layer * 4;
    p.cu_seqlens = cu_seqlens;
    p.n_seqs = n_seqs;
    p.window = w;
    p.window_keep = window_keep;
    p.tau = tau;
    p.status = ctx->status_dev;
    p.wait_before_load = ctx->trusted ? 0 : 1;
    // every launch finds its counter at zero: it was cleared by the launch before the previous one
    p.tile_counter = ctx->tile_counters + ctx->score_turn % kMaskRing;
    p.tile_counter_reset = ctx->tile_counters + (ctx->score_turn + 2) % kMaskRing;
    ctx->score_turn += 1;
    const size_t scores_bytes = scores ? sizeof(float) * static_cast<size_t>(n_layers) * n_tokens * c.n_kv_heads : 0;
    bool scores_clash = scores_busy;     // the previous launch may still be writing the same buffer
    if (scores && ctx->last_scores) {
        const char *a0 = reinterpret_cast<const char *>(scores), *b0 = static_cast<const char *>(ctx->last_scores);
        scores_clash = scores_clash || (a0 < b0 + ctx->last_scores_bytes && b0 < a0 + scores_bytes);
    }
    ctx->last_scores = scores;
    ctx->last_scores_bytes = scores_bytes;
    ctx->last_score_early = false;       // (only the decode step's update kernel looks at this)
    {
        ProfScope prof(ctx, KVZAP_KERNEL_SCORE, stream);
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attrs[2];
        if (pair) {
            const int n_clusters = static_cast<int>(n_tiles < ctx->pair_clusters ? n_tiles : ctx->pair_clusters);
            const bool early = !ctx->profiling;
            p.wait_before_write = (scores_clash || 2 * n_clusters < ctx->sm_count / 2 * 2) ? 1 : 0;
            make_launch(&cfg, attrs, dim3(static_cast<unsigned>(2 * n_clusters)), dim3(kScoreThreads), sc.smem, stream,
                        early, 2);
            KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, score_kernel<true, true>, tmap_x, sc.tmap_w, p));
        } else {
            const int grid = static_cast<int>(n_tiles < ctx->sm_count ? n_tiles : ctx->sm_count);
            const bool early = !ctx->profiling;
            p.wait_before_write = (scores_clash || grid < ctx->sm_count) ? 1 : 0;
            make_launch(&cfg, attrs, dim3(static_cast<unsigned>(grid)), dim3(kScoreThreads), sc.smem, stream, early, 1);
            if (c.hidden > 0)
                KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, score_kernel<true, false>, tmap_x, sc.tmap_w, p));
            else
                KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, score_kernel<false, false>, tmap_x, sc.tmap_w, p));
        }
    }
    KVZAP_CUDA(ctx, cudaGetLastError());
    ctx->launches += 1;
    return KVZAP_OK;
}

// Scoring with 8-bit inputs: hidden [n_tokens][d_model] E4M3 bytes with one scale per token, the layer's first-layer
// weights given by kvzap_set_weights_fp8.  Always the persistent kernel (CTA pairs for the MLP from two blocks on);
// the waits before loads and stores follow the rules of launch_score.
static kvzap_status launch_score_fp8(kvzap_ctx *ctx, int32_t layer, const void *hidden8, const float *x_scale, int64_t n_tokens,
                                     float *scores, uint32_t *maskbits, const int32_t *cu_seqlens, int32_t n_seqs, float tau,
                                     int32_t w, cudaStream_t stream)
{
    const kvzap_config &c = ctx->cfg;
    const int64_t blocks_per_layer = (n_tokens + kTileM - 1) / kTileM;
    const bool pair = c.hidden > 0 && ctx->pair_clusters > 0 && blocks_per_layer >= 2;
    const kvzap_ctx::Schedule &sc = ctx->sched[pair ? 1 : 0];
    const int64_t n_tiles = pair ? (blocks_per_layer + 1) / 2 : blocks_per_layer;
    CUtensorMap tmap_x;
    kvzap_status st = make_tmap8(ctx, &tmap_x, hidden8, static_cast<uint64_t>(n_tokens), static_cast<uint64_t>(c.d_model), kTileM, 1, false);
    if (st != KVZAP_OK) return st;
    ScoreParams p;
    memset(&p, 0, sizeof p);
    p.n_tokens = n_tokens;
    p.n_tiles = static_cast<int32_t>(n_tiles);
    p.tiles_per_layer = static_cast<int32_t>(n_tiles);
    p.blocks_per_layer = static_cast<int32_t>(blocks_per_layer);
    p.n_layers_call = 1;
    p.layer0 = layer;
    p.w_rows = ctx->w1_rows;
    p.d_model = c.d_model;
    p.group_w = sc.group_w;
    p.n_groups = sc.n_groups;
    p.chunk_n = sc.chunk_n;
    p.n_chunks = sc.n_chunks;
    p.n_stages = sc.n_stages;
    p.acc_bufs = sc.acc_bufs;
    p.acc_stride = sc.acc_stride;
    p.tmem_cols = sc.tmem_cols;
    p.n_hidden = c.hidden;
    p.n_heads = c.n_kv_heads;
    p.b1 = ctx->b1_all;
    p.w2t = ctx->w2t_all;
    p.b2 = ctx->b2_all;
    p.scores = scores;
    p.maskbits = maskbits;
    p.n_words = blocks_per_layer * 4;
    p.cu_seqlens = cu_seqlens;
    p.n_seqs = n_seqs;
    p.window = w;
    p.window_keep = 1;
    p.tau = tau;
    p.status = ctx->status_dev;
    p.wait_before_load = ctx->trusted ? 0 : 1;
    p.k_blocks = c.d_model / 128;
    p.k_elems = 128;
    p.x_scale = x_scale;
    p.w1_scale = ctx->w1_scale_all;
    p.tile_counter = ctx->tile_counters + ctx->score_turn % kMaskRing;
    p.tile_counter_reset = ctx->tile_counters + (ctx->score_turn + 2) % kMaskRing;
    ctx->score_turn += 1;
    const size_t scores_bytes = scores ? sizeof(float) * static_cast<size_t>(n_tokens) * c.n_kv_heads : 0;
    bool scores_clash = scores != nullptr && hazard(ctx, scores, scores_bytes, true);
    if (scores && ctx->last_scores) {
        const char *a0 = reinterpret_cast<const char *>(scores), *b0 = static_cast<const char *>(ctx->last_scores);
        scores_clash = scores_clash || (a0 < b0 + ctx->last_scores_bytes && b0 < a0 + scores_bytes);
    }
    ctx->last_scores = scores;
    ctx->last_scores_bytes = scores_bytes;
    ctx->last_score_early = false;
    {
        ProfScope prof(ctx, KVZAP_KERNEL_SCORE, stream);
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attrs[2];
        const bool early = !ctx->profiling;
        if (pair) {
            const int n_clusters = static_cast<int>(n_tiles < ctx->pair_clusters ? n_tiles : ctx->pair_clusters);
            p.wait_before_write = (scores_clash || 2 * n_clusters < ctx->sm_count / 2 * 2) ? 1 : 0;
            make_launch(&cfg, attrs, dim3(static_cast<unsigned>(2 * n_clusters)), dim3(kScoreThreads), sc.smem, stream, early, 2);
            KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, score_kernel<true, true, true>, tmap_x, ctx->tmap_w8[1], p));
        } else {
            const int grid = static_cast<int>(n_tiles < ctx->sm_count ? n_tiles : ctx->sm_count);
            p.wait_before_write = (scores_clash || grid < ctx->sm_count) ? 1 : 0;
            make_launch(&cfg, attrs, dim3(static_cast<unsigned>(grid)), dim3(kScoreThreads), sc.smem, stream, early, 1);
            if (c.hidden > 0)
                KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, score_kernel<true, false, true>, tmap_x, ctx->tmap_w8[0], p));
            else
                KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, score_kernel<false, false, true>, tmap_x, ctx->tmap_w8[0], p));
        }
    }
    ctx->launches += 1;
    return KVZAP_OK;
}

// Dense-ragged compaction over the mask words in `mask` (one kernel, no scan pass).
static kvzap_status launch_compaction(kvzap_ctx *ctx, const uint32_t *mask, const void *K, const void *V,
                                      const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens, void *K_out,
                                      void *V_out, int32_t *lengths, cudaStream_t stream, bool beside_scoring = true,
                                      bool tok_major = false)
{
    const kvzap_config &c = ctx->cfg;
    const int64_t n_blocks = (n_tokens + kBlockTokens - 1) / kBlockTokens;
    const int64_t n_words = n_blocks * 4;
    // A grid that is resident all at once, next to the scoring kernel's CTAs: the MLP scoring kernel
    // leaves registers for two of these CTAs per SM, the Linear one for several.
    // On its own (kvzap_prune_prefill) the kernel fills every SM instead: eight CTAs each.
    const int per_sm = !beside_scoring ? 8 : (c.hidden > 0 ? 2 : 6);
    const int64_t max_ctas = static_cast<int64_t>(ctx->sm_count) * per_sm;
    int64_t chunks = max_ctas / c.n_kv_heads;
    if (chunks < 1) chunks = 1;
    if (chunks > n_blocks) chunks = n_blocks;
    const int blocks_per_cta = static_cast<int>((n_blocks + chunks - 1) / chunks);
    chunks = (n_blocks + blocks_per_cta - 1) / blocks_per_cta;
    {
        ProfScope prof(ctx, KVZAP_KERNEL_COMPACT, stream);
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attrs[2];
        // a short input (one block per CTA, a grid that is resident at once anyway): CTAs of 256 threads
        const bool short_input = blocks_per_cta == 1 && chunks * c.n_kv_heads <= 4 * static_cast<int64_t>(ctx->sm_count);
        make_launch(&cfg, attrs, dim3(static_cast<unsigned>(chunks), static_cast<unsigned>(c.n_kv_heads)),
                    dim3(short_input ? kDenseThreadsShort : kDenseThreads), 0, stream, !ctx->profiling, 1);
        KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, short_input ? compact_dense_kernel<kDenseThreadsShort> : compact_dense_kernel<kDenseThreads>,
                                           static_cast<const uint4 *>(K),
                                           static_cast<const uint4 *>(V), static_cast<uint4 *>(K_out),
                                           static_cast<uint4 *>(V_out), mask, n_words, n_blocks, blocks_per_cta,
                                           cu_seqlens, n_seqs, n_tokens, c.n_kv_heads, c.head_dim / 8, lengths, 0,
                                           static_cast<const int32_t *>(nullptr),
                                           tok_major ? int64_t{1} : n_tokens,
                                           tok_major ? static_cast<int64_t>(c.n_kv_heads) : int64_t{1},
                                           static_cast<const int32_t *>(nullptr), static_cast<const int32_t *>(nullptr), 0,
                                           static_cast<const int64_t *>(nullptr)));
    }
    ctx->launches += 1;
    return KVZAP_OK;
}

// Threshold / window mask, counts, prefix sums and the ordered gather in one launch (prune_onepass_kernel),
// dense-ragged (page_tokens == 0) or paged.  tau_list != nullptr: a threshold per list, written by the
// kernel ahead in the stream.
static kvzap_status launch_prune_onepass(kvzap_ctx *ctx, const float *scores, const float *tau_list, float tau, int32_t w,
                                         const void *K, const void *V, const int32_t *cu_seqlens, int32_t n_seqs,
                                         int64_t n_tokens, void *K_out, void *V_out, int32_t *lengths, int32_t page_tokens,
                                         int32_t first_page, int64_t n_pages_pool, int32_t max_pages, int32_t *page_table,
                                         int32_t *n_pages_used, cudaStream_t stream, int32_t *slot_out = nullptr,
                                         bool scores_just_made = false)
{
    const kvzap_config &c = ctx->cfg;
    if (page_tokens > 0 && n_pages_pool * page_tokens >= 0xffffffffLL)
        return fail(ctx, KVZAP_ERR_UNSUPPORTED, "paged pruning: the pool must hold fewer than 2^32 - 1 rows");
    const int64_t n_blocks = (n_tokens + kBlockTokens - 1) / kBlockTokens;
    // Heads per CTA: as many as still leave a CTA a dozen blocks or more.  The one CTA that holds a sequence's window
    // keeps all rows of a block where the others keep a quarter or a third; with many blocks per CTA that is a small
    // surplus, with two or three it would make that CTA the last to finish by far.
    int heads_per_cta = kMaxHeads, groups = 1;
    int64_t grid = 1, per_cta = n_blocks;
    for (int hg = kMaxHeads; hg >= 1; hg >>= 1) {
        heads_per_cta = hg;
        groups = (c.n_kv_heads + hg - 1) / hg;
        grid = ctx->op_capacity / groups;
        if (grid < 1) grid = 1;
        if (grid > n_blocks) grid = n_blocks;
        per_cta = (n_blocks + grid - 1) / grid;
        grid = (n_blocks + per_cta - 1) / per_cta;
        if (per_cta >= 12) break;
    }
    const int set = static_cast<int>(ctx->op_turn % kOpRing);
    ctx->op_turn += 1;
    ctx->op_epoch = ctx->op_epoch == 0x7fffffff ? 1 : ctx->op_epoch + 1;
    const size_t n_lists = static_cast<size_t>(n_seqs) * c.n_kv_heads;
    const size_t kv_bytes = static_cast<size_t>(c.n_kv_heads) * n_tokens * c.head_dim * 2;
    const size_t out_bytes = page_tokens > 0 ? static_cast<size_t>(n_pages_pool) * page_tokens * c.head_dim * 2 : kv_bytes;
    const size_t sc_bytes = sizeof(float) * static_cast<size_t>(n_tokens) * c.n_kv_heads;
    // Started before the work ahead of it has completed only on a context that trusts its producers,
    // directly behind another launch of this kernel (whose memory is on the pending list, and whose scratch
    // set is a different one for kOpRing - 2 launches in a row), and when it conflicts with none of them.
    bool wait_first = !ctx->trusted || ctx->profiling || tau_list != nullptr || scores_just_made ||
                      ctx->op_last_seq + 1 != ctx->op_seq || ctx->op_chain >= kOpRing - 2;
    if (!wait_first)
        wait_first = hazard(ctx, scores, sc_bytes, false) || hazard(ctx, K, kv_bytes, false) || hazard(ctx, V, kv_bytes, false) ||
                     hazard(ctx, cu_seqlens, sizeof(int32_t) * (n_seqs + 1), false) ||
                     hazard(ctx, K_out, out_bytes, true) || hazard(ctx, V_out, out_bytes, true) ||
                     hazard(ctx, lengths, sizeof(int32_t) * n_lists, true) ||
                     hazard(ctx, page_table, sizeof(int32_t) * n_lists * max_pages, true) ||
                     hazard(ctx, n_pages_used, sizeof(int32_t), true) ||
                     hazard(ctx, slot_out, sizeof(int32_t) * static_cast<size_t>(n_tokens) * c.n_kv_heads, true);
    if (wait_first) serial_point(ctx);
    else ctx->op_chain += 1;
    ctx->op_last_seq = ctx->op_seq;
    note_range(ctx, scores, sc_bytes, false);
    note_range(ctx, K, kv_bytes, false);
    note_range(ctx, V, kv_bytes, false);
    note_range(ctx, K_out, out_bytes, true);
    note_range(ctx, V_out, out_bytes, true);
    note_range(ctx, lengths, sizeof(int32_t) * n_lists, true);
    note_range(ctx, slot_out, sizeof(int32_t) * static_cast<size_t>(n_tokens) * c.n_kv_heads, true);
    if (page_tokens > 0) {
        note_range(ctx, page_table, sizeof(int32_t) * n_lists * max_pages, true);
        note_range(ctx, n_pages_used, sizeof(int32_t), true);
    }
    PruneParams p;
    memset(&p, 0, sizeof p);
    p.scores = scores;
    p.tau_list = tau_list;
    p.tau = tau;
    p.window = w;
    p.n_tokens = n_tokens;
    p.n_blocks = n_blocks;
    p.n_words = n_blocks * 4;
    p.n_heads = c.n_kv_heads;
    p.n_seqs = n_seqs;
    p.cu_seqlens = cu_seqlens;
    p.blocks_per_cta = static_cast<int32_t>(per_cta);
    p.heads_per_cta = heads_per_cta;
    p.K = static_cast<const uint4 *>(K);
    p.V = static_cast<const uint4 *>(V);
    p.K_out = static_cast<uint4 *>(K_out);
    p.V_out = static_cast<uint4 *>(V_out);
    p.in_stride_h = n_tokens;
    p.in_stride_t = 1;
    p.row_units = c.head_dim / 8;
    p.lengths = lengths;
    p.slot_out = slot_out;
    p.page_tokens = page_tokens;
    p.first_page = first_page;
    p.max_pages = max_pages;
    p.n_pages_pool = n_pages_pool;
    p.list_page0 = ctx->op_page0 + static_cast<size_t>(set) * c.max_seqs * c.n_kv_heads;
    p.page_table = page_table;
    p.n_pages_used = n_pages_used;
    p.status = ctx->status_dev;
    p.maskbits = ctx->op_mask + static_cast<size_t>(set) * ctx->max_words * c.n_kv_heads;
    p.cta_counts = ctx->op_counts + static_cast<size_t>(set) * ctx->op_capacity * kMaxHeads;
    p.len_acc = ctx->op_len_acc + static_cast<size_t>(set) * c.max_seqs * c.n_kv_heads;
    p.arrive = ctx->op_arrive + set;
    p.scan_flag = ctx->op_scan_flag + set;
    p.epoch = ctx->op_epoch;
    p.wait_limit = ctx->wait_limit;
    p.wait_first = wait_first ? 1 : 0;
    {
        ProfScope prof(ctx, KVZAP_KERNEL_COMPACT, stream);
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attrs[2];
        make_launch(&cfg, attrs, dim3(static_cast<unsigned>(grid), static_cast<unsigned>(groups)), dim3(kOpThreads), kOpDynSmem,
                    stream, !ctx->profiling, 1);
        KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, prune_onepass_kernel<kOpRows>, p));
    }
    ctx->launches += 1;
    return KVZAP_OK;
}

static kvzap_status check_prune_args(kvzap_ctx *ctx, const void *K, const void *V, const void *K_out,
                                     const void *V_out, const int32_t *lengths, int32_t w)
{
    if (!K || !V || !K_out || !V_out || !lengths)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "K, V, K_out, V_out and lengths must not be NULL");
    if (!aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out))
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "K/V pointers must be 16-byte aligned");
    if (w < 0) return fail(ctx, KVZAP_ERR_INVALID_ARG, "window w is negative");
    return KVZAP_OK;
}

}  // namespace kvzap

using namespace kvzap;

extern "C" {

kvzap_status kvzap_create(kvzap_ctx **out, const kvzap_config *cfg)
{
    if (!out) return fail(nullptr, KVZAP_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (!cfg) return fail(nullptr, KVZAP_ERR_INVALID_ARG, "cfg is NULL");
    const kvzap_config c = *cfg;
    if (c.d_model < 64 || c.d_model > 16384 || c.d_model % 64)
        return fail(nullptr, KVZAP_ERR_UNSUPPORTED, "d_model %d: need a multiple of 64 in 64..16384", c.d_model);
    if (c.hidden < 0 || c.hidden > 1024 || (c.hidden <= 512 && c.hidden % 64) || (c.hidden > 512 && c.hidden % 128))
        return fail(nullptr, KVZAP_ERR_UNSUPPORTED,
                    "hidden %d: need 0, a multiple of 64 up to 512, or a multiple of 128 up to 1024", c.hidden);
    if (c.n_kv_heads < 1 || c.n_kv_heads > kMaxHeads)
        return fail(nullptr, KVZAP_ERR_UNSUPPORTED, "n_kv_heads %d: need 1..8", c.n_kv_heads);
    if (c.head_dim < 8 || c.head_dim > 1024 || c.head_dim % 8)
        return fail(nullptr, KVZAP_ERR_UNSUPPORTED, "head_dim %d: need a multiple of 8 in 8..1024", c.head_dim);
    if (c.n_layers < 1) return fail(nullptr, KVZAP_ERR_INVALID_ARG, "n_layers %d: need >= 1", c.n_layers);
    if (c.max_tokens < 1 || c.max_tokens > (int64_t(1) << 30))
        return fail(nullptr, KVZAP_ERR_INVALID_ARG, "max_tokens out of range (1..2^30)");
    if (c.max_seqs < 1 || c.max_seqs > (1 << 20))
        return fail(nullptr, KVZAP_ERR_INVALID_ARG, "max_seqs out of range (1..2^20)");
    if (c.flags & ~KVZAP_FLAG_TRUSTED_PRODUCERS)
        return fail(nullptr, KVZAP_ERR_INVALID_ARG, "flags 0x%x: unknown bits set", static_cast<unsigned>(c.flags));

    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || c.device < 0 || c.device >= n_dev)
        return fail(nullptr, KVZAP_ERR_CUDA, "CUDA device %d not available (%d devices)", c.device, n_dev);
    DeviceGuard guard(c.device);
    if (!guard.ok) return fail(nullptr, KVZAP_ERR_CUDA, "cudaSetDevice(%d) failed", c.device);
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, c.device) != cudaSuccess)
        return fail(nullptr, KVZAP_ERR_CUDA, "cudaGetDeviceProperties failed");
    if (prop.major != 10)
        return fail(nullptr, KVZAP_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library is built for sm_100a only",
                    c.device, prop.major, prop.minor);

    kvzap_ctx *ctx = new (std::nothrow) kvzap_ctx();
    if (!ctx) return fail(nullptr, KVZAP_ERR_CUDA, "out of host memory");
    ctx->cfg = c;
    ctx->trusted = (c.flags & KVZAP_FLAG_TRUSTED_PRODUCERS) != 0;
    ctx->sm_count = prop.multiProcessorCount;

    // scoring schedules
    const int budget = static_cast<int>(prop.sharedMemPerBlockOptin) - 1024;
    for (int mode = 0; mode < (c.hidden > 0 ? 2 : 1); ++mode) {
        kvzap_ctx::Schedule &sc = ctx->sched[mode];
        if (c.hidden == 0) {
            ctx->w1_rows = 16;            // H <= 8 outputs padded to the smallest N of a 128-row MMA
            sc.group_w = 16; sc.n_groups = 1; sc.chunk_n = 16; sc.n_chunks = 1;
            sc.acc_bufs = 2; sc.acc_stride = 32;
        } else {
            ctx->w1_rows = c.hidden;
            sc.n_groups = c.hidden > 512 ? 2 : 1;
            sc.group_w = c.hidden / sc.n_groups;
            sc.n_chunks = sc.group_w > 256 ? 2 : 1;
            sc.chunk_n = sc.group_w / sc.n_chunks;
            sc.acc_bufs = 512 / sc.group_w >= 2 ? 2 : 1;
            sc.acc_stride = sc.group_w;
        }
        sc.tmem_cols = next_pow2(sc.acc_bufs * sc.acc_stride);
        const int b_rows = sc.group_w / (mode + 1);
        int stages = kMaxStages;
        for (; stages >= 2; --stages)
            if (static_cast<int>(score_smem_layout(b_rows, stages, c.hidden).total) <= budget) break;
        if (stages < 2) {
            delete ctx;
            return fail(nullptr, KVZAP_ERR_UNSUPPORTED, "shared memory too small for this surrogate shape");
        }
        sc.n_stages = stages;
        sc.smem = score_smem_layout(b_rows, stages, c.hidden).total + 1024;
    }

#define CREATE_CUDA(call)                                                                              \
    do {                                                                                               \
        cudaError_t e_ = (call);                                                                       \
        if (e_ != cudaSuccess) {                                                                       \
            fail(nullptr, KVZAP_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));             \
            free_all(ctx);                                                                             \
            delete ctx;                                                                                \
            return KVZAP_ERR_CUDA;                                                                     \
        }                                                                                              \
    } while (0)

    {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        CREATE_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (q != cudaDriverEntryPointSuccess || fn == nullptr) {
            delete ctx;
            return fail(nullptr, KVZAP_ERR_CUDA, "driver entry point cuTensorMapEncodeTiled not found");
        }
        ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    if (c.hidden > 0) {
        CREATE_CUDA(cudaFuncSetAttribute(score_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(ctx->sched[0].smem)));
        CREATE_CUDA(cudaFuncSetAttribute(score_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(ctx->sched[1].smem)));
        // how many CTA pairs fit on the device at once (one CTA per SM, both SMs of a pair adjacent)
        cudaLaunchConfig_t qcfg;
        memset(&qcfg, 0, sizeof qcfg);
        qcfg.gridDim = dim3(static_cast<unsigned>(ctx->sm_count / 2 * 2));
        qcfg.blockDim = dim3(kScoreThreads);
        qcfg.dynamicSmemBytes = ctx->sched[1].smem;
        cudaLaunchAttribute qattr[1];
        qattr[0].id = cudaLaunchAttributeClusterDimension;
        qattr[0].val.clusterDim.x = 2;
        qattr[0].val.clusterDim.y = 1;
        qattr[0].val.clusterDim.z = 1;
        qcfg.attrs = qattr;
        qcfg.numAttrs = 1;
        int n_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&n_clusters, score_kernel<true, true>, &qcfg) == cudaSuccess && n_clusters > 0)
            ctx->pair_clusters = n_clusters < ctx->sm_count / 2 ? n_clusters : ctx->sm_count / 2;
        else
            cudaGetLastError();          // pairs unavailable: the one-CTA kernel serves every size
    } else {
        CREATE_CUDA(cudaFuncSetAttribute(score_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(ctx->sched[0].smem)));
    }

    // Kernels share an SM only if they ask for the same split of the L1 / shared-memory array; the
    // scoring kernels need the largest shared-memory split, so the compaction asks for it too.
    CREATE_CUDA(cudaFuncSetAttribute(compact_dense_kernel<kDenseThreads>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     static_cast<int>(cudaSharedmemCarveoutMaxShared)));
    CREATE_CUDA(cudaFuncSetAttribute(compact_dense_kernel<kDenseThreadsShort>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     static_cast<int>(cudaSharedmemCarveoutMaxShared)));
    CREATE_CUDA(cudaFuncSetAttribute(decode_update_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     static_cast<int>(cudaSharedmemCarveoutMaxShared)));
    if (c.hidden > 0)
        CREATE_CUDA(cudaFuncSetAttribute(score_split_kernel<false>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                         static_cast<int>(cudaSharedmemCarveoutMaxShared)));
    if (c.hidden > 0) {
        CREATE_CUDA(cudaFuncSetAttribute(score_kernel<true, false>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                         static_cast<int>(cudaSharedmemCarveoutMaxShared)));
        CREATE_CUDA(cudaFuncSetAttribute(score_kernel<true, true>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                         static_cast<int>(cudaSharedmemCarveoutMaxShared)));
    } else {
        CREATE_CUDA(cudaFuncSetAttribute(score_kernel<false, false>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                         static_cast<int>(cudaSharedmemCarveoutMaxShared)));
        if ((c.d_model / kBlockK) % kLinSplit == 0 && static_cast<int>(kLinSmemBytes) <= budget + 1024) {
            CREATE_CUDA(cudaFuncSetAttribute(score_linear_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(kLinSmemBytes)));
            CREATE_CUDA(cudaFuncSetAttribute(score_linear_split_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                             static_cast<int>(cudaSharedmemCarveoutMaxShared)));
            ctx->lin_split_ok = true;
        }
    }

    ctx->layer_set.assign(c.n_layers, 0);
    ctx->layer_fp8.assign(c.n_layers, 0);
    {
        const size_t w1_bytes = static_cast<size_t>(c.n_layers) * ctx->w1_rows * c.d_model * 2;
        CREATE_CUDA(cudaMalloc(&ctx->w1_all, w1_bytes));
        CREATE_CUDA(cudaMemset(ctx->w1_all, 0, w1_bytes));
        CREATE_CUDA(cudaMalloc(&ctx->b1_all, sizeof(float) * c.n_layers * ctx->w1_rows));
        CREATE_CUDA(cudaMemset(ctx->b1_all, 0, sizeof(float) * c.n_layers * ctx->w1_rows));
        if (c.hidden > 0) {
            CREATE_CUDA(cudaMalloc(&ctx->w2t_all, sizeof(float) * c.n_layers * c.hidden * kMaxHeads));
            CREATE_CUDA(cudaMalloc(&ctx->b2_all, sizeof(float) * c.n_layers * kMaxHeads));
        }
        ctx->err[0] = 0;
        for (int mode = 0; mode < (c.hidden > 0 ? 2 : 1); ++mode) {
            kvzap_ctx::Schedule &sc = ctx->sched[mode];
            if (make_tmap_w(ctx, &sc.tmap_w, ctx->w1_all, static_cast<uint64_t>(c.n_layers) * ctx->w1_rows,
                            static_cast<uint64_t>(c.d_model / kBlockK), static_cast<uint32_t>(sc.chunk_n / (mode + 1))) != KVZAP_OK) {
                snprintf(g_create_error, sizeof g_create_error, "%s", ctx->err);
                free_all(ctx);
                delete ctx;
                return KVZAP_ERR_CUDA;
            }
        }
    }
    if (c.hidden > 0) {
        // few-token schedule: four CTAs per tile.  2 x 2 (two slices of hidden units, two halves of K) when
        // a slice of hidden / 2 units fits one MMA and the K blocks divide evenly, else four slices.
        const bool two_by_two = c.hidden / 2 <= 256 && (c.hidden / 4) % 16 == 0 && (c.d_model / kBlockK) % 2 == 0;
        const int n_split = two_by_two ? 2 : 4, k_split = two_by_two ? 2 : 1, ns = c.hidden / n_split;
        int stages = kMaxStages;
        for (; stages >= 2; --stages)
            if (static_cast<int>(split_smem_layout(ns, stages, 4).total) <= budget - 4096) break;   // 4 KB static
        if (stages >= 2 && ns % 16 == 0 && ns <= 256) {
            ctx->split_stages = stages;
            ctx->split_smem = split_smem_layout(ns, stages, 4).total + 1024;
            ctx->split_tmem_cols = next_pow2(ns);
            CREATE_CUDA(cudaFuncSetAttribute(score_split_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(ctx->split_smem)));
            if (make_tmap_w(ctx, &ctx->split_tmap_w, ctx->w1_all, static_cast<uint64_t>(c.n_layers) * ctx->w1_rows,
                            static_cast<uint64_t>(c.d_model / kBlockK), static_cast<uint32_t>(ns)) == KVZAP_OK) {
                ctx->split_n = n_split;
                ctx->split_k = k_split;
            }
        }
        // 4 x 2: slices of hidden / 4 units, each CTA finishing hidden / 8 of them
        const int ns8 = c.hidden / 4;
        if (ctx->split_n > 0 && c.hidden % 128 == 0 && ns8 <= 256 && (c.d_model / kBlockK) % 2 == 0) {
            int st8 = kMaxStages;
            for (; st8 >= 2; --st8)
                if (static_cast<int>(split_smem_layout(ns8, st8, 8).total) <= budget - 4096) break;
            if (st8 >= 2) {
                ctx->wide_stages = st8;
                ctx->wide_smem = split_smem_layout(ns8, st8, 8).total + 1024;
                ctx->wide_tmem_cols = next_pow2(ns8);
                if (ctx->wide_smem > ctx->split_smem)
                    CREATE_CUDA(cudaFuncSetAttribute(score_split_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     static_cast<int>(ctx->wide_smem)));
                if (make_tmap_w(ctx, &ctx->wide_tmap_w, ctx->w1_all, static_cast<uint64_t>(c.n_layers) * ctx->w1_rows,
                                static_cast<uint64_t>(c.d_model / kBlockK), static_cast<uint32_t>(ns8)) == KVZAP_OK) {
                    ctx->wide_n = 4;
                    ctx->wide_k = 2;
                }
            }
        }
    }
    ctx->max_blocks = (c.max_tokens + kBlockTokens - 1) / kBlockTokens;
    ctx->max_words = ctx->max_blocks * 4;
    CREATE_CUDA(cudaMalloc(&ctx->maskbits, sizeof(uint32_t) * kMaskRing * ctx->max_words * c.n_kv_heads));
    CREATE_CUDA(cudaMalloc(&ctx->list_page0, sizeof(int32_t) * static_cast<int64_t>(c.max_seqs) * c.n_kv_heads));
    CREATE_CUDA(cudaMalloc(&ctx->list_base, sizeof(int32_t) * static_cast<int64_t>(c.max_seqs) * c.n_kv_heads));
    CREATE_CUDA(cudaMalloc(&ctx->tile_counters, sizeof(int32_t) * kMaskRing));
    CREATE_CUDA(cudaMemset(ctx->tile_counters, 0, sizeof(int32_t) * kMaskRing));
    CREATE_CUDA(cudaMalloc(&ctx->select_hist, sizeof(uint32_t) * 4 * static_cast<size_t>(c.max_seqs) * c.n_kv_heads * 256));
    CREATE_CUDA(cudaMalloc(&ctx->select_tau, sizeof(float) * static_cast<size_t>(c.max_seqs) * c.n_kv_heads));
    if (ctx->split_n > 0) {
        CREATE_CUDA(cudaMalloc(&ctx->split_part, sizeof(float) * static_cast<size_t>(ctx->sm_count) * 4 * kTileM * kMaxHeads));
        CREATE_CUDA(cudaMalloc(&ctx->split_arrive, sizeof(uint32_t) * static_cast<size_t>(ctx->sm_count)));
        CREATE_CUDA(cudaMemset(ctx->split_arrive, 0, sizeof(uint32_t) * static_cast<size_t>(ctx->sm_count)));
        CREATE_CUDA(cudaMalloc(&ctx->wide_arrive, sizeof(uint32_t) * static_cast<size_t>(ctx->sm_count)));
        CREATE_CUDA(cudaMemset(ctx->wide_arrive, 0, sizeof(uint32_t) * static_cast<size_t>(ctx->sm_count)));
    }
    {
        // one-launch pruning: a grid never larger than what the device holds at once (its CTAs wait for one another)
        // No shared-memory carve-out is asked for: with the largest one (which the compaction that runs beside
        // a scoring kernel needs) the L1 that is left holds too few lines in flight, and this kernel alone moved
        // rows at 2.4 TB/s instead of 4.9.
        CREATE_CUDA(cudaFuncSetAttribute(prune_onepass_kernel<kOpRows>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kOpDynSmem)));
        int per_sm = 0;
        CREATE_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, prune_onepass_kernel<kOpRows>, kOpThreads, kOpDynSmem));
        if (per_sm < 1) per_sm = 1;
        // half of what fits: the next call's kernel then finds room beside this one
        ctx->op_capacity = per_sm * ctx->sm_count / 2;
        if (ctx->op_capacity < 1) ctx->op_capacity = 1;
        const size_t cap = static_cast<size_t>(ctx->op_capacity);
        CREATE_CUDA(cudaMalloc(&ctx->op_mask, sizeof(uint32_t) * kOpRing * ctx->max_words * c.n_kv_heads));
        CREATE_CUDA(cudaMalloc(&ctx->op_counts, sizeof(uint64_t) * kOpRing * cap * kMaxHeads));
        CREATE_CUDA(cudaMemset(ctx->op_counts, 0, sizeof(uint64_t) * kOpRing * cap * kMaxHeads));
        CREATE_CUDA(cudaMalloc(&ctx->op_len_acc, sizeof(int32_t) * kOpRing * static_cast<size_t>(c.max_seqs) * c.n_kv_heads));
        CREATE_CUDA(cudaMemset(ctx->op_len_acc, 0, sizeof(int32_t) * kOpRing * static_cast<size_t>(c.max_seqs) * c.n_kv_heads));
        CREATE_CUDA(cudaMalloc(&ctx->op_arrive, sizeof(uint32_t) * kOpRing));
        CREATE_CUDA(cudaMemset(ctx->op_arrive, 0, sizeof(uint32_t) * kOpRing));
        CREATE_CUDA(cudaMalloc(&ctx->op_scan_flag, sizeof(int32_t) * kOpRing));
        CREATE_CUDA(cudaMemset(ctx->op_scan_flag, 0, sizeof(int32_t) * kOpRing));
        CREATE_CUDA(cudaMalloc(&ctx->op_page0, sizeof(int32_t) * kOpRing * static_cast<size_t>(c.max_seqs) * c.n_kv_heads));
        CREATE_CUDA(cudaMalloc(&ctx->lin_counts, sizeof(uint64_t) * kOpRing * kLinMaxTiles * kMaxHeads));
        CREATE_CUDA(cudaMemset(ctx->lin_counts, 0, sizeof(uint64_t) * kOpRing * kLinMaxTiles * kMaxHeads));
    }
    CREATE_CUDA(cudaMalloc(&ctx->status_dev, sizeof(int32_t)));
    CREATE_CUDA(cudaMemset(ctx->status_dev, 0, sizeof(int32_t)));
    CREATE_CUDA(cudaMallocHost(&ctx->status_host, sizeof(int32_t)));
    CREATE_CUDA(cudaDeviceSynchronize());
#undef CREATE_CUDA
    g_create_error[0] = 0;
    *out = ctx;
    return KVZAP_OK;
}

kvzap_status kvzap_destroy(kvzap_ctx *ctx)
{
    if (!ctx) return KVZAP_OK;
    DeviceGuard guard(ctx->cfg.device);
    cudaDeviceSynchronize();
    free_all(ctx);
    delete ctx;
    return KVZAP_OK;
}

const char *kvzap_last_error(const kvzap_ctx *ctx) { return ctx ? ctx->err : g_create_error; }

int64_t kvzap_launch_count(const kvzap_ctx *ctx) { return ctx ? ctx->launches : 0; }

kvzap_status kvzap_set_weights(kvzap_ctx *ctx, int32_t layer, const void *W1, const float *b1, const void *W2,
                               const float *b2, void *stream_)
{
    NvtxRange nvtx_range("kvzap_set_weights");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const kvzap_config &c = ctx->cfg;
    if (layer < 0 || layer >= c.n_layers) return fail(ctx, KVZAP_ERR_INVALID_ARG, "layer %d out of range", layer);
    if (!W1) return fail(ctx, KVZAP_ERR_INVALID_ARG, "W1 is NULL");
    if (c.hidden == 0 && (W2 || b2)) return fail(ctx, KVZAP_ERR_INVALID_ARG, "KVzap-Linear takes no W2/b2");
    if (c.hidden > 0 && !W2) return fail(ctx, KVZAP_ERR_INVALID_ARG, "KVzap-MLP needs W2");
    DeviceGuard guard(c.device);
    const int rows = c.hidden > 0 ? c.hidden : c.n_kv_heads;
    if (!aligned16(W1)) return fail(ctx, KVZAP_ERR_INVALID_ARG, "W1 must be 16-byte aligned");
    float *b1_dst = ctx->b1_all + static_cast<size_t>(layer) * ctx->w1_rows;
    {
        const int64_t units = static_cast<int64_t>(rows) * (c.d_model / 8);
        pack_w1_kernel<<<static_cast<unsigned>((units + 255) / 256), 256, 0, stream>>>(
            static_cast<const uint4 *>(W1), rows, c.d_model, static_cast<int64_t>(c.n_layers) * ctx->w1_rows,
            static_cast<int64_t>(layer) * ctx->w1_rows, static_cast<uint4 *>(ctx->w1_all));
        KVZAP_CUDA(ctx, cudaGetLastError());
        ctx->launches += 1;
    }
    if (b1)
        KVZAP_CUDA(ctx, cudaMemcpyAsync(b1_dst, b1, sizeof(float) * rows, cudaMemcpyDeviceToDevice, stream));
    else
        KVZAP_CUDA(ctx, cudaMemsetAsync(b1_dst, 0, sizeof(float) * rows, stream));
    if (c.hidden > 0) {
        const int n = c.hidden * kMaxHeads;
        pack_w2_kernel<<<(n + 255) / 256, 256, 0, stream>>>(static_cast<const uint16_t *>(W2), b2, c.n_kv_heads,
                                                            c.hidden,
                                                            ctx->w2t_all + static_cast<size_t>(layer) * n,
                                                            ctx->b2_all + static_cast<size_t>(layer) * kMaxHeads);
        KVZAP_CUDA(ctx, cudaGetLastError());
        ctx->launches += 1;
    }
    ctx->layer_set[layer] = 1;
    ctx->layer_fp8[layer] = 0;
    return KVZAP_OK;
}

kvzap_status kvzap_set_weights_fp8(kvzap_ctx *ctx, int32_t layer, const void *W1_e4m3, const float *w1_scale, const float *b1,
                                   const void *W2, const float *b2, void *stream_)
{
    NvtxRange nvtx_range("kvzap_set_weights_fp8");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    serial_point(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const kvzap_config &c = ctx->cfg;
    if (layer < 0 || layer >= c.n_layers) return fail(ctx, KVZAP_ERR_INVALID_ARG, "layer %d out of range", layer);
    if (c.d_model % 128) return fail(ctx, KVZAP_ERR_UNSUPPORTED, "8-bit inputs need d_model to be a multiple of 128 (is %d)", c.d_model);
    if (!W1_e4m3 || !aligned16(W1_e4m3)) return fail(ctx, KVZAP_ERR_INVALID_ARG, "W1 must be non-NULL and 16-byte aligned");
    if (c.hidden == 0 && (W2 || b2)) return fail(ctx, KVZAP_ERR_INVALID_ARG, "KVzap-Linear takes no W2/b2");
    if (c.hidden > 0 && !W2) return fail(ctx, KVZAP_ERR_INVALID_ARG, "KVzap-MLP needs W2");
    DeviceGuard guard(c.device);
    const int rows = c.hidden > 0 ? c.hidden : c.n_kv_heads;
    const int64_t rows_total = static_cast<int64_t>(c.n_layers) * ctx->w1_rows;
    if (!ctx->w1_fp8_all) {
        const size_t bytes = static_cast<size_t>(rows_total) * c.d_model;
        KVZAP_CUDA(ctx, cudaMalloc(&ctx->w1_fp8_all, bytes));
        KVZAP_CUDA(ctx, cudaMemsetAsync(ctx->w1_fp8_all, 0, bytes, stream));
        KVZAP_CUDA(ctx, cudaMalloc(&ctx->w1_scale_all, sizeof(float) * rows_total));
        for (int mode = 0; mode < (c.hidden > 0 ? 2 : 1); ++mode) {
            kvzap_status st = make_tmap8(ctx, &ctx->tmap_w8[mode], ctx->w1_fp8_all, static_cast<uint64_t>(rows_total),
                                         static_cast<uint64_t>(c.d_model), static_cast<uint32_t>(ctx->sched[mode].chunk_n / (mode + 1)), 0, true);
            if (st != KVZAP_OK) return st;
        }
        if (c.hidden > 0 && ctx->split_n > 0 && (c.d_model / 128) % ctx->split_k == 0) {
            // the few-token layout (a decode step): the same slices of hidden units, K blocks of 128 codes
            if (make_tmap8(ctx, &ctx->split_tmap_w8, ctx->w1_fp8_all, static_cast<uint64_t>(rows_total), static_cast<uint64_t>(c.d_model),
                           static_cast<uint32_t>(c.hidden / ctx->split_n), 0, true) == KVZAP_OK &&
                cudaFuncSetAttribute(score_split_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     static_cast<int>(ctx->split_smem)) == cudaSuccess &&
                cudaFuncSetAttribute(score_split_kernel<true>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     static_cast<int>(cudaSharedmemCarveoutMaxShared)) == cudaSuccess)
                ctx->split8_ok = true;
        }
        if (c.hidden > 0) {
            KVZAP_CUDA(ctx, cudaFuncSetAttribute(score_kernel<true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(ctx->sched[0].smem)));
            KVZAP_CUDA(ctx, cudaFuncSetAttribute(score_kernel<true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(ctx->sched[1].smem)));
            KVZAP_CUDA(ctx, cudaFuncSetAttribute(score_kernel<true, false, true>, cudaFuncAttributePreferredSharedMemoryCarveout, static_cast<int>(cudaSharedmemCarveoutMaxShared)));
            KVZAP_CUDA(ctx, cudaFuncSetAttribute(score_kernel<true, true, true>, cudaFuncAttributePreferredSharedMemoryCarveout, static_cast<int>(cudaSharedmemCarveoutMaxShared)));
        } else {
            KVZAP_CUDA(ctx, cudaFuncSetAttribute(score_kernel<false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(ctx->sched[0].smem)));
            KVZAP_CUDA(ctx, cudaFuncSetAttribute(score_kernel<false, false, true>, cudaFuncAttributePreferredSharedMemoryCarveout, static_cast<int>(cudaSharedmemCarveoutMaxShared)));
        }
    }
    {
        const int64_t units = static_cast<int64_t>(rows) * (c.d_model / 16);
        pack_w1_fp8_kernel<<<static_cast<unsigned>((units + 255) / 256), 256, 0, stream>>>(
            static_cast<const uint4 *>(W1_e4m3), rows, c.d_model, rows_total, static_cast<int64_t>(layer) * ctx->w1_rows,
            static_cast<uint4 *>(ctx->w1_fp8_all));
        fill_scale_kernel<<<(ctx->w1_rows + 255) / 256, 256, 0, stream>>>(w1_scale, rows, ctx->w1_rows,
                                                                         ctx->w1_scale_all + static_cast<size_t>(layer) * ctx->w1_rows);
        KVZAP_CUDA(ctx, cudaGetLastError());
        ctx->launches += 2;
    }
    float *b1_dst = ctx->b1_all + static_cast<size_t>(layer) * ctx->w1_rows;
    if (b1)
        KVZAP_CUDA(ctx, cudaMemcpyAsync(b1_dst, b1, sizeof(float) * rows, cudaMemcpyDeviceToDevice, stream));
    else
        KVZAP_CUDA(ctx, cudaMemsetAsync(b1_dst, 0, sizeof(float) * rows, stream));
    if (c.hidden > 0) {
        const int n = c.hidden * kMaxHeads;
        pack_w2_kernel<<<(n + 255) / 256, 256, 0, stream>>>(static_cast<const uint16_t *>(W2), b2, c.n_kv_heads, c.hidden,
                                                            ctx->w2t_all + static_cast<size_t>(layer) * n,
                                                            ctx->b2_all + static_cast<size_t>(layer) * kMaxHeads);
        KVZAP_CUDA(ctx, cudaGetLastError());
        ctx->launches += 1;
    }
    ctx->layer_set[layer] = 0;       // the bf16 entry points refuse this layer from now on
    ctx->layer_fp8[layer] = 1;
    return KVZAP_OK;
}

kvzap_status kvzap_score_fp8(kvzap_ctx *ctx, int32_t layer, const void *hidden_e4m3, const float *x_scale, int64_t n_tokens,
                             float *scores, void *stream_)
{
    NvtxRange nvtx_range("kvzap_score_fp8");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, KVZAP_ERR_INVALID_ARG, "layer %d out of range", layer);
    kvzap_status st = check_common(ctx, n_tokens, 1, nullptr);
    if (st != KVZAP_OK) return st;
    if (!ctx->layer_fp8[layer])
        return fail(ctx, KVZAP_ERR_STATE, "layer %d has no 8-bit weights (kvzap_set_weights_fp8)", layer);
    if (n_tokens == 0) return KVZAP_OK;
    if (!hidden_e4m3 || !scores || !aligned16(hidden_e4m3)) return fail(ctx, KVZAP_ERR_INVALID_ARG, "hidden (16-byte aligned) and scores must not be NULL");
    DeviceGuard guard(ctx->cfg.device);
    return launch_score_fp8(ctx, layer, hidden_e4m3, x_scale, n_tokens, scores, nullptr, nullptr, 1, 0.0f, 0, static_cast<cudaStream_t>(stream_));
}

kvzap_status kvzap_prefill_fused_fp8(kvzap_ctx *ctx, int32_t layer, const void *hidden_e4m3, const float *x_scale, const void *K,
                                     const void *V, const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens, float tau,
                                     int32_t w, void *K_out, void *V_out, int32_t *lengths, float *scores_out, void *stream_)
{
    NvtxRange nvtx_range("kvzap_prefill_fused_fp8");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, KVZAP_ERR_INVALID_ARG, "layer %d out of range", layer);
    kvzap_status st = check_common(ctx, n_tokens, n_seqs, cu_seqlens);
    if (st != KVZAP_OK) return st;
    if (!ctx->layer_fp8[layer])
        return fail(ctx, KVZAP_ERR_STATE, "layer %d has no 8-bit weights (kvzap_set_weights_fp8)", layer);
    if (!lengths) return fail(ctx, KVZAP_ERR_INVALID_ARG, "lengths is NULL");
    if (w < 0) return fail(ctx, KVZAP_ERR_INVALID_ARG, "window w is negative");
    DeviceGuard guard(ctx->cfg.device);
    if (n_tokens == 0) {
        KVZAP_CUDA(ctx, cudaMemsetAsync(lengths, 0, sizeof(int32_t) * n_seqs * ctx->cfg.n_kv_heads, stream));
        return KVZAP_OK;
    }
    st = check_prune_args(ctx, K, V, K_out, V_out, lengths, w);
    if (st != KVZAP_OK) return st;
    if (!hidden_e4m3 || !aligned16(hidden_e4m3)) return fail(ctx, KVZAP_ERR_INVALID_ARG, "hidden must be non-NULL, 16-byte aligned");
    uint32_t *mask = next_mask_slice(ctx);
    st = launch_score_fp8(ctx, layer, hidden_e4m3, x_scale, n_tokens, scores_out, mask, cu_seqlens, n_seqs, tau, w, stream);
    if (st != KVZAP_OK) return st;
    return launch_compaction(ctx, mask, K, V, cu_seqlens, n_seqs, n_tokens, K_out, V_out, lengths, stream, true, false);
}

kvzap_status kvzap_score(kvzap_ctx *ctx, int32_t layer, const void *hidden, int64_t n_tokens, float *scores,
                         void *stream_)
{
    NvtxRange nvtx_range("kvzap_score");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, KVZAP_ERR_INVALID_ARG, "layer %d out of range", layer);
    kvzap_status st = check_common(ctx, n_tokens, 1, nullptr);
    if (st != KVZAP_OK) return st;
    if (!ctx->layer_set[layer]) return fail(ctx, KVZAP_ERR_STATE, "layer %d has no weights", layer);
    if (n_tokens == 0) return KVZAP_OK;
    if (!hidden || !scores) return fail(ctx, KVZAP_ERR_INVALID_ARG, "hidden and scores must not be NULL");
    if (!aligned16(hidden)) return fail(ctx, KVZAP_ERR_INVALID_ARG, "hidden must be 16-byte aligned");
    DeviceGuard guard(ctx->cfg.device);
    return launch_score(ctx, layer, 1, hidden, n_tokens, scores, nullptr, nullptr, 1, 0.0f, 0,
                        static_cast<cudaStream_t>(stream_));
}

kvzap_status kvzap_prune_prefill(kvzap_ctx *ctx, const void *K, const void *V, const float *scores,
                                 const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens, float tau, int32_t w,
                                 void *K_out, void *V_out, int32_t *lengths, void *stream_)
{
    NvtxRange nvtx_range("kvzap_prune_prefill");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    kvzap_status st = check_common(ctx, n_tokens, n_seqs, cu_seqlens);
    if (st != KVZAP_OK) return st;
    if (!lengths) return fail(ctx, KVZAP_ERR_INVALID_ARG, "lengths is NULL");
    if (w < 0) return fail(ctx, KVZAP_ERR_INVALID_ARG, "window w is negative");
    DeviceGuard guard(ctx->cfg.device);
    if (n_tokens == 0) {
        KVZAP_CUDA(ctx, cudaMemsetAsync(lengths, 0, sizeof(int32_t) * n_seqs * ctx->cfg.n_kv_heads, stream));
        return KVZAP_OK;
    }
    st = check_prune_args(ctx, K, V, K_out, V_out, lengths, w);
    if (st != KVZAP_OK) return st;
    if (!scores) return fail(ctx, KVZAP_ERR_INVALID_ARG, "scores is NULL");
    return launch_prune_onepass(ctx, scores, nullptr, tau, w, K, V, cu_seqlens, n_seqs, n_tokens, K_out, V_out, lengths, 0, 0,
                                0, 0, nullptr, nullptr, stream);
}

kvzap_status kvzap_prune_prefill_topk(kvzap_ctx *ctx, const void *K, const void *V, const float *scores,
                                      const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens, float keep_ratio,
                                      int32_t w, int32_t per_layer, void *K_out, void *V_out, int32_t *lengths,
                                      float *tau_out, void *stream_)
{
    NvtxRange nvtx_range("kvzap_prune_prefill_topk");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    kvzap_status st = check_common(ctx, n_tokens, n_seqs, cu_seqlens);
    if (st != KVZAP_OK) return st;
    if (!lengths) return fail(ctx, KVZAP_ERR_INVALID_ARG, "lengths is NULL");
    if (w < 0) return fail(ctx, KVZAP_ERR_INVALID_ARG, "window w is negative");
    if (!(keep_ratio >= 0.0f && keep_ratio <= 1.0f)) return fail(ctx, KVZAP_ERR_INVALID_ARG, "keep_ratio outside [0, 1]");
    const kvzap_config &c = ctx->cfg;
    DeviceGuard guard(c.device);
    float *tau_list = tau_out ? tau_out : ctx->select_tau;
    if (n_tokens == 0) {
        KVZAP_CUDA(ctx, cudaMemsetAsync(lengths, 0, sizeof(int32_t) * n_seqs * c.n_kv_heads, stream));
        return KVZAP_OK;
    }
    st = check_prune_args(ctx, K, V, K_out, V_out, lengths, w);
    if (st != KVZAP_OK) return st;
    if (!scores) return fail(ctx, KVZAP_ERR_INVALID_ARG, "scores is NULL");
    const int n_sel = per_layer ? 1 : c.n_kv_heads;
    KVZAP_CUDA(ctx, cudaMemsetAsync(ctx->select_hist, 0, sizeof(uint32_t) * 4 * static_cast<size_t>(n_seqs) * n_sel * 256, stream));
    const dim3 grid(static_cast<unsigned>((n_tokens + kSelectThreads - 1) / kSelectThreads), static_cast<unsigned>(n_seqs));
    const bool early = !ctx->profiling;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attrs[2];
    for (int pass = 0; pass < 4; ++pass) {
        make_launch(&cfg, attrs, grid, dim3(kSelectThreads), 0, stream, early, 1);
        KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, select_hist_kernel, scores, n_tokens, static_cast<int>(c.n_kv_heads), cu_seqlens,
                                           static_cast<int>(n_seqs), static_cast<int>(w), keep_ratio, per_layer ? 1 : 0, pass,
                                           ctx->select_hist));
    }
    make_launch(&cfg, attrs, dim3(static_cast<unsigned>(n_seqs)), dim3(kSelectThreads), 0, stream, early, 1);
    KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, select_finish_kernel, n_tokens, static_cast<int>(c.n_kv_heads), cu_seqlens,
                                       static_cast<int>(n_seqs), static_cast<int>(w), keep_ratio, per_layer ? 1 : 0,
                                       static_cast<const uint32_t *>(ctx->select_hist), tau_list, ctx->status_dev));
    KVZAP_CUDA(ctx, cudaGetLastError());
    ctx->launches += 5;
    // the same mask + compaction launch as kvzap_prune_prefill, with the cut values as per-list thresholds
    return launch_prune_onepass(ctx, scores, tau_list, 0.0f, w, K, V, cu_seqlens, n_seqs, n_tokens, K_out, V_out, lengths, 0,
                                0, 0, 0, nullptr, nullptr, stream);
}

// tok_major: K and V are [n_tokens][H][D] (the K/V projection's output) instead of [H][n_tokens][D]
static kvzap_status prefill_fused_impl(kvzap_ctx *ctx, int32_t layer, const void *hidden, const void *K, const void *V,
                                       const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens, float tau,
                                       int32_t w, void *K_out, void *V_out, int32_t *lengths, float *scores_out,
                                       void *stream_, bool tok_major)
{
    NvtxRange nvtx_range("kvzap_prefill_fused / kvzap_prefill_write");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, KVZAP_ERR_INVALID_ARG, "layer %d out of range", layer);
    kvzap_status st = check_common(ctx, n_tokens, n_seqs, cu_seqlens);
    if (st != KVZAP_OK) return st;
    if (!ctx->layer_set[layer]) return fail(ctx, KVZAP_ERR_STATE, "layer %d has no weights", layer);
    if (!lengths) return fail(ctx, KVZAP_ERR_INVALID_ARG, "lengths is NULL");
    if (w < 0) return fail(ctx, KVZAP_ERR_INVALID_ARG, "window w is negative");
    DeviceGuard guard(ctx->cfg.device);
    if (n_tokens == 0) {
        KVZAP_CUDA(ctx, cudaMemsetAsync(lengths, 0, sizeof(int32_t) * n_seqs * ctx->cfg.n_kv_heads, stream));
        return KVZAP_OK;
    }
    st = check_prune_args(ctx, K, V, K_out, V_out, lengths, w);
    if (st != KVZAP_OK) return st;
    if (!hidden || !aligned16(hidden)) return fail(ctx, KVZAP_ERR_INVALID_ARG, "hidden must be non-NULL, 16-byte aligned");
    uint32_t *mask = next_mask_slice(ctx);
    const CompactArgs compact{K, V, K_out, V_out, lengths, tok_major};
    bool compacted = false;
    st = launch_score(ctx, layer, 1, hidden, n_tokens, scores_out, mask, cu_seqlens, n_seqs, tau, w, stream, 1, nullptr, nullptr,
                      false, &compact, &compacted);
    if (st != KVZAP_OK || compacted) return st;
    return launch_compaction(ctx, mask, K, V, cu_seqlens, n_seqs, n_tokens, K_out, V_out, lengths, stream, true, tok_major);
}

kvzap_status kvzap_prefill_fused(kvzap_ctx *ctx, int32_t layer, const void *hidden, const void *K, const void *V,
                                 const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens, float tau, int32_t w,
                                 void *K_out, void *V_out, int32_t *lengths, float *scores_out, void *stream_)
{
    return prefill_fused_impl(ctx, layer, hidden, K, V, cu_seqlens, n_seqs, n_tokens, tau, w, K_out, V_out, lengths,
                              scores_out, stream_, false);
}

kvzap_status kvzap_prefill_write(kvzap_ctx *ctx, int32_t layer, const void *hidden, const void *K_proj,
                                 const void *V_proj, const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                 float tau, int32_t w, void *K_out, void *V_out, int32_t *lengths, float *scores_out,
                                 void *stream_)
{
    return prefill_fused_impl(ctx, layer, hidden, K_proj, V_proj, cu_seqlens, n_seqs, n_tokens, tau, w, K_out, V_out,
                              lengths, scores_out, stream_, true);
}

kvzap_status kvzap_prefill_plan(kvzap_ctx *ctx, int32_t layer, const void *hidden, const int32_t *cu_seqlens, int32_t n_seqs,
                                int64_t n_tokens, float tau, int32_t w, int32_t *slot, int32_t *lengths, float *scores_out,
                                int32_t page_tokens, int64_t n_pages_pool, int32_t first_page, int32_t *page_table,
                                int32_t max_pages_per_list, int32_t *n_pages_used, void *stream_)
{
    NvtxRange nvtx_range("kvzap_prefill_plan");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const kvzap_config &c = ctx->cfg;
    if (layer < 0 || layer >= c.n_layers) return fail(ctx, KVZAP_ERR_INVALID_ARG, "layer %d out of range", layer);
    kvzap_status st = check_common(ctx, n_tokens, n_seqs, cu_seqlens);
    if (st != KVZAP_OK) return st;
    if (!ctx->layer_set[layer]) return fail(ctx, KVZAP_ERR_STATE, "layer %d has no weights", layer);
    if (!lengths || w < 0) return fail(ctx, KVZAP_ERR_INVALID_ARG, "plan: lengths is NULL or w negative");
    const bool paged = page_tokens > 0;
    if (page_tokens < 0 || (paged && (!page_table || !n_pages_used || max_pages_per_list < 1 || n_pages_pool < 0 || first_page < 0)))
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "plan: paged output needs page_table, n_pages_used, max_pages_per_list >= 1, first_page >= 0");
    DeviceGuard guard(c.device);
    if (n_tokens == 0) {
        KVZAP_CUDA(ctx, cudaMemsetAsync(lengths, 0, sizeof(int32_t) * n_seqs * c.n_kv_heads, stream));
        if (paged) KVZAP_CUDA(ctx, cudaMemsetAsync(n_pages_used, 0, sizeof(int32_t), stream));
        return KVZAP_OK;
    }
    if (!hidden || !aligned16(hidden) || !slot) return fail(ctx, KVZAP_ERR_INVALID_ARG, "plan: hidden (16-byte aligned) and slot must not be NULL");
    float *scores = scores_out;
    if (!scores) {
        if (!ctx->plan_scores) KVZAP_CUDA(ctx, cudaMalloc(&ctx->plan_scores, sizeof(float) * static_cast<size_t>(c.max_tokens) * c.n_kv_heads));
        scores = ctx->plan_scores;
    }
    st = launch_score(ctx, layer, 1, hidden, n_tokens, scores, nullptr, nullptr, 1, 0.0f, 0, stream);
    if (st != KVZAP_OK) return st;
    return launch_prune_onepass(ctx, scores, nullptr, tau, w, nullptr, nullptr, cu_seqlens, n_seqs, n_tokens, nullptr, nullptr, lengths,
                                page_tokens, first_page, n_pages_pool, max_pages_per_list, page_table, n_pages_used, stream, slot, true);
}

kvzap_status kvzap_poll_status(kvzap_ctx *ctx, void *stream_)
{
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    DeviceGuard guard(ctx->cfg.device);
    KVZAP_CUDA(ctx, cudaMemcpyAsync(ctx->status_host, ctx->status_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    KVZAP_CUDA(ctx, cudaMemsetAsync(ctx->status_dev, 0, sizeof(int32_t), stream));
    KVZAP_CUDA(ctx, cudaStreamSynchronize(stream));
    const int32_t v = *ctx->status_host;
    if (v == 0) return KVZAP_OK;
    // a scoring kernel that gave up may have left its work-tile counter in an unknown state
    cudaMemsetAsync(ctx->tile_counters, 0, sizeof(int32_t) * kMaskRing, stream);
    if (ctx->split_arrive) cudaMemsetAsync(ctx->split_arrive, 0, sizeof(uint32_t) * static_cast<size_t>(ctx->sm_count), stream);
    if (ctx->wide_arrive) cudaMemsetAsync(ctx->wide_arrive, 0, sizeof(uint32_t) * static_cast<size_t>(ctx->sm_count), stream);
    if (v == KVZAP_ERR_TIMEOUT) {
        reset_step_counters(ctx, stream);
        // a one-launch pruning call that gave up may have left its list-length sums and arrival count behind
        cudaMemsetAsync(ctx->op_len_acc, 0, sizeof(int32_t) * kOpRing * static_cast<size_t>(ctx->cfg.max_seqs) * ctx->cfg.n_kv_heads, stream);
        cudaMemsetAsync(ctx->op_arrive, 0, sizeof(uint32_t) * kOpRing, stream);
    }
    cudaStreamSynchronize(stream);
    fail(ctx, static_cast<kvzap_status>(v), "device-side condition %d recorded", v);
    return static_cast<kvzap_status>(v);
}

kvzap_status kvzap_set_wait_limit(kvzap_ctx *ctx, int64_t cycles)
{
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    if (cycles < 1000) return fail(ctx, KVZAP_ERR_INVALID_ARG, "wait limit %lld: need at least 1000 cycles", static_cast<long long>(cycles));
    ctx->wait_limit = cycles;
    return KVZAP_OK;
}

kvzap_status kvzap_set_profiling(kvzap_ctx *ctx, int32_t enable)
{
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    for (auto &r : ctx->prof) { cudaEventDestroy(r.start); cudaEventDestroy(r.stop); }
    ctx->prof.clear();
    ctx->profiling = enable != 0;
    return KVZAP_OK;
}

kvzap_status kvzap_get_profile(kvzap_ctx *ctx, int32_t kernel, double *total_ms, int64_t *n_launches)
{
    if (!ctx || !total_ms || !n_launches) return KVZAP_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    KVZAP_CUDA(ctx, cudaDeviceSynchronize());
    double sum = 0.0;
    int64_t n = 0;
    for (auto &r : ctx->prof) {
        if (r.kind != kernel) continue;
        float ms = 0.0f;
        KVZAP_CUDA(ctx, cudaEventElapsedTime(&ms, r.start, r.stop));
        sum += ms;
        ++n;
    }
    *total_ms = sum;
    *n_launches = n;
    return KVZAP_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------
// Allocation-free variant of kvzap_prune_prefill.
//
// Its scratch (mask words, block prefix sums, per-sequence bases, a status word)
// lives in the file-scope device array below instead of a context's cudaMalloc'd
// buffers, so that a caller who must not allocate can still prune.  Every GPU that
// loads this library carries the array (about 170 KB) until the process exits.
namespace kvzap {

constexpr int64_t kNoAllocMaxTokens = KVZAP_NOALLOC_MAX_TOKENS;
constexpr int kNoAllocMaxSeqs = KVZAP_NOALLOC_MAX_SEQS;
constexpr int64_t kNoAllocMaxBlocks = (kNoAllocMaxTokens + kBlockTokens - 1) / kBlockTokens;
constexpr size_t round256(size_t v) { return (v + 255) / 256 * 256; }
constexpr size_t kNoAllocMaskOff = 0;
constexpr size_t kNoAllocMaskBytes = round256(sizeof(uint32_t) * kMaxHeads * kNoAllocMaxBlocks * 4);
constexpr size_t kNoAllocPrefixOff = kNoAllocMaskOff + kNoAllocMaskBytes;
constexpr size_t kNoAllocPrefixBytes = round256(sizeof(int32_t) * kMaxHeads * (kNoAllocMaxBlocks + 1));
constexpr size_t kNoAllocSeqOff = kNoAllocPrefixOff + kNoAllocPrefixBytes;
constexpr size_t kNoAllocSeqBytes = round256(sizeof(int32_t) * kMaxHeads * (kNoAllocMaxSeqs + 1));
constexpr size_t kNoAllocStatusOff = kNoAllocSeqOff + kNoAllocSeqBytes;
constexpr size_t kNoAllocBytes = kNoAllocStatusOff + 256;

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

constexpr int kNoAllocMaxDevices = 64;
static void *g_noalloc_dev_ptr[kNoAllocMaxDevices];      // device address of the array, per device ordinal

}  // namespace kvzap

extern "C" kvzap_status kvzap_prune_prefill_noalloc(const void *K, const void *V, const float *scores,
                                                    const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                                    int32_t n_kv_heads, int32_t head_dim, float tau, int32_t w,
                                                    void *K_out, void *V_out, int32_t *lengths, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (n_kv_heads < 1 || n_kv_heads > kMaxHeads)
        return fail(nullptr, KVZAP_ERR_UNSUPPORTED, "noalloc: n_kv_heads %d: need 1..8", n_kv_heads);
    if (head_dim < 8 || head_dim > 1024 || head_dim % 8)
        return fail(nullptr, KVZAP_ERR_UNSUPPORTED, "noalloc: head_dim %d: need a multiple of 8 in 8..1024", head_dim);
    if (n_tokens < 0) return fail(nullptr, KVZAP_ERR_INVALID_ARG, "noalloc: n_tokens is negative");
    if (n_tokens > kNoAllocMaxTokens)
        return fail(nullptr, KVZAP_ERR_UNSUPPORTED,
                    "noalloc: n_tokens %lld exceeds the static scratch's limit KVZAP_NOALLOC_MAX_TOKENS = %lld",
                    static_cast<long long>(n_tokens), static_cast<long long>(kNoAllocMaxTokens));
    if (n_seqs < 1 || n_seqs > kNoAllocMaxSeqs)
        return fail(nullptr, KVZAP_ERR_UNSUPPORTED,
                    "noalloc: n_seqs %d outside 1..KVZAP_NOALLOC_MAX_SEQS (%d)", n_seqs, kNoAllocMaxSeqs);
    if (cu_seqlens == nullptr && n_seqs != 1)
        return fail(nullptr, KVZAP_ERR_INVALID_ARG, "noalloc: cu_seqlens is NULL but n_seqs is %d", n_seqs);
    if (!lengths) return fail(nullptr, KVZAP_ERR_INVALID_ARG, "noalloc: lengths is NULL");
    if (w < 0) return fail(nullptr, KVZAP_ERR_INVALID_ARG, "noalloc: window w is negative");

    // once per device, with that device current: resolve the array's device address
    int dev = -1;
    KVZAP_CUDA(nullptr, cudaGetDevice(&dev));
    if (dev < 0 || dev >= kNoAllocMaxDevices)
        return fail(nullptr, KVZAP_ERR_UNSUPPORTED, "noalloc: device ordinal %d not supported", dev);
    void *base = g_noalloc_dev_ptr[dev];
    if (base == nullptr) {
        void *ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || ptr == nullptr)
            return fail(nullptr, KVZAP_ERR_CUDA, "noalloc: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
        g_noalloc_dev_ptr[dev] = ptr;
        base = ptr;
    }
    if (n_tokens == 0) {
        KVZAP_CUDA(nullptr, cudaMemsetAsync(lengths, 0, sizeof(int32_t) * n_seqs * n_kv_heads, stream));
        return KVZAP_OK;
    }
    if (!K || !V || !K_out || !V_out || !scores)
        return fail(nullptr, KVZAP_ERR_INVALID_ARG, "noalloc: K, V, scores, K_out and V_out must not be NULL");
    if (!aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out))
        return fail(nullptr, KVZAP_ERR_INVALID_ARG, "noalloc: K/V pointers must be 16-byte aligned");

    unsigned char *b8 = static_cast<unsigned char *>(base);
    uint32_t *maskbits = reinterpret_cast<uint32_t *>(b8 + kNoAllocMaskOff);
    int32_t *blockprefix = reinterpret_cast<int32_t *>(b8 + kNoAllocPrefixOff);
    int32_t *seqbase = reinterpret_cast<int32_t *>(b8 + kNoAllocSeqOff);
    int32_t *status = reinterpret_cast<int32_t *>(b8 + kNoAllocStatusOff);
    const int64_t n_blocks = (n_tokens + kBlockTokens - 1) / kBlockTokens;
    const int64_t n_words = n_blocks * 4;
    // The array keeps whatever the previous call left.  Every mask word, prefix and base entry
    // that this call reads is first written by it; only the status word must start at zero.
    KVZAP_CUDA(nullptr, cudaMemsetAsync(status, 0, sizeof(int32_t), stream));
    mask_kernel<<<static_cast<unsigned>(n_blocks), 128, 0, stream>>>(scores, n_tokens, n_kv_heads, cu_seqlens, n_seqs,
                                                                     tau, w, 1, maskbits, n_words, nullptr);
    KVZAP_CUDA(nullptr, cudaGetLastError());
    scan_kernel<<<1, 1024, 0, stream>>>(maskbits, n_words, n_blocks, n_kv_heads, cu_seqlens, n_seqs, n_tokens,
                                        blockprefix, seqbase, lengths, 0, 0, 0, 0, nullptr, nullptr, nullptr, nullptr, status, 0, nullptr, nullptr, nullptr,
                                        nullptr);
    KVZAP_CUDA(nullptr, cudaGetLastError());
    const dim3 grid(static_cast<unsigned>(n_blocks), static_cast<unsigned>(n_kv_heads));
    compact_kernel<false><<<grid, kCompactThreads, 0, stream>>>(
        static_cast<const uint4 *>(K), static_cast<const uint4 *>(V), static_cast<uint4 *>(K_out),
        static_cast<uint4 *>(V_out), maskbits, n_words, n_blocks, blockprefix, seqbase, cu_seqlens, n_seqs, n_tokens,
        n_kv_heads, head_dim / 8, 0, nullptr);
    KVZAP_CUDA(nullptr, cudaGetLastError());
    return KVZAP_OK;
}

// ---------------------------------------------------------------------------
// Paged output and the decode-time cache.
struct kvzap_cache {
    kvzap_ctx *ctx = nullptr;
    kvzap::CacheView v;
    float *scores = nullptr;        // [L][B][H] scratch when the caller does not want the scores
    int64_t n_lists = 0;
    int step_parity = 0;
    // fused decode steps: per-cluster count of completed steps on the device, and the host's view of it
    int32_t *done = nullptr;             // [n_layers * ceil(n_seqs / 128)][4]: one per cluster of the fused step
    int32_t *ticket = nullptr;           // behind `done`: [tiles][4][2] steps started per (slice, rank), see DecodeFuse
    size_t n_step_counters = 0;          // ints in done + ticket together
    // attention over the cache: tensor maps of the page pools and of the window rings (built on first use)
    CUtensorMap tm_kpool, tm_vpool, tm_kring, tm_vring;
    int attn_state = 0;                  // 0 not built yet, 1 ready, -1 this cache's geometry is not supported
    float *attn_scratch = nullptr;       // partial results of lists that are split over several CTAs
    uint32_t *attn_arrive = nullptr;     // [attn_split_lists] arrival counts, zero between launches
    int64_t attn_units = 0;              // capacity of attn_scratch in (list, part) units
};

namespace kvzap {

static void reset_step_counters(kvzap_ctx *ctx, cudaStream_t stream)
{
    for (kvzap_cache *cache : ctx->caches) {
        cudaMemsetAsync(cache->done, 0, sizeof(int32_t) * cache->n_step_counters, stream);
    }
    ctx->fused_cache = nullptr;
}

static kvzap_status launch_compaction_paged(kvzap_ctx *ctx, const uint32_t *mask, const void *K, const void *V,
                                            const int32_t *cu_seqlens,
                                            int32_t n_seqs, int64_t n_tokens, void *K_pool, void *V_pool,
                                            int64_t n_pages_pool, int32_t page_tokens, int32_t first_page,
                                            int32_t *page_table, int32_t max_pages, int32_t *lengths,
                                            int32_t *n_pages_used, cudaStream_t stream,
                                            int32_t *page_cursor = nullptr, bool tok_major = false, bool append = false,
                                            bool beside_scoring = true, const int32_t *free_stack = nullptr,
                                            int32_t *free_top = nullptr, const int64_t *list_map = nullptr)
{
    const kvzap_config &c = ctx->cfg;
    const int64_t n_blocks = (n_tokens + kBlockTokens - 1) / kBlockTokens;
    const int64_t n_words = n_blocks * 4;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attrs[2];
    {
        // lengths and the first page of every list (the only step that needs all lists at once)
        ProfScope prof(ctx, KVZAP_KERNEL_SCAN, stream);
        make_launch(&cfg, attrs, dim3(1), dim3(1024), 0, stream, !ctx->profiling, 1);
        KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, scan_kernel, mask, n_words, n_blocks, static_cast<int>(c.n_kv_heads),
                                           cu_seqlens, static_cast<int>(n_seqs), n_tokens, static_cast<int32_t *>(nullptr),
                                           static_cast<int32_t *>(nullptr),
                                           lengths, static_cast<int>(page_tokens), first_page, n_pages_pool,
                                           static_cast<int>(max_pages), ctx->list_page0, page_table, n_pages_used,
                                           page_cursor, ctx->status_dev, append ? 1 : 0, ctx->list_base, free_stack, free_top, list_map));
    }
    // the same resident-at-once grid as the dense-ragged output (see launch_compaction)
    const int64_t max_ctas = static_cast<int64_t>(ctx->sm_count) * (!beside_scoring ? 8 : (c.hidden > 0 ? 2 : 6));
    int64_t chunks = max_ctas / c.n_kv_heads;
    if (chunks < 1) chunks = 1;
    if (chunks > n_blocks) chunks = n_blocks;
    const int blocks_per_cta = static_cast<int>((n_blocks + chunks - 1) / chunks);
    chunks = (n_blocks + blocks_per_cta - 1) / blocks_per_cta;
    {
        ProfScope prof(ctx, KVZAP_KERNEL_COMPACT, stream);
        make_launch(&cfg, attrs, dim3(static_cast<unsigned>(chunks), static_cast<unsigned>(c.n_kv_heads)),
                    dim3(kDenseThreads), 0, stream, !ctx->profiling, 1);
        KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, compact_dense_kernel<kDenseThreads>, static_cast<const uint4 *>(K),
                                           static_cast<const uint4 *>(V), static_cast<uint4 *>(K_pool),
                                           static_cast<uint4 *>(V_pool), mask, n_words, n_blocks, blocks_per_cta,
                                           cu_seqlens, static_cast<int>(n_seqs), n_tokens, static_cast<int>(c.n_kv_heads),
                                           static_cast<int>(c.head_dim / 8), lengths, static_cast<int>(page_tokens),
                                           static_cast<const int32_t *>(ctx->list_page0),
                                           tok_major ? int64_t{1} : n_tokens,
                                           tok_major ? static_cast<int64_t>(c.n_kv_heads) : int64_t{1},
                                           static_cast<const int32_t *>(append ? ctx->list_base : nullptr),
                                           static_cast<const int32_t *>(page_table), static_cast<int>(max_pages), list_map));
    }
    ctx->launches += 2;
    return KVZAP_OK;
}

static kvzap_status check_paged_args(kvzap_ctx *ctx, const void *K, const void *V, const void *K_pool,
                                     const void *V_pool, int64_t n_pages_pool, int32_t page_tokens, int32_t first_page,
                                     const int32_t *page_table, int32_t max_pages, const int32_t *lengths,
                                     const int32_t *n_pages_used, int32_t w)
{
    if (!K || !V || !K_pool || !V_pool || !page_table || !lengths || !n_pages_used)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "paged: K, V, pools, page_table, lengths, n_pages_used must not be NULL");
    if (!aligned16(K) || !aligned16(V) || !aligned16(K_pool) || !aligned16(V_pool))
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "paged: K/V and pool pointers must be 16-byte aligned");
    if (page_tokens < 1 || max_pages < 1 || n_pages_pool < 0 || first_page < 0)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "paged: page_tokens, max_pages_per_list >= 1; n_pages_pool, first_page >= 0");
    if (w < 0) return fail(ctx, KVZAP_ERR_INVALID_ARG, "window w is negative");
    return KVZAP_OK;
}

}  // namespace kvzap

extern "C" {

kvzap_status kvzap_prune_prefill_paged(kvzap_ctx *ctx, const void *K, const void *V, const float *scores,
                                       const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens, float tau,
                                       int32_t w, void *K_pool, void *V_pool, int64_t n_pages_pool,
                                       int32_t page_tokens, int32_t first_page, int32_t *page_table,
                                       int32_t max_pages_per_list, int32_t *lengths, int32_t *n_pages_used,
                                       void *stream_)
{
    NvtxRange nvtx_range("kvzap_prune_prefill_paged");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    kvzap_status st = check_common(ctx, n_tokens, n_seqs, cu_seqlens);
    if (st != KVZAP_OK) return st;
    if (!lengths || !n_pages_used) return fail(ctx, KVZAP_ERR_INVALID_ARG, "lengths / n_pages_used is NULL");
    DeviceGuard guard(ctx->cfg.device);
    if (n_tokens == 0) {
        KVZAP_CUDA(ctx, cudaMemsetAsync(lengths, 0, sizeof(int32_t) * n_seqs * ctx->cfg.n_kv_heads, stream));
        KVZAP_CUDA(ctx, cudaMemsetAsync(n_pages_used, 0, sizeof(int32_t), stream));
        return KVZAP_OK;
    }
    st = check_paged_args(ctx, K, V, K_pool, V_pool, n_pages_pool, page_tokens, first_page, page_table,
                          max_pages_per_list, lengths, n_pages_used, w);
    if (st != KVZAP_OK) return st;
    if (!scores) return fail(ctx, KVZAP_ERR_INVALID_ARG, "scores is NULL");
    return launch_prune_onepass(ctx, scores, nullptr, tau, w, K, V, cu_seqlens, n_seqs, n_tokens, K_pool, V_pool, lengths,
                                page_tokens, first_page, n_pages_pool, max_pages_per_list, page_table, n_pages_used, stream);
}

static kvzap_status prefill_fused_paged_impl(kvzap_ctx *ctx, int32_t layer, const void *hidden, const void *K,
                                             const void *V, const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                             float tau, int32_t w, void *K_pool, void *V_pool, int64_t n_pages_pool,
                                             int32_t page_tokens, int32_t first_page, int32_t *page_table,
                                             int32_t max_pages_per_list, int32_t *lengths, int32_t *n_pages_used,
                                             float *scores_out, void *stream_, bool tok_major, bool fp8 = false,
                                             const float *x_scale = nullptr)
{
    NvtxRange nvtx_range("kvzap_prefill_fused_paged / kvzap_prefill_write_paged");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, KVZAP_ERR_INVALID_ARG, "layer %d out of range", layer);
    kvzap_status st = check_common(ctx, n_tokens, n_seqs, cu_seqlens);
    if (st != KVZAP_OK) return st;
    if (fp8 ? !ctx->layer_fp8[layer] : !ctx->layer_set[layer])
        return fail(ctx, KVZAP_ERR_STATE, fp8 ? "layer %d has no 8-bit weights (kvzap_set_weights_fp8)" : "layer %d has no weights", layer);
    if (!lengths || !n_pages_used) return fail(ctx, KVZAP_ERR_INVALID_ARG, "lengths / n_pages_used is NULL");
    DeviceGuard guard(ctx->cfg.device);
    if (n_tokens == 0) {
        KVZAP_CUDA(ctx, cudaMemsetAsync(lengths, 0, sizeof(int32_t) * n_seqs * ctx->cfg.n_kv_heads, stream));
        KVZAP_CUDA(ctx, cudaMemsetAsync(n_pages_used, 0, sizeof(int32_t), stream));
        return KVZAP_OK;
    }
    st = check_paged_args(ctx, K, V, K_pool, V_pool, n_pages_pool, page_tokens, first_page, page_table,
                          max_pages_per_list, lengths, n_pages_used, w);
    if (st != KVZAP_OK) return st;
    if (!hidden || !aligned16(hidden)) return fail(ctx, KVZAP_ERR_INVALID_ARG, "hidden must be non-NULL, 16-byte aligned");
    uint32_t *mask = next_mask_slice(ctx);
    st = fp8 ? launch_score_fp8(ctx, layer, hidden, x_scale, n_tokens, scores_out, mask, cu_seqlens, n_seqs, tau, w, stream)
             : launch_score(ctx, layer, 1, hidden, n_tokens, scores_out, mask, cu_seqlens, n_seqs, tau, w, stream);
    if (st != KVZAP_OK) return st;
    return launch_compaction_paged(ctx, mask, K, V, cu_seqlens, n_seqs, n_tokens, K_pool, V_pool, n_pages_pool, page_tokens,
                                   first_page, page_table, max_pages_per_list, lengths, n_pages_used, stream, nullptr,
                                   tok_major);
}

kvzap_status kvzap_prefill_fused_paged(kvzap_ctx *ctx, int32_t layer, const void *hidden, const void *K, const void *V,
                                       const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens, float tau,
                                       int32_t w, void *K_pool, void *V_pool, int64_t n_pages_pool,
                                       int32_t page_tokens, int32_t first_page, int32_t *page_table,
                                       int32_t max_pages_per_list, int32_t *lengths, int32_t *n_pages_used,
                                       float *scores_out, void *stream_)
{
    return prefill_fused_paged_impl(ctx, layer, hidden, K, V, cu_seqlens, n_seqs, n_tokens, tau, w, K_pool, V_pool,
                                    n_pages_pool, page_tokens, first_page, page_table, max_pages_per_list, lengths,
                                    n_pages_used, scores_out, stream_, false);
}

kvzap_status kvzap_prefill_fused_paged_fp8(kvzap_ctx *ctx, int32_t layer, const void *hidden_e4m3, const float *x_scale,
                                           const void *K, const void *V, const int32_t *cu_seqlens, int32_t n_seqs,
                                           int64_t n_tokens, float tau, int32_t w, void *K_pool, void *V_pool,
                                           int64_t n_pages_pool, int32_t page_tokens, int32_t first_page, int32_t *page_table,
                                           int32_t max_pages_per_list, int32_t *lengths, int32_t *n_pages_used,
                                           float *scores_out, void *stream_)
{
    return prefill_fused_paged_impl(ctx, layer, hidden_e4m3, K, V, cu_seqlens, n_seqs, n_tokens, tau, w, K_pool, V_pool,
                                    n_pages_pool, page_tokens, first_page, page_table, max_pages_per_list, lengths,
                                    n_pages_used, scores_out, stream_, false, true, x_scale);
}

kvzap_status kvzap_prefill_write_paged(kvzap_ctx *ctx, int32_t layer, const void *hidden, const void *K_proj,
                                       const void *V_proj, const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                       float tau, int32_t w, void *K_pool, void *V_pool, int64_t n_pages_pool,
                                       int32_t page_tokens, int32_t first_page, int32_t *page_table,
                                       int32_t max_pages_per_list, int32_t *lengths, int32_t *n_pages_used,
                                       float *scores_out, void *stream_)
{
    return prefill_fused_paged_impl(ctx, layer, hidden, K_proj, V_proj, cu_seqlens, n_seqs, n_tokens, tau, w, K_pool,
                                    V_pool, n_pages_pool, page_tokens, first_page, page_table, max_pages_per_list,
                                    lengths, n_pages_used, scores_out, stream_, true);
}

kvzap_status kvzap_cache_create(kvzap_ctx *ctx, kvzap_cache **out, int32_t n_seqs, int32_t window,
                                int32_t page_tokens, void *K_pool, void *V_pool, int64_t n_pages_pool,
                                int32_t max_pages_per_list)
{
    if (!ctx || !out) return KVZAP_ERR_INVALID_ARG;
    *out = nullptr;
    const kvzap_config &c = ctx->cfg;
    if (n_seqs < 1 || n_seqs > c.max_tokens)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "cache: n_seqs %d outside 1..max_tokens", n_seqs);
    if (window < 0 || page_tokens < 1 || max_pages_per_list < 1 || n_pages_pool < 0)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "cache: window >= 0, page_tokens >= 1, max_pages_per_list >= 1 required");
    if (!K_pool || !V_pool || !aligned16(K_pool) || !aligned16(V_pool))
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "cache: pools must be non-NULL and 16-byte aligned");
    DeviceGuard guard(c.device);
    kvzap_cache *cache = new (std::nothrow) kvzap_cache();
    if (!cache) return fail(ctx, KVZAP_ERR_CUDA, "out of host memory");
    cache->ctx = ctx;
    cache->n_lists = static_cast<int64_t>(n_seqs) * c.n_layers * c.n_kv_heads;
    CacheView &v = cache->v;
    memset(&v, 0, sizeof v);
    v.n_seqs = n_seqs; v.n_layers = c.n_layers; v.n_heads = c.n_kv_heads; v.row_units = c.head_dim / 8;
    v.window = window; v.page_tokens = page_tokens; v.max_pages = max_pages_per_list; v.n_pages_pool = n_pages_pool;
    v.k_pool = static_cast<uint4 *>(K_pool); v.v_pool = static_cast<uint4 *>(V_pool);
    const size_t ring_bytes = static_cast<size_t>(cache->n_lists) * (window > 0 ? window : 1) * c.head_dim * 2;
    const size_t n = static_cast<size_t>(cache->n_lists);
    cudaError_t e = cudaSuccess;
    auto alloc = [&](void **p, size_t bytes, bool zero) {
        if (e != cudaSuccess) return;
        e = cudaMalloc(p, bytes);
        if (e == cudaSuccess && zero) e = cudaMemset(*p, 0, bytes);
    };
    alloc(reinterpret_cast<void **>(&v.k_ring), ring_bytes, false);
    alloc(reinterpret_cast<void **>(&v.v_ring), ring_bytes, false);
    alloc(reinterpret_cast<void **>(&v.score_ring), sizeof(float) * n * (window > 0 ? window : 1), true);
    alloc(reinterpret_cast<void **>(&v.n_tokens), sizeof(int32_t) * n, true);
    alloc(reinterpret_cast<void **>(&v.prefix_len), sizeof(int32_t) * n, true);
    alloc(reinterpret_cast<void **>(&v.page_table), sizeof(int32_t) * n * max_pages_per_list, true);
    alloc(reinterpret_cast<void **>(&v.page_cursor), sizeof(int32_t), true);
    alloc(reinterpret_cast<void **>(&v.free_stack), sizeof(int32_t) * static_cast<size_t>(n_pages_pool > 0 ? n_pages_pool : 1), false);
    alloc(reinterpret_cast<void **>(&v.free_top), sizeof(int32_t), true);
    alloc(reinterpret_cast<void **>(&v.active), static_cast<size_t>(n_seqs), false);
    if (e == cudaSuccess) e = cudaMemset(v.active, 1, static_cast<size_t>(n_seqs));      // every slot takes part until released
    {
        const size_t tiles = static_cast<size_t>(c.n_layers) * ((n_seqs + 127) / 128);
        cache->n_step_counters = 12 * tiles;          // done [tiles][4], then ticket [tiles][4][2]
        alloc(reinterpret_cast<void **>(&cache->done), sizeof(int32_t) * cache->n_step_counters, true);
        cache->ticket = cache->done ? cache->done + 4 * tiles : nullptr;
    }
    // two halves used by alternate steps when the caller does not ask for the scores
    alloc(reinterpret_cast<void **>(&cache->scores), 2 * sizeof(float) * static_cast<size_t>(c.n_layers) * n_seqs * c.n_kv_heads,
          false);
    // attention: calls with few lists cut each list into parts; room for 32 units per SM
    cache->attn_units = static_cast<int64_t>(ctx->sm_count) * 32;
    alloc(reinterpret_cast<void **>(&cache->attn_scratch),
          sizeof(float) * static_cast<size_t>(cache->attn_units) * (16 + kAttnMaxGroup * 128), false);
    alloc(reinterpret_cast<void **>(&cache->attn_arrive), sizeof(uint32_t) * static_cast<size_t>(cache->attn_units), true);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        fail(ctx, KVZAP_ERR_CUDA, "cache allocation failed: %s", cudaGetErrorString(e));
        kvzap_cache_destroy(cache);
        return KVZAP_ERR_CUDA;
    }
    ctx->caches.push_back(cache);
    *out = cache;
    return KVZAP_OK;
}

kvzap_status kvzap_cache_debug_skew_steps(kvzap_cache *cache, int32_t delta)
{
    if (!cache) return KVZAP_ERR_INVALID_ARG;
    DeviceGuard guard(cache->ctx->cfg.device);
    if (cudaDeviceSynchronize() != cudaSuccess) return KVZAP_ERR_CUDA;
    const int n = static_cast<int>(cache->n_step_counters / 3 * 2);
    add_int_kernel<<<(n + 255) / 256, 256>>>(cache->ticket, n, delta);
    if (cudaDeviceSynchronize() != cudaSuccess) return KVZAP_ERR_CUDA;
    return KVZAP_OK;
}

kvzap_status kvzap_cache_destroy(kvzap_cache *cache)
{
    if (!cache) return KVZAP_OK;
    DeviceGuard guard(cache->ctx->cfg.device);
    cudaDeviceSynchronize();
    {
        auto &list = cache->ctx->caches;
        for (size_t i = 0; i < list.size(); ++i)
            if (list[i] == cache) { list.erase(list.begin() + static_cast<long>(i)); break; }
        if (cache->ctx->fused_cache == cache) cache->ctx->fused_cache = nullptr;
    }
    cudaFree(cache->v.k_ring); cudaFree(cache->v.v_ring); cudaFree(cache->v.score_ring);
    cudaFree(cache->v.n_tokens); cudaFree(cache->v.prefix_len); cudaFree(cache->v.page_table);
    cudaFree(cache->v.page_cursor); cudaFree(cache->scores); cudaFree(cache->done);
    cudaFree(cache->v.free_stack); cudaFree(cache->v.free_top); cudaFree(cache->v.active);
    cudaFree(cache->attn_scratch); cudaFree(cache->attn_arrive);
    delete cache;
    return KVZAP_OK;
}

static kvzap_status decode_step_impl(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer_begin, int32_t layer_end,
                                     const void *hidden, const float *x_scale, const void *K_new, const void *V_new, float tau,
                                     float *scores_out, void *stream_, bool fp8)
{
    NvtxRange nvtx_range(fp8 ? "kvzap_decode_step_fp8" : "kvzap_decode_step");
    if (!ctx || !cache || cache->ctx != ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const kvzap_config &c = ctx->cfg;
    if (layer_begin < 0 || layer_end > c.n_layers || layer_begin >= layer_end)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "decode: layer range [%d, %d) invalid", layer_begin, layer_end);
    for (int l = layer_begin; l < layer_end; ++l)
        if (fp8 ? !ctx->layer_fp8[l] : !ctx->layer_set[l])
            return fail(ctx, KVZAP_ERR_STATE, fp8 ? "layer %d has no 8-bit weights (kvzap_set_weights_fp8)" : "layer %d has no weights", l);
    if (!hidden || !K_new || !V_new || !aligned16(hidden) || !aligned16(K_new) || !aligned16(V_new))
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "decode: hidden, K_new, V_new must be non-NULL, 16-byte aligned");
    DeviceGuard guard(c.device);
    const int n_layers = layer_end - layer_begin;
    float *scores = scores_out;
    if (!scores) {
        scores = cache->scores + (cache->step_parity ? static_cast<size_t>(c.n_layers) * cache->v.n_seqs * c.n_kv_heads : 0);
        cache->step_parity ^= 1;
    }
    // The whole step in one launch when the few-token scoring kernel applies: the cache update runs in
    // its idle warps.  Needs a window (else the new score decides at once) and every layer of the range
    // at the same step count.
    DecodeFuse fuse;
    memset(&fuse, 0, sizeof fuse);
    const bool can_fuse = cache->v.window > 0 && c.hidden > 0;
    if (can_fuse) {
        fuse.ticket = cache->ticket;
        fuse.c = cache->v;
        fuse.K_new = static_cast<const uint4 *>(K_new);
        fuse.V_new = static_cast<const uint4 *>(V_new);
        fuse.tau = tau;
        fuse.done = cache->done;
        fuse.wait_limit = ctx->wait_limit;
    }
    bool fused = false;
    // the call just before this one was a fused step on this cache: the two may overlap
    const bool chain = ctx->fused_cache == cache && ctx->fused_seq + 1 == ctx->op_seq;
    kvzap_status st = KVZAP_OK;
    const int64_t step_tiles = (static_cast<int64_t>(cache->v.n_seqs) + kTileM - 1) / kTileM * n_layers;
    if (fp8 && !(c.hidden > 0 && ctx->split8_ok && step_tiles * ctx->split_n * ctx->split_k <= ctx->sm_count)) {
        // no few-token layout for this shape: layer after layer through the prefill scoring kernel
        for (int l = 0; l < n_layers && st == KVZAP_OK; ++l)
            st = launch_score_fp8(ctx, layer_begin + l, static_cast<const uint8_t *>(hidden) + static_cast<size_t>(l) * cache->v.n_seqs * c.d_model,
                                  x_scale ? x_scale + static_cast<size_t>(l) * cache->v.n_seqs : nullptr, cache->v.n_seqs,
                                  scores + static_cast<size_t>(l) * cache->v.n_seqs * c.n_kv_heads, nullptr, nullptr, 1, 0.0f, 0, stream);
    } else {
        st = launch_score(ctx, layer_begin, n_layers, hidden, cache->v.n_seqs, scores, nullptr, nullptr, 1,
                          0.0f, 0, stream, 1, can_fuse ? &fuse : nullptr, &fused, chain, nullptr, nullptr, fp8, x_scale);
    }
    if (st != KVZAP_OK) return st;
    if (fused) {
        ctx->fused_cache = cache;
        ctx->fused_seq = ctx->op_seq;
        return KVZAP_OK;
    }
    const int64_t n_groups = static_cast<int64_t>(n_layers) * cache->v.n_seqs * c.n_kv_heads;
    const int64_t threads = n_groups * kDecodeLanes;
    int64_t blocks = (threads + kDecodeThreads - 1) / kDecodeThreads;
    {
        ProfScope prof(ctx, KVZAP_KERNEL_DECODE_UPDATE, stream);
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attrs[2];
        make_launch(&cfg, attrs, dim3(static_cast<unsigned>(blocks)), dim3(kDecodeThreads), 0, stream, !ctx->profiling, 1);
        KVZAP_CUDA(ctx, cudaLaunchKernelEx(&cfg, decode_update_kernel, cache->v, layer_begin, n_layers,
                                           static_cast<const float *>(scores), static_cast<const uint4 *>(K_new),
                                           static_cast<const uint4 *>(V_new), tau, ctx->status_dev,
                                           ctx->last_score_early ? 1 : 0));
    }
    ctx->launches += 1;
    return KVZAP_OK;
}

kvzap_status kvzap_decode_step(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer_begin, int32_t layer_end,
                               const void *hidden, const void *K_new, const void *V_new, float tau,
                               float *scores_out, void *stream_)
{
    return decode_step_impl(ctx, cache, layer_begin, layer_end, hidden, nullptr, K_new, V_new, tau, scores_out, stream_, false);
}

kvzap_status kvzap_decode_step_fp8(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer_begin, int32_t layer_end,
                                   const void *hidden_e4m3, const float *x_scale, const void *K_new, const void *V_new,
                                   float tau, float *scores_out, void *stream_)
{
    return decode_step_impl(ctx, cache, layer_begin, layer_end, hidden_e4m3, x_scale, K_new, V_new, tau, scores_out, stream_, true);
}

static kvzap_status attention_impl(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer_begin, int32_t layer_end,
                                   const void *Q, int32_t n_q_heads, float scale, void *O, void *stream_, bool fp8)
{
    NvtxRange nvtx_range(fp8 ? "kvzap_decode_attention_fp8" : "kvzap_decode_attention");
    if (!ctx || !cache || cache->ctx != ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const kvzap_config &c = ctx->cfg;
    const CacheView &v = cache->v;
    if (layer_begin < 0 || layer_end > c.n_layers || layer_begin >= layer_end)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "attention: layer range [%d, %d) invalid", layer_begin, layer_end);
    if (!Q || !O || !aligned16(Q) || !aligned16(O))
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "attention: Q and O must be non-NULL and 16-byte aligned");
    if (n_q_heads < c.n_kv_heads || n_q_heads % c.n_kv_heads != 0 || n_q_heads / c.n_kv_heads > kAttnMaxGroup)
        return fail(ctx, KVZAP_ERR_UNSUPPORTED, "attention: n_q_heads must be 1..%d times the number of KV heads",
                    kAttnMaxGroup);
    if (!(scale == scale) || scale < 0.0f) return fail(ctx, KVZAP_ERR_INVALID_ARG, "attention: scale must be >= 0");
    DeviceGuard guard(c.device);
    // elements per row as the attention sees them: head_dim bf16 values, or head_dim * 2 - 16 E4M3 codes
    const int d_attn = fp8 ? c.head_dim * 2 - kAttnTrailerBytes : c.head_dim;
    if (d_attn != 64 && d_attn != 128)
        return fail(ctx, KVZAP_ERR_UNSUPPORTED,
                    fp8 ? "8-bit attention needs head_dim 40 or 72 (64 or 128 codes and a 16-byte trailer per row)"
                        : "attention needs head_dim 64 or 128");
    if (cache->attn_state == 0) {
        // tiles of 16 rows: pages and the window must be whole numbers of them; rows of 64 or 128 elements
        const int64_t pool_rows = v.n_pages_pool * v.page_tokens;
        const int64_t ring_rows = cache->n_lists * (v.window > 0 ? v.window : 1);
        const bool ok = (d_attn == 64 || d_attn == 128) && v.page_tokens % kAttnTileRows == 0 &&
                        v.window % kAttnTileRows == 0 && pool_rows < (int64_t{1} << 31) && ring_rows < (int64_t{1} << 31) &&
                        pool_rows >= kAttnTileRows;
        cache->attn_state = -1;
        if (ok) {
            const void *kring = v.window > 0 ? static_cast<const void *>(v.k_ring) : static_cast<const void *>(v.k_pool);
            const void *vring = v.window > 0 ? static_cast<const void *>(v.v_ring) : static_cast<const void *>(v.v_pool);
            const uint64_t rr = v.window > 0 ? static_cast<uint64_t>(ring_rows) : static_cast<uint64_t>(pool_rows);
            const uint32_t rb = static_cast<uint32_t>(c.head_dim) * 2;
            const bool maps_ok = fp8
                ? make_tmap_rows(ctx, &cache->tm_kpool, v.k_pool, static_cast<uint64_t>(pool_rows), rb, kAttnTileRows) == KVZAP_OK &&
                  make_tmap_rows(ctx, &cache->tm_vpool, v.v_pool, static_cast<uint64_t>(pool_rows), rb, kAttnTileRows) == KVZAP_OK &&
                  make_tmap_rows(ctx, &cache->tm_kring, kring, rr, rb, kAttnTileRows) == KVZAP_OK &&
                  make_tmap_rows(ctx, &cache->tm_vring, vring, rr, rb, kAttnTileRows) == KVZAP_OK
                : make_tmap(ctx, &cache->tm_kpool, v.k_pool, static_cast<uint64_t>(pool_rows), c.head_dim, kAttnTileRows) == KVZAP_OK &&
                  make_tmap(ctx, &cache->tm_vpool, v.v_pool, static_cast<uint64_t>(pool_rows), c.head_dim, kAttnTileRows) == KVZAP_OK &&
                  make_tmap(ctx, &cache->tm_kring, kring, rr, c.head_dim, kAttnTileRows) == KVZAP_OK &&
                  make_tmap(ctx, &cache->tm_vring, vring, rr, c.head_dim, kAttnTileRows) == KVZAP_OK;
            if (maps_ok) {
                const int smem = static_cast<int>(attn_smem_bytes(d_attn, fp8));
                cudaError_t e;
                if (fp8)
                    e = d_attn == 128 ? cudaFuncSetAttribute(decode_attn_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)
                                      : cudaFuncSetAttribute(decode_attn_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
                else
                    e = d_attn == 128 ? cudaFuncSetAttribute(decode_attn_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)
                                      : cudaFuncSetAttribute(decode_attn_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
                if (e == cudaSuccess) cache->attn_state = fp8 ? 2 : 1;
            }
        }
    }
    if (cache->attn_state != (fp8 ? 2 : 1))
        return fail(ctx, KVZAP_ERR_UNSUPPORTED,
                    fp8 ? "8-bit attention needs head_dim 40 or 72 (64 or 128 codes and a 16-byte trailer per row), page_tokens and "
                          "window multiples of %d, fewer than 2^31 rows, and a cache not yet used by kvzap_decode_attention"
                        : "attention needs head_dim 64 or 128, page_tokens and window multiples of %d, fewer than 2^31 rows",
                    kAttnTileRows);
    AttnParams p;
    memset(&p, 0, sizeof p);
    p.c = v;
    p.layer0 = layer_begin;
    p.n_layers_call = layer_end - layer_begin;
    p.group = n_q_heads / c.n_kv_heads;
    p.scale_log2e = scale * 1.4426950408889634f;
    p.q = static_cast<const uint16_t *>(Q);
    p.out = static_cast<uint16_t *>(O);
    p.status = ctx->status_dev;
    const int64_t n_lists_call = static_cast<int64_t>(p.n_layers_call) * v.n_seqs * v.n_heads;
    if (n_lists_call > 0x7fffffffLL) return fail(ctx, KVZAP_ERR_UNSUPPORTED, "attention: too many lists for one launch");
    // Two CTAs fit an SM.  With fewer than sixteen CTAs per slot the last, longest lists leave most SMs
    // idle: cut every list into parts so that there are about that many units -- up to 16 parts, or up
    // to 64 when a handful of long lists (a single sequence) is all there is, but never parts shorter
    // than about a thousand rows of the longest list the cache can hold.
    p.n_parts = 1;
    const int64_t want_units = static_cast<int64_t>(ctx->sm_count) * 32;
    if (n_lists_call * 2 <= want_units) {
        int64_t parts = want_units / n_lists_call;
        const int64_t cap = n_lists_call * 16 < 2 * static_cast<int64_t>(ctx->sm_count) ? 64 : 16;
        if (parts > cap) parts = cap;
        const int64_t max_rows = static_cast<int64_t>(v.max_pages) * v.page_tokens + v.window;
        if (parts > 16 && parts > (max_rows + 1023) / 1024) parts = (max_rows + 1023) / 1024 > 16 ? (max_rows + 1023) / 1024 : 16;
        // fewer lists than resident CTA slots: one full wave of equal parts (a second, partly filled wave
        // would cost as much as the first)
        const int64_t slots = 2 * static_cast<int64_t>(ctx->sm_count);
        if (n_lists_call < slots) {
            parts = slots / n_lists_call;
            if (parts > 64) parts = 64;
        }
        if (parts * n_lists_call > cache->attn_units) parts = cache->attn_units / n_lists_call;
        if (parts > 1) p.n_parts = static_cast<int32_t>(parts);
    }
    p.part_scratch = cache->attn_scratch;
    p.part_arrive = cache->attn_arrive;
    const int64_t n_ctas = n_lists_call * p.n_parts;
    {
        ProfScope prof(ctx, KVZAP_KERNEL_ATTENTION, stream);
        const unsigned grid = static_cast<unsigned>(n_ctas);
        const uint32_t smem = attn_smem_bytes(d_attn, fp8);
        if (fp8 && d_attn == 128)
            decode_attn_kernel<128, true><<<grid, kAttnThreads, smem, stream>>>(cache->tm_kpool, cache->tm_vpool, cache->tm_kring, cache->tm_vring, p);
        else if (fp8)
            decode_attn_kernel<64, true><<<grid, kAttnThreads, smem, stream>>>(cache->tm_kpool, cache->tm_vpool, cache->tm_kring, cache->tm_vring, p);
        else if (d_attn == 128)
            decode_attn_kernel<128, false><<<grid, kAttnThreads, smem, stream>>>(cache->tm_kpool, cache->tm_vpool, cache->tm_kring, cache->tm_vring, p);
        else
            decode_attn_kernel<64, false><<<grid, kAttnThreads, smem, stream>>>(cache->tm_kpool, cache->tm_vpool, cache->tm_kring, cache->tm_vring, p);
        KVZAP_CUDA(ctx, cudaGetLastError());
    }
    ctx->launches += 1;
    return KVZAP_OK;
}

kvzap_status kvzap_decode_attention(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer_begin, int32_t layer_end,
                                    const void *Q, int32_t n_q_heads, float scale, void *O, void *stream_)
{
    return attention_impl(ctx, cache, layer_begin, layer_end, Q, n_q_heads, scale, O, stream_, false);
}

kvzap_status kvzap_decode_attention_fp8(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer_begin, int32_t layer_end,
                                        const void *Q, int32_t n_q_heads, float scale, void *O, void *stream_)
{
    return attention_impl(ctx, cache, layer_begin, layer_end, Q, n_q_heads, scale, O, stream_, true);
}

kvzap_status kvzap_cache_release_seq(kvzap_cache *cache, int32_t seq, void *stream_)
{
    if (!cache) return KVZAP_ERR_INVALID_ARG;
    kvzap_ctx *ctx = cache->ctx;
    begin_op(ctx);
    if (seq < 0 || seq >= cache->v.n_seqs) return fail(ctx, KVZAP_ERR_INVALID_ARG, "release: seq %d out of range", seq);
    DeviceGuard guard(ctx->cfg.device);
    release_seq_kernel<<<static_cast<unsigned>(cache->v.n_layers * cache->v.n_heads), 32, 0,
                         static_cast<cudaStream_t>(stream_)>>>(cache->v, seq);
    KVZAP_CUDA(ctx, cudaGetLastError());
    ctx->launches += 1;
    return KVZAP_OK;
}

kvzap_status kvzap_cache_lengths(kvzap_cache *cache, int32_t *lengths, void *stream_)
{
    if (!cache || !lengths) return KVZAP_ERR_INVALID_ARG;
    begin_op(cache->ctx);
    DeviceGuard guard(cache->ctx->cfg.device);
    cache_lengths_kernel<<<static_cast<unsigned>((cache->n_lists + 255) / 256), 256, 0,
                           static_cast<cudaStream_t>(stream_)>>>(cache->v, lengths);
    KVZAP_CUDA(cache->ctx, cudaGetLastError());
    cache->ctx->launches += 1;
    return KVZAP_OK;
}

kvzap_status kvzap_cache_export(kvzap_cache *cache, int32_t seq, int32_t layer, int32_t head, void *K_out, void *V_out,
                                int64_t capacity_rows, int32_t *n_rows, void *stream_)
{
    if (!cache || !K_out || !V_out || !n_rows || capacity_rows < 0) return KVZAP_ERR_INVALID_ARG;
    begin_op(cache->ctx);
    const CacheView &v = cache->v;
    if (seq < 0 || seq >= v.n_seqs || layer < 0 || layer >= v.n_layers || head < 0 || head >= v.n_heads)
        return fail(cache->ctx, KVZAP_ERR_INVALID_ARG, "export: (seq, layer, head) out of range");
    DeviceGuard guard(cache->ctx->cfg.device);
    const int64_t li = (static_cast<int64_t>(seq) * v.n_layers + layer) * v.n_heads + head;
    cache_export_kernel<<<64, 256, 0, static_cast<cudaStream_t>(stream_)>>>(v, li, static_cast<uint4 *>(K_out),
                                                                         static_cast<uint4 *>(V_out), capacity_rows,
                                                                         n_rows);
    KVZAP_CUDA(cache->ctx, cudaGetLastError());
    cache->ctx->launches += 1;
    return KVZAP_OK;
}

kvzap_status kvzap_cache_import(kvzap_cache *cache, const int32_t *prefix_len, const int32_t *page_table,
                                int32_t next_free_page, void *stream_)
{
    if (!cache || !prefix_len || !page_table || next_free_page < 0) return KVZAP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    kvzap_ctx *ctx = cache->ctx;
    begin_op(ctx);
    DeviceGuard guard(ctx->cfg.device);
    const size_t n = static_cast<size_t>(cache->n_lists);
    KVZAP_CUDA(ctx, cudaMemcpyAsync(cache->v.prefix_len, prefix_len, sizeof(int32_t) * n, cudaMemcpyDeviceToDevice, stream));
    KVZAP_CUDA(ctx, cudaMemcpyAsync(cache->v.page_table, page_table, sizeof(int32_t) * n * cache->v.max_pages,
                                    cudaMemcpyDeviceToDevice, stream));
    KVZAP_CUDA(ctx, cudaMemsetAsync(cache->v.n_tokens, 0, sizeof(int32_t) * n, stream));
    KVZAP_CUDA(ctx, cudaMemcpyAsync(cache->v.page_cursor, &next_free_page, sizeof(int32_t), cudaMemcpyHostToDevice, stream));
    KVZAP_CUDA(ctx, cudaMemsetAsync(cache->v.free_top, 0, sizeof(int32_t), stream));
    KVZAP_CUDA(ctx, cudaMemsetAsync(cache->v.active, 1, static_cast<size_t>(cache->v.n_seqs), stream));
    KVZAP_CUDA(ctx, cudaStreamSynchronize(stream));
    return KVZAP_OK;
}

kvzap_status kvzap_cache_snapshot(kvzap_cache *cache, int32_t *prefix_len, int32_t *page_table, int32_t *next_free_page,
                                  void *stream_)
{
    if (!cache || !prefix_len || !page_table || !next_free_page) return KVZAP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    kvzap_ctx *ctx = cache->ctx;
    begin_op(ctx);
    DeviceGuard guard(ctx->cfg.device);
    const size_t n = static_cast<size_t>(cache->n_lists);
    KVZAP_CUDA(ctx, cudaMemcpyAsync(prefix_len, cache->v.prefix_len, sizeof(int32_t) * n, cudaMemcpyDeviceToDevice, stream));
    KVZAP_CUDA(ctx, cudaMemcpyAsync(page_table, cache->v.page_table, sizeof(int32_t) * n * cache->v.max_pages,
                                    cudaMemcpyDeviceToDevice, stream));
    KVZAP_CUDA(ctx, cudaMemcpyAsync(next_free_page, cache->v.page_cursor, sizeof(int32_t), cudaMemcpyDeviceToDevice, stream));
    return KVZAP_OK;
}

kvzap_status kvzap_prefill_to_cache(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer, int32_t seq, const void *hidden,
                                    const void *K, const void *V, int64_t n_tokens, float tau, float *scores_out,
                                    void *stream_)
{
    NvtxRange nvtx_range("kvzap_prefill_to_cache");
    if (!ctx || !cache || cache->ctx != ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const kvzap_config &c = ctx->cfg;
    const CacheView &v = cache->v;
    if (layer < 0 || layer >= c.n_layers || seq < 0 || seq >= v.n_seqs)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "prefill_to_cache: layer %d / seq %d out of range", layer, seq);
    kvzap_status st = check_common(ctx, n_tokens, 1, nullptr);
    if (st != KVZAP_OK) return st;
    if (!ctx->layer_set[layer]) return fail(ctx, KVZAP_ERR_STATE, "layer %d has no weights", layer);
    if (n_tokens == 0) return KVZAP_OK;
    if (!hidden || !K || !V || !scores_out || !aligned16(hidden) || !aligned16(K) || !aligned16(V))
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "prefill_to_cache: hidden, K, V, scores_out must be non-NULL, aligned");
    DeviceGuard guard(c.device);
    const int64_t li0 = (static_cast<int64_t>(seq) * v.n_layers + layer) * v.n_heads;
    // The lists may already hold earlier chunks of the prompt.  Scoring first (mask = threshold only, the
    // chunk's last `window` tokens left out: they go to the ring); then the window side -- the tokens the
    // chunk pushes out of the present window are decided by their buffered scores and appended to the
    // prefix, the chunk's last tokens take their ring slots; then the chunk's kept tokens are appended
    // behind what the lists hold by then.
    uint32_t *mask = next_mask_slice(ctx);
    st = launch_score(ctx, layer, 1, hidden, n_tokens, scores_out, mask, nullptr, 1, tau, v.window, stream, 0);
    if (st != KVZAP_OK) return st;
    if (v.window > 0)
        chunk_ring_kernel<<<static_cast<unsigned>(v.n_heads), 256, 0, stream>>>(
            v, li0, scores_out, static_cast<const uint4 *>(K), static_cast<const uint4 *>(V), n_tokens, tau, ctx->status_dev,
            nullptr, nullptr);
    else
        tokens_add_kernel<<<1, 32, 0, stream>>>(v, li0, n_tokens, nullptr, nullptr);
    KVZAP_CUDA(ctx, cudaGetLastError());
    ctx->launches += 1;
    return launch_compaction_paged(ctx, mask, K, V, nullptr, 1, n_tokens, v.k_pool, v.v_pool, v.n_pages_pool, v.page_tokens, 0,
                                   v.page_table + li0 * v.max_pages, v.max_pages, v.prefix_len + li0, nullptr, stream,
                                   v.page_cursor, false, true, true, v.free_stack, v.free_top);
}

kvzap_status kvzap_prefill_to_cache_batch(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer, const int32_t *seq_ids,
                                          const int32_t *cu_seqlens, int32_t n_seqs, const void *hidden, const void *K,
                                          const void *V, int64_t n_tokens, float tau, float *scores_out, void *stream_)
{
    NvtxRange nvtx_range("kvzap_prefill_to_cache_batch");
    if (!ctx || !cache || cache->ctx != ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const kvzap_config &c = ctx->cfg;
    const CacheView &v = cache->v;
    if (layer < 0 || layer >= c.n_layers) return fail(ctx, KVZAP_ERR_INVALID_ARG, "prefill_to_cache_batch: layer %d out of range", layer);
    if (!seq_ids || !cu_seqlens || n_seqs < 1)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "prefill_to_cache_batch: seq_ids (host), cu_seqlens (device), n_seqs >= 1 are required");
    kvzap_status st = check_common(ctx, n_tokens, n_seqs, cu_seqlens);
    if (st != KVZAP_OK) return st;
    if (!ctx->layer_set[layer]) return fail(ctx, KVZAP_ERR_STATE, "layer %d has no weights", layer);
    // the lists of head 0 of every sequence; slots must be in range and distinct (two chunks for one list in
    // one launch would race)
    std::vector<int64_t> map(static_cast<size_t>(n_seqs));
    {
        std::vector<int32_t> sorted(seq_ids, seq_ids + n_seqs);
        std::sort(sorted.begin(), sorted.end());
        for (int i = 0; i < n_seqs; ++i) {
            if (sorted[i] < 0 || sorted[i] >= v.n_seqs)
                return fail(ctx, KVZAP_ERR_INVALID_ARG, "prefill_to_cache_batch: sequence slot %d out of range", sorted[i]);
            if (i > 0 && sorted[i] == sorted[i - 1])
                return fail(ctx, KVZAP_ERR_INVALID_ARG, "prefill_to_cache_batch: sequence slot %d given twice", sorted[i]);
            map[i] = (static_cast<int64_t>(seq_ids[i]) * v.n_layers + layer) * v.n_heads;
        }
    }
    if (n_tokens == 0) return KVZAP_OK;
    if (!hidden || !K || !V || !scores_out || !aligned16(hidden) || !aligned16(K) || !aligned16(V))
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "prefill_to_cache_batch: hidden, K, V, scores_out must be non-NULL, aligned");
    DeviceGuard guard(c.device);
    if (!ctx->batch_map) KVZAP_CUDA(ctx, cudaMalloc(&ctx->batch_map, sizeof(int64_t) * static_cast<size_t>(c.max_seqs)));
    // from pageable host memory: staged by the driver before the call returns; ordered on the stream behind the
    // kernels of an earlier batch that still read the previous map
    KVZAP_CUDA(ctx, cudaMemcpyAsync(ctx->batch_map, map.data(), sizeof(int64_t) * map.size(), cudaMemcpyHostToDevice, stream));
    uint32_t *mask = next_mask_slice(ctx);
    st = launch_score(ctx, layer, 1, hidden, n_tokens, scores_out, mask, cu_seqlens, n_seqs, tau, v.window, stream, 0);
    if (st != KVZAP_OK) return st;
    if (v.window > 0)
        chunk_ring_kernel<<<dim3(static_cast<unsigned>(v.n_heads), static_cast<unsigned>(n_seqs)), 256, 0, stream>>>(
            v, 0, scores_out, static_cast<const uint4 *>(K), static_cast<const uint4 *>(V), n_tokens, tau, ctx->status_dev,
            ctx->batch_map, cu_seqlens);
    else
        tokens_add_kernel<<<static_cast<unsigned>(n_seqs), 32, 0, stream>>>(v, 0, 0, ctx->batch_map, cu_seqlens);
    KVZAP_CUDA(ctx, cudaGetLastError());
    ctx->launches += 1;
    return launch_compaction_paged(ctx, mask, K, V, cu_seqlens, n_seqs, n_tokens, v.k_pool, v.v_pool, v.n_pages_pool,
                                   v.page_tokens, 0, v.page_table, v.max_pages, v.prefix_len, nullptr, stream, v.page_cursor,
                                   false, true, true, v.free_stack, v.free_top, ctx->batch_map);
}

}  // extern "C"

// ---------------------------------------------------------------------------
// Host-buffer entry points: Algorithm 1 on tensors that live in host memory, layer after layer, with the
// copies of neighbouring layers overlapped.
namespace kvzap {

static kvzap_status host_stage_prepare(kvzap_ctx *ctx, size_t out_bytes, size_t table_ints)
{
    const kvzap_config &c = ctx->cfg;
    const size_t kv_cap = static_cast<size_t>(c.n_kv_heads) * c.max_tokens * c.head_dim * 2;
    const size_t n_lists = static_cast<size_t>(c.max_seqs) * c.n_kv_heads;
    if (!ctx->h2d_stream) {
        KVZAP_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->h2d_stream, cudaStreamNonBlocking));
        KVZAP_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->d2h_stream, cudaStreamNonBlocking));
        KVZAP_CUDA(ctx, cudaMalloc(&ctx->stage_cu, sizeof(int32_t) * (static_cast<size_t>(c.max_seqs) + 1)));
    }
    for (auto &g : ctx->stage) {
        if (!g.x) {
            KVZAP_CUDA(ctx, cudaMalloc(&g.x, static_cast<size_t>(c.max_tokens) * c.d_model * 2));
            KVZAP_CUDA(ctx, cudaMalloc(&g.k, kv_cap));
            KVZAP_CUDA(ctx, cudaMalloc(&g.v, kv_cap));
            KVZAP_CUDA(ctx, cudaMalloc(&g.scores, sizeof(float) * c.max_tokens * c.n_kv_heads));
            KVZAP_CUDA(ctx, cudaMalloc(&g.lengths, sizeof(int32_t) * n_lists));
            KVZAP_CUDA(ctx, cudaMalloc(&g.used, sizeof(int32_t)));
            KVZAP_CUDA(ctx, cudaMallocHost(&g.lengths_pinned, sizeof(int32_t) * (n_lists + 1)));
            KVZAP_CUDA(ctx, cudaEventCreateWithFlags(&g.copied_in, cudaEventDisableTiming));
            KVZAP_CUDA(ctx, cudaEventCreateWithFlags(&g.computed, cudaEventDisableTiming));
        }
        if (g.out_bytes < out_bytes) {          // the output staging grows with the largest call seen (page size is a call argument)
            cudaFree(g.ko); cudaFree(g.vo);
            g.ko = g.vo = nullptr;
            g.out_bytes = 0;
            KVZAP_CUDA(ctx, cudaMalloc(&g.ko, out_bytes));
            KVZAP_CUDA(ctx, cudaMalloc(&g.vo, out_bytes));
            g.out_bytes = out_bytes;
        }
        if (g.table_ints < table_ints) {
            cudaFree(g.table);
            g.table = nullptr;
            g.table_ints = 0;
            KVZAP_CUDA(ctx, cudaMalloc(&g.table, sizeof(int32_t) * table_ints));
            g.table_ints = table_ints;
        }
    }
    return KVZAP_OK;
}

}  // namespace kvzap

extern "C" {

kvzap_status kvzap_prefill_layers_host(kvzap_ctx *ctx, int32_t layer_begin, int32_t layer_end, const void *const *hidden,
                                       const void *const *K, const void *const *V, const int32_t *cu_seqlens, int32_t n_seqs,
                                       int64_t n_tokens, float tau, int32_t w, void *const *K_out, void *const *V_out,
                                       int32_t *const *lengths, float *const *scores_out, int32_t page_tokens,
                                       int64_t n_pages_pool, const int32_t *first_page, int32_t *const *page_table,
                                       int32_t max_pages_per_list, int32_t *const *n_pages_used, void *stream_)
{
    NvtxRange nvtx_range("kvzap_prefill_layers_host");
    if (!ctx) return KVZAP_ERR_INVALID_ARG;
    begin_op(ctx);
    serial_point(ctx);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const kvzap_config &c = ctx->cfg;
    if (layer_begin < 0 || layer_end > c.n_layers || layer_begin >= layer_end)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "host prefill: layer range [%d, %d) invalid", layer_begin, layer_end);
    const int n_layers = layer_end - layer_begin;
    for (int l = layer_begin; l < layer_end; ++l)
        if (!ctx->layer_set[l]) return fail(ctx, KVZAP_ERR_STATE, "layer %d has no weights", l);
    kvzap_status st = check_common(ctx, n_tokens, n_seqs, cu_seqlens);
    if (st != KVZAP_OK) return st;
    if (!lengths || w < 0) return fail(ctx, KVZAP_ERR_INVALID_ARG, "host prefill: lengths is NULL or w negative");
    const bool paged = page_tokens > 0;
    if (page_tokens < 0 || (paged && (!page_table || !n_pages_used || max_pages_per_list < 1 || n_pages_pool < 0)))
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "host prefill: paged output needs page_table, n_pages_used, max_pages_per_list >= 1");
    const size_t n_lists = static_cast<size_t>(n_seqs) * c.n_kv_heads;
    for (int i = 0; i < n_layers; ++i) {
        if (!lengths[i]) return fail(ctx, KVZAP_ERR_INVALID_ARG, "host prefill: lengths[%d] is NULL", i);
        if (paged && (!page_table[i] || !n_pages_used[i])) return fail(ctx, KVZAP_ERR_INVALID_ARG, "host prefill: page_table[%d] / n_pages_used[%d] is NULL", i, i);
        if (paged && first_page && first_page[i] < 0) return fail(ctx, KVZAP_ERR_INVALID_ARG, "host prefill: first_page[%d] negative", i);
    }
    if (n_tokens == 0) {
        for (int i = 0; i < n_layers; ++i) {
            memset(lengths[i], 0, sizeof(int32_t) * n_lists);
            if (paged) *n_pages_used[i] = 0;
        }
        return KVZAP_OK;
    }
    if (!hidden || !K || !V || !K_out || !V_out)
        return fail(ctx, KVZAP_ERR_INVALID_ARG, "host prefill: hidden, K, V, K_out and V_out must not be NULL");
    for (int i = 0; i < n_layers; ++i)
        if (!hidden[i] || !K[i] || !V[i] || !K_out[i] || !V_out[i])
            return fail(ctx, KVZAP_ERR_INVALID_ARG, "host prefill: a tensor pointer of layer %d is NULL", layer_begin + i);
    DeviceGuard guard(c.device);
    const size_t row_bytes = static_cast<size_t>(c.head_dim) * 2;
    const size_t kv_bytes = static_cast<size_t>(c.n_kv_heads) * n_tokens * row_bytes;
    const size_t x_bytes = static_cast<size_t>(n_tokens) * c.d_model * 2;
    const size_t page_bytes = paged ? static_cast<size_t>(page_tokens) * row_bytes : 0;
    // pages one layer can need at most: every list's rows rounded up to whole pages
    const size_t stage_pages = paged ? static_cast<size_t>(c.n_kv_heads) * n_tokens / page_tokens + n_lists + 1 : 0;
    st = host_stage_prepare(ctx, paged ? stage_pages * page_bytes : kv_bytes, paged ? n_lists * max_pages_per_list : 0);
    if (st != KVZAP_OK) return st;
    // everything enqueued on the caller's stream so far comes first
    KVZAP_CUDA(ctx, cudaEventRecord(ctx->stage[0].computed, stream));
    KVZAP_CUDA(ctx, cudaStreamWaitEvent(ctx->h2d_stream, ctx->stage[0].computed, 0));
    if (cu_seqlens)
        KVZAP_CUDA(ctx, cudaMemcpyAsync(ctx->stage_cu, cu_seqlens, sizeof(int32_t) * (n_seqs + 1), cudaMemcpyHostToDevice, ctx->h2d_stream));
    auto copy_in = [&](int i) -> kvzap_status {
        kvzap_ctx::HostStage &g = ctx->stage[i & 1];
        KVZAP_CUDA(ctx, cudaMemcpyAsync(g.x, hidden[i], x_bytes, cudaMemcpyHostToDevice, ctx->h2d_stream));
        KVZAP_CUDA(ctx, cudaMemcpyAsync(g.k, K[i], kv_bytes, cudaMemcpyHostToDevice, ctx->h2d_stream));
        KVZAP_CUDA(ctx, cudaMemcpyAsync(g.v, V[i], kv_bytes, cudaMemcpyHostToDevice, ctx->h2d_stream));
        if (paged)      // the caller's table goes in and comes back whole, so that entries no list uses stay as they were
            KVZAP_CUDA(ctx, cudaMemcpyAsync(g.table, page_table[i], sizeof(int32_t) * n_lists * max_pages_per_list,
                                            cudaMemcpyHostToDevice, ctx->h2d_stream));
        KVZAP_CUDA(ctx, cudaEventRecord(g.copied_in, ctx->h2d_stream));
        return KVZAP_OK;
    };
    st = copy_in(0);
    if (st != KVZAP_OK) return st;
    const int32_t *cu_dev = cu_seqlens ? ctx->stage_cu : nullptr;
    for (int i = 0; i < n_layers; ++i) {
        kvzap_ctx::HostStage &g = ctx->stage[i & 1];
        // the other set is free: the layer that used it was copied out before the previous iteration ended
        if (i + 1 < n_layers && (st = copy_in(i + 1)) != KVZAP_OK) return st;
        KVZAP_CUDA(ctx, cudaStreamWaitEvent(stream, g.copied_in, 0));
        const bool want_scores = scores_out != nullptr && scores_out[i] != nullptr;
        const int32_t fp = paged && first_page ? first_page[i] : 0;
        uint32_t *mask = next_mask_slice(ctx);
        st = launch_score(ctx, layer_begin + i, 1, g.x, n_tokens, want_scores ? g.scores : nullptr, mask, cu_dev, n_seqs, tau, w, stream);
        if (st != KVZAP_OK) return st;
        if (paged) {
            // the staging pool stands for pages first_page .. of the caller's pool
            char *kp = static_cast<char *>(g.ko) - static_cast<size_t>(fp) * page_bytes;
            char *vp = static_cast<char *>(g.vo) - static_cast<size_t>(fp) * page_bytes;
            st = launch_compaction_paged(ctx, mask, g.k, g.v, cu_dev, n_seqs, n_tokens, kp, vp, n_pages_pool, page_tokens, fp, g.table,
                                         max_pages_per_list, g.lengths, g.used, stream);
        } else {
            st = launch_compaction(ctx, mask, g.k, g.v, cu_dev, n_seqs, n_tokens, g.ko, g.vo, g.lengths, stream);
        }
        if (st != KVZAP_OK) return st;
        KVZAP_CUDA(ctx, cudaMemcpyAsync(g.lengths_pinned, g.lengths, sizeof(int32_t) * n_lists, cudaMemcpyDeviceToHost, stream));
        if (paged)
            KVZAP_CUDA(ctx, cudaMemcpyAsync(g.lengths_pinned + n_lists, g.used, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
        KVZAP_CUDA(ctx, cudaEventRecord(g.computed, stream));
        KVZAP_CUDA(ctx, cudaEventSynchronize(g.computed));
        memcpy(lengths[i], g.lengths_pinned, sizeof(int32_t) * n_lists);
        if (want_scores)
            KVZAP_CUDA(ctx, cudaMemcpyAsync(scores_out[i], g.scores, sizeof(float) * n_tokens * c.n_kv_heads, cudaMemcpyDeviceToHost, ctx->d2h_stream));
        if (paged) {
            const int32_t used = g.lengths_pinned[n_lists];
            *n_pages_used[i] = used;
            if (used > 0) {
                // Lists own consecutive pages in list order.  Rows are copied in runs that end where a list's
                // last page is only partly filled, so that the rows behind a list's end stay as the caller had them.
                const int64_t row0 = static_cast<int64_t>(fp) * page_tokens;
                int64_t run_begin = row0, pos = row0;
                auto copy_rows = [&](int64_t from, int64_t to) -> kvzap_status {
                    if (to <= from) return KVZAP_OK;
                    const size_t host_off = static_cast<size_t>(from) * row_bytes, dev_off = static_cast<size_t>(from - row0) * row_bytes;
                    const size_t n = static_cast<size_t>(to - from) * row_bytes;
                    KVZAP_CUDA(ctx, cudaMemcpyAsync(static_cast<char *>(K_out[i]) + host_off, static_cast<char *>(g.ko) + dev_off, n, cudaMemcpyDeviceToHost, ctx->d2h_stream));
                    KVZAP_CUDA(ctx, cudaMemcpyAsync(static_cast<char *>(V_out[i]) + host_off, static_cast<char *>(g.vo) + dev_off, n, cudaMemcpyDeviceToHost, ctx->d2h_stream));
                    return KVZAP_OK;
                };
                for (size_t li = 0; li < n_lists; ++li) {
                    const int64_t len = g.lengths_pinned[li];
                    if (len <= 0) continue;
                    const int64_t n_pages = (len + page_tokens - 1) / page_tokens;
                    if (len % page_tokens != 0) {
                        if ((st = copy_rows(run_begin, pos + len)) != KVZAP_OK) return st;
                        run_begin = pos + n_pages * page_tokens;
                    }
                    pos += n_pages * page_tokens;
                }
                if ((st = copy_rows(run_begin, pos)) != KVZAP_OK) return st;
                KVZAP_CUDA(ctx, cudaMemcpyAsync(page_table[i], g.table, sizeof(int32_t) * n_lists * max_pages_per_list, cudaMemcpyDeviceToHost, ctx->d2h_stream));
            }
        } else {
            for (int b = 0; b < n_seqs; ++b) {
                const int64_t seq_start = cu_seqlens ? cu_seqlens[b] : 0;
                for (int h = 0; h < c.n_kv_heads; ++h) {
                    const int32_t n = g.lengths_pinned[b * c.n_kv_heads + h];
                    if (n <= 0) continue;
                    const size_t off = (static_cast<size_t>(h) * n_tokens + seq_start) * row_bytes;
                    KVZAP_CUDA(ctx, cudaMemcpyAsync(static_cast<char *>(K_out[i]) + off, static_cast<char *>(g.ko) + off, n * row_bytes, cudaMemcpyDeviceToHost, ctx->d2h_stream));
                    KVZAP_CUDA(ctx, cudaMemcpyAsync(static_cast<char *>(V_out[i]) + off, static_cast<char *>(g.vo) + off, n * row_bytes, cudaMemcpyDeviceToHost, ctx->d2h_stream));
                }
            }
        }
        KVZAP_CUDA(ctx, cudaStreamSynchronize(ctx->d2h_stream));
    }
    return KVZAP_OK;
}

kvzap_status kvzap_prefill_fused_host(kvzap_ctx *ctx, int32_t layer, const void *hidden, const void *K, const void *V,
                                      const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens, float tau,
                                      int32_t w, void *K_out, void *V_out, int32_t *lengths, float *scores_out,
                                      void *stream_)
{
    return kvzap_prefill_layers_host(ctx, layer, layer + 1, &hidden, &K, &V, cu_seqlens, n_seqs, n_tokens, tau, w, &K_out, &V_out,
                                     &lengths, &scores_out, 0, 0, nullptr, nullptr, 0, nullptr, stream_);
}

kvzap_status kvzap_prefill_fused_paged_host(kvzap_ctx *ctx, int32_t layer, const void *hidden, const void *K, const void *V,
                                            const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens, float tau, int32_t w,
                                            void *K_pool, void *V_pool, int64_t n_pages_pool, int32_t page_tokens,
                                            int32_t first_page, int32_t *page_table, int32_t max_pages_per_list,
                                            int32_t *lengths, int32_t *n_pages_used, float *scores_out, void *stream_)
{
    if (page_tokens < 1) return ctx ? kvzap::fail(ctx, KVZAP_ERR_INVALID_ARG, "paged host prefill: page_tokens must be >= 1") : KVZAP_ERR_INVALID_ARG;
    return kvzap_prefill_layers_host(ctx, layer, layer + 1, &hidden, &K, &V, cu_seqlens, n_seqs, n_tokens, tau, w, &K_pool, &V_pool,
                                     &lengths, &scores_out, page_tokens, n_pages_pool, &first_page, &page_table,
                                     max_pages_per_list, &n_pages_used, stream_);
}

}  // extern "C"
