// Surrogate scoring on the 5th-generation tensor cores (Method, "KVzap").
//
// Persistent CTAs walk 128-token tiles.  Per tile the first layer
//   Z[128, N] = X[128, D_h] * W1^T          (bf16 x bf16 -> fp32)
// is a chain of tcgen05.mma instructions fed by TMA through a ring of shared
// memory stages, with the accumulator in tensor memory.  The epilogue reads
// the accumulator row by row (one thread per token), and without ever
// touching global memory applies
//   Linear: + b                                         -> H scores
//   MLP:    + b1, GELU (erf form), dot with W2, + b2     -> H scores
// then the threshold / sliding-window test of Algorithm 1, and writes the
// scores (optional) and one keep bit per (head, token) as 32-token words.
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = MMA issuer and
// TMEM owner, warps 2..9 = epilogue (two warps per TMEM lane quarter; in the
// MLP each takes one half of the hidden units and the halves are combined
// through shared memory).
//
// kPair = true runs the kernel as clusters of two CTAs on neighbouring SMs
// (tcgen05 cta_group::2): a pair works on 256 tokens, each CTA holds its own
// 128 rows of X and of the accumulator but only HALF of the W1 rows of every
// K step, and the MMAs issued by the pair's first CTA read both halves.  That
// halves the W1 bytes each SM has to pull from L2 per FLOP, which is what
// bounds the one-CTA version when the hidden layer is wide.
//
// Work tiles are handed out at run time (first tile = the CTA's or pair's own index, further ones from
// a global counter), and the kernel cooperates with the launches around it: it lets the kernel behind
// it in the stream be placed at once, may itself be started before the kernel ahead has finished
// (it reads nothing that kernel writes) and in that case waits for it before it exits -- or, when the
// grid does not fill the machine, before its first store.  The host side explains why that is safe.
#pragma once

#include "ptx.cuh"

namespace kvzap {

constexpr int kTileM = 128;            // tokens per CTA tile = rows of one CTA's accumulator
constexpr int kBlockK = 64;            // bf16 elements per 128-byte swizzled row
constexpr int kUmmaK = 16;             // K of one tcgen05.mma for 16-bit inputs
constexpr int kATileBytes = kTileM * kBlockK * 2;
constexpr int kMaxStages = 8;
constexpr int kScoreThreads = 320;
constexpr int kMaxHeads = 8;

struct ScoreParams {
    int64_t n_tokens;        // rows (tokens) per layer
    int32_t n_tiles;         // work tiles = tiles_per_layer * n_layers_call (a work tile is 128 rows, or 256 for a pair)
    int32_t tiles_per_layer;
    int32_t blocks_per_layer;   // 128-token blocks per layer = ceil(n_tokens / 128)
    int32_t n_layers_call;   // layers scored by this launch (hidden is [n_layers_call][n_tokens][d_model])
    int32_t layer0;          // first layer: selects the rows of the stacked weights
    int32_t w_rows;          // rows of W1 per layer in the stacked weight matrix
    int32_t d_model;
    int32_t group_w;      // accumulator columns computed together (one pass over K)
    int32_t n_groups;     // passes per tile
    int32_t chunk_n;      // N of one MMA instruction
    int32_t n_chunks;     // MMA instructions per K step (group_w = chunk_n * n_chunks)
    int32_t n_stages;
    int32_t acc_bufs;     // accumulator buffers in TMEM (1 or 2)
    int32_t acc_stride;   // TMEM columns between buffers
    int32_t tmem_cols;    // allocation, power of two >= 32
    int32_t n_hidden;     // MLP hidden width (0 for Linear)
    int32_t n_heads;
    // W1 (through the tensor map): K-blocked copy [d_model / 64][L * w_rows][64], see make_tmap_w
    const float *b1;      // stacked over all layers: MLP [L][n_hidden]; Linear [L][16] (zero padded)
    const float *w2t;     // MLP: [L][n_hidden][8] fp32, heads beyond n_heads are zero
    const float *b2;      // MLP: [L][8]
    float *scores;        // [n_layers_call][n_tokens, n_heads] or nullptr
    uint32_t *maskbits;   // [n_layers_call][n_heads][n_words] or nullptr
    int64_t n_words;      // 32-token words per head and layer (= 4 * blocks_per_layer)
    const int32_t *cu_seqlens;   // [n_seqs + 1] or nullptr (one sequence)
    int32_t n_seqs;
    int32_t window;
    int32_t window_keep;  // 1: tokens inside the window are kept (Algorithm 1); 0: they are left out of the mask
    float tau;
    int32_t *status;      // device status word
    int32_t wait_before_write;    // 1: the epilogue waits for the kernel ahead in the stream before its first store
    int32_t wait_before_load;     // 1: every thread waits for the work ahead in the stream before caller data is read
    int32_t *tile_counter;        // work tiles handed out beyond the first one of every CTA (or pair); starts at 0
    int32_t *tile_counter_reset;  // the counter of the launch after next: set to 0 by this launch
    // 8-bit inputs (score_kernel<.., .., true>): hidden states and first-layer weights are E4M3 bytes, a 128-byte
    // swizzled row then holds 128 elements
    int32_t k_blocks;             // K blocks per row of X (0: d_model / 64, the bf16 layout)
    int32_t k_elems;              // elements per K block (0: 64)
    const float *x_scale;         // [n_layers_call][n_tokens] one scale per token, or nullptr (= 1)
    const float *w1_scale;        // stacked over all layers [L][w_rows], one scale per first-layer output row
    // few-token kernel only: the clusters of one tile combine their partial scores through global memory
    float *split_part;            // [n_tiles][n_split][128][8]
    uint32_t *split_arrive;       // [n_tiles] arrivals so far, over all launches (never reset in normal use)
};

// Byte offsets inside the dynamic shared memory block (after 1024-byte alignment).
// `b_rows` = rows of W1 one CTA stages per K step (group_w, or group_w / 2 for a pair).
struct ScoreSmemLayout {
    uint32_t stage_bytes, stages_end, w2s, b1s, w1s, part, bars, total;
};
__host__ __device__ inline ScoreSmemLayout score_smem_layout(int b_rows, int n_stages, int n_hidden)
{
    ScoreSmemLayout L;
    L.stage_bytes = kATileBytes + static_cast<uint32_t>(b_rows) * kBlockK * 2;
    L.stages_end = L.stage_bytes * n_stages;
    L.w2s = L.stages_end;
    L.b1s = L.w2s + static_cast<uint32_t>(n_hidden) * kMaxHeads * 4;
    L.w1s = L.b1s + static_cast<uint32_t>(n_hidden) * 4;        // first-layer row scales (8-bit inputs)
    L.part = L.w1s + static_cast<uint32_t>(n_hidden) * 4;
    L.bars = L.part + kTileM * kMaxHeads * 4;
    L.total = L.bars + 512;
    return L;
}

// GELU(z) = z * Phi(z) for two values at once, through the complementary error function
//   erfc(x) = (a1 t + a2 t^2 + a3 t^3 + a4 t^4 + a5 t^5) exp(-x^2),  t = 1 / (1 + p x),  x >= 0
// (Abramowitz & Stegun, formula 7.1.26, |error| <= 1.5e-7), with x = |z| / sqrt(2):
//   q = erfc(x) / 2,   GELU(z) = z / 2 + |z| (1/2 - q).
// Measured against the fp64 erf form: absolute error below 5e-7 for |z| <= 12.
__device__ __forceinline__ uint64_t gelu_pair(uint64_t z2)
{
    constexpr float kP = 0.3275911f * 0.70710678118654752f;     // p / sqrt(2): t is computed from |z| directly
    constexpr float kA1 = 0.5f * 0.254829592f, kA2 = 0.5f * -0.284496736f, kA3 = 0.5f * 1.421413741f,
                    kA4 = 0.5f * -1.453152027f, kA5 = 0.5f * 1.061405429f;
    constexpr float kC = -0.5f * 1.4426950408889634f;            // exp(-z^2/2) = 2^(kC z^2)
    float z0, z1;
    f2_unpack(z2, z0, z1);
    const uint64_t t = f2_pack(fast_rcp(fmaf(kP, fabsf(z0), 1.0f)), fast_rcp(fmaf(kP, fabsf(z1), 1.0f)));
    uint64_t u = f2_fma(f2_pack(kA5, kA5), t, f2_pack(kA4, kA4));
    u = f2_fma(u, t, f2_pack(kA3, kA3));
    u = f2_fma(u, t, f2_pack(kA2, kA2));
    u = f2_fma(u, t, f2_pack(kA1, kA1));
    u = f2_mul(u, t);
    float m0, m1;
    f2_unpack(f2_mul(f2_mul(z2, z2), f2_pack(kC, kC)), m0, m1);
    const uint64_t q = f2_mul(u, f2_pack(fast_ex2(m0), fast_ex2(m1)));
    float h0, h1;
    f2_unpack(f2_fma(q, f2_pack(-1.0f, -1.0f), f2_pack(0.5f, 0.5f)), h0, h1);
    return f2_pack(fmaf(fabsf(z0), h0, 0.5f * z0), fmaf(fabsf(z1), h1, 0.5f * z1));
}

// Index of the sequence that owns packed token t (cu[b] <= t < cu[b+1]).
__device__ __forceinline__ int seq_of_token(const int32_t *cu, int n_seqs, int64_t t)
{
    int lo = 0, hi = n_seqs;          // invariant: cu[lo] <= t < cu[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (static_cast<int64_t>(__ldg(cu + mid)) <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// Second layer for kCols accumulator columns j0 .. j0+kCols-1 of one token: acc[h] (+)= GELU(r + b1) . W2.
// Hidden units are taken two at a time; acc[h] holds the partial sums of the even and of the odd
// units of head h.  w2p is W2 repacked as [j / 2][h] pairs {W2[h][j], W2[h][j+1]}.
template <int kCols>
__device__ __forceinline__ void mlp_columns(const uint32_t (&r)[kCols], int j0, const float *b1s, const ulonglong2 *w2p,
                                            uint64_t (&acc)[kMaxHeads])
{
#pragma unroll
    for (int i = 0; i < kCols; i += 2) {
        const int j = j0 + i;
        const float2 b = *reinterpret_cast<const float2 *>(b1s + j);
        const uint64_t z2 = f2_add(f2_pack(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), f2_pack(b.x, b.y));
        const uint64_t g2 = gelu_pair(z2);
        const ulonglong2 *w = w2p + (j >> 1) * 4;
#pragma unroll
        for (int hp = 0; hp < 4; ++hp) {
            const ulonglong2 ww = w[hp];
            acc[2 * hp] = f2_fma(g2, ww.x, acc[2 * hp]);
            acc[2 * hp + 1] = f2_fma(g2, ww.y, acc[2 * hp + 1]);
        }
    }
}

// The same with the pre-activation scaled first: z = r * (scale of the token) * (scale of the hidden unit) + b1.
template <int kCols>
__device__ __forceinline__ void mlp_columns_scaled(const uint32_t (&r)[kCols], int j0, const float *b1s, const float *w1s,
                                                   uint64_t sx2, const ulonglong2 *w2p, uint64_t (&acc)[kMaxHeads])
{
#pragma unroll
    for (int i = 0; i < kCols; i += 2) {
        const int j = j0 + i;
        const float2 b = *reinterpret_cast<const float2 *>(b1s + j);
        const float2 sw = *reinterpret_cast<const float2 *>(w1s + j);
        const uint64_t z2 = f2_fma(f2_pack(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), f2_mul(f2_pack(sw.x, sw.y), sx2),
                                   f2_pack(b.x, b.y));
        const uint64_t g2 = gelu_pair(z2);
        const ulonglong2 *w = w2p + (j >> 1) * 4;
#pragma unroll
        for (int hp = 0; hp < 4; ++hp) {
            const ulonglong2 ww = w[hp];
            acc[2 * hp] = f2_fma(g2, ww.x, acc[2 * hp]);
            acc[2 * hp + 1] = f2_fma(g2, ww.y, acc[2 * hp + 1]);
        }
    }
}

// Issues the MMAs of one 64-element K block: kBlockK / kUmmaK steps times kChunks accumulator chunks,
// fully unrolled, descriptors formed by adding constants to the low word (the start-address field).
// a_lo / b_lo: low descriptor words of the stage's A tile and first B chunk; `first` = this is the
// first K block of the accumulation (its first step overwrites the accumulator).
template <bool kPair, int kChunks, bool kFp8 = false>
__device__ __forceinline__ void issue_k_block(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                              uint32_t b_chunk_step, uint32_t chunk_n, uint32_t idesc, bool first)
{
#pragma unroll
    for (int k = 0; k < kBlockK / kUmmaK; ++k) {
#pragma unroll
        for (int c = 0; c < kChunks; ++c) {
            // advancing K by 16 elements = 32 bytes = 2 units of the 16-byte address field
            const uint64_t a_desc = (static_cast<uint64_t>(desc_hi) << 32) | (a_lo + 2 * k);
            const uint64_t b_desc = (static_cast<uint64_t>(desc_hi) << 32) | (b_lo + c * b_chunk_step + 2 * k);
            const uint32_t acc = (k != 0 || !first) ? 1u : 0u;
            if constexpr (kFp8) {
                if constexpr (kPair) umma_fp8_pair(d_tmem + c * chunk_n, a_desc, b_desc, idesc, acc);
                else umma_fp8(d_tmem + c * chunk_n, a_desc, b_desc, idesc, acc);
            } else {
                if constexpr (kPair) umma_bf16_pair(d_tmem + c * chunk_n, a_desc, b_desc, idesc, acc);
                else umma_bf16(d_tmem + c * chunk_n, a_desc, b_desc, idesc, acc);
            }
        }
    }
}

// At most 128 registers per thread: the register file is split over the SM's four schedulers, three
// of this kernel's ten warps share one of them, and a warp of the compaction kernel must still fit
// beside them for the two kernels to run on the same SM at the same time.
template <bool kMlp, bool kPair, bool kFp8 = false>
__global__ void __maxnreg__(128)
score_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
             const ScoreParams p)
{
    static_assert(kMlp || !kPair, "CTA pairs are used for the MLP surrogate only");
    constexpr int kCtas = kPair ? 2 : 1;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t *smem = smem_raw + pad;
    const uint32_t smem_base = raw_addr + pad;
    const int b_rows_chunk = p.chunk_n / kCtas;                 // W1 rows this CTA stages per MMA chunk
    const ScoreSmemLayout L = score_smem_layout(p.group_w / kCtas, p.n_stages, kMlp ? p.n_hidden : 0);

    ulonglong2 *w2p = reinterpret_cast<ulonglong2 *>(smem + L.w2s);
    float *w2f = reinterpret_cast<float *>(smem + L.w2s);
    float *b1s = reinterpret_cast<float *>(smem + L.b1s);
    float *w1s = reinterpret_cast<float *>(smem + L.w1s);
    float *part = reinterpret_cast<float *>(smem + L.part);
    const uint32_t bars = smem_base + L.bars;
    const uint32_t bar_full = bars;                      // [kMaxStages] TMA -> MMA (the pair's first CTA's is used)
    const uint32_t bar_empty = bars + 8 * kMaxStages;    // [kMaxStages] MMA -> TMA
    const uint32_t bar_tfull = bars + 16 * kMaxStages;   // [2] MMA -> epilogue
    const uint32_t bar_tempty = bar_tfull + 16;          // [2] epilogue -> MMA (the pair's first CTA's is used)
    const uint32_t bar_done = bar_tempty + 16;           // [1] abort path only
    const uint32_t bar_pfull = bar_done + 8;             // [1] MLP: second column half -> first
    const uint32_t bar_pempty = bar_pfull + 8;           // [1] MLP: first column half -> second
    const uint32_t bar_epi = bar_pempty + 8;             // [1] MLP: all epilogue warps (weight reload)
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + L.bars + 16 * kMaxStages + 72);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L.bars + 16 * kMaxStages + 76);
    // Work tiles are handed out at run time (see the producer warp): a ring of tile numbers with its own
    // full / empty barriers carries them to the other warps of the CTA (and of the pair's second CTA).
    constexpr uint32_t kSchedSlots = 4;
    const uint32_t bar_sfull = bars + 16 * kMaxStages + 80;      // [kSchedSlots] scheduler -> consumers
    const uint32_t bar_sempty = bar_sfull + 8 * kSchedSlots;     // [kSchedSlots] consumers -> scheduler (first CTA's)
    volatile int32_t *tile_ring = reinterpret_cast<volatile int32_t *>(smem + L.bars + 16 * kMaxStages + 80 + 16 * kSchedSlots);
    const uint32_t tile_ring_addr = bars + 16 * kMaxStages + 80 + 16 * kSchedSlots;

    // Let the kernel behind this one in the stream (the compaction) be placed right away; it waits
    // for this kernel's results itself.
    griddep_launch_dependents();
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    constexpr int kEpiWarps = kMlp ? 8 : 4;
    uint32_t cta_rank = 0;
    if constexpr (kPair) cta_rank = cluster_cta_rank();
    const bool leader = cta_rank == 0;
    const int unit = kPair ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
    const int n_units = kPair ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tfull + 8 * b, 1);
            mbar_init(bar_tempty + 8 * b, kEpiWarps * kCtas);
        }
        mbar_init(bar_done, 1);
        mbar_init(bar_pfull, 4);
        mbar_init(bar_pempty, 4);
        mbar_init(bar_epi, kEpiWarps);
        // consumers of a tile number: the second CTA's producer warp, the MMA warp, every epilogue warp
        for (uint32_t i = 0; i < kSchedSlots; ++i) {
            mbar_init(bar_sfull + 8 * i, 1);
            mbar_init(bar_sempty + 8 * i, (kCtas - 1) + 1 + kEpiWarps * kCtas);
        }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_x);
        prefetch_tensormap(&tmap_w);
    }
    if (warp == 1) {
        if constexpr (kPair) {
            tmem_alloc_pair(smem_u32(const_cast<uint32_t *>(tmem_slot)), static_cast<uint32_t>(p.tmem_cols));
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), static_cast<uint32_t>(p.tmem_cols));
            tmem_relinquish();
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if constexpr (kPair) cluster_sync_all();     // the other CTA's barriers exist before anything signals them
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // The set-up above overlaps the tail of the work ahead in the stream either way; unless the caller
    // vouches for the producers of its inputs, nothing of them is read before that work has completed.
    if (p.wait_before_load) griddep_wait();

    const int k_blocks = p.k_blocks > 0 ? p.k_blocks : p.d_model / kBlockK;
    const int k_elems = p.k_elems > 0 ? p.k_elems : kBlockK;
    if (blockIdx.x == 0 && threadIdx.x == 0) *p.tile_counter_reset = 0;

    // The seq-th work tile of this CTA (pair), as published by the scheduler; -1 if the kernel is
    // aborting.  Called by all lanes of a warp; values >= p.n_tiles mean "no more work".
    uint32_t sempty_addr = bar_sempty;
    if constexpr (kPair) sempty_addr = map_to_cta(bar_sempty, 0);
    auto sched_get = [&](uint32_t seq) -> int {
        const uint32_t slot = seq % kSchedSlots;
        if (!__all_sync(0xffffffffu, mbar_wait_cluster(bar_sfull + 8 * slot, (seq / kSchedSlots) & 1u, abort_flag)))
            return -1;
        const int t = tile_ring[slot];
        __syncwarp();
        if (lane == 0) {
            if constexpr (kPair) mbar_arrive_cluster(sempty_addr + 8 * slot);
            else mbar_arrive(bar_sempty + 8 * slot);
        }
        return t;
    };

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs of a pair)
        const uint64_t pol_x1 = l2_policy_evict_first();  // hidden states are streamed once ...
        const uint64_t pol_xn = l2_policy_evict_normal(); // ... unless a second pass over K follows (hidden > 512)
        const uint64_t pol_w = l2_policy_evict_last();    // weights are re-read by every tile
        uint32_t full0_cluster = bar_full;                // the pair's first CTA's full barriers
        if constexpr (kPair) full0_cluster = map_to_cta(bar_full, 0);
        // Ring position kept incrementally (stage index, its shared-memory address, the parity to wait
        // for): the loop body is a chain of dependent instructions in one warp, so every one counts.
        uint32_t it = 0, seq = 0;
        uint32_t st = 0, st_par = 1, st_addr = smem_base;       // empty barriers: the first pass is free
        const bool elected = elect_one();
        bool ok = true;
        // The first CTA's producer warp is also the scheduler: every CTA (pair) starts with the tile of
        // its own index and takes further ones from a global counter, so that CTAs that start early
        // (on SMs the previous launch left first) end up with more tiles than those that start late.
        auto publish = [&](uint32_t q, int t) -> bool {
            const uint32_t slot = q % kSchedSlots;
            if (q >= kSchedSlots &&
                !__all_sync(0xffffffffu, mbar_wait_cluster(bar_sempty + 8 * slot, ((q / kSchedSlots) & 1u) ^ 1u, abort_flag)))
                return false;
            if (lane == 0) {
                tile_ring[slot] = t;
                mbar_arrive(bar_sfull + 8 * slot);
                if constexpr (kPair) {
                    st_shared_cluster_u32(map_to_cta(tile_ring_addr + 4 * slot, 1), static_cast<uint32_t>(t));
                    mbar_arrive_cluster(map_to_cta(bar_sfull + 8 * slot, 1));
                }
            }
            __syncwarp();
            return true;
        };
        int tile = unit;
        if (leader) ok = publish(0, tile);
        else tile = sched_get(0);
        while (ok && tile >= 0 && tile < p.n_tiles) {
            int tile_next = 0;
            if (leader && lane == 0) tile_next = n_units + atomicAdd(p.tile_counter, 1);   // used after this tile's loads
            const int l_rel = tile / p.tiles_per_layer;
            const int m_tile = (tile - l_rel * p.tiles_per_layer) * kCtas + static_cast<int>(cta_rank);
            const int row0 = m_tile * kTileM;
            for (int g = 0; g < p.n_groups && ok; ++g) {
                const int w_row0 = (p.layer0 + l_rel) * p.w_rows + g * p.group_w + static_cast<int>(cta_rank) * b_rows_chunk;
                // Two passes over K: the second walks the K blocks backwards, so that it starts with the X
                // blocks the first pass loaded last (still in L2; all CTAs together have more X in flight
                // than L2 holds, walking forwards again every block would come from HBM a second time).
                const bool backwards = (g & 1) != 0;
                const uint64_t pol_x = (g + 1 < p.n_groups) ? pol_xn : pol_x1;
                for (int i = 0; i < k_blocks; ++i, ++it) {
                    const int kb = backwards ? k_blocks - 1 - i : i;
                    const int kx = kb * k_elems;
                    if (!__all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * st, st_par, abort_flag))) {
                        ok = false;
                        break;
                    }
                    if (elected) {
                        const uint32_t sa = st_addr;
                        if constexpr (kPair) {
                            // the first CTA's barrier counts the bytes of both CTAs
                            if (leader) mbar_arrive_expect_tx(bar_full + 8 * st, L.stage_bytes * 2);
                            const uint32_t bar = full0_cluster + 8 * st;
                            tma_load_3d_pair(sa, &tmap_x, bar, kx, row0, l_rel, pol_x);
                            tma_load_3d_pair(sa + kATileBytes, &tmap_w, bar, 0, w_row0, kb, pol_w);
                            if (p.n_chunks == 2)
                                tma_load_3d_pair(sa + kATileBytes + b_rows_chunk * kBlockK * 2, &tmap_w, bar, 0,
                                                 w_row0 + p.chunk_n, kb, pol_w);
                        } else {
                            mbar_arrive_expect_tx(bar_full + 8 * st, L.stage_bytes);
                            tma_load_3d(sa, &tmap_x, bar_full + 8 * st, kx, row0, l_rel, pol_x);
                            tma_load_3d(sa + kATileBytes, &tmap_w, bar_full + 8 * st, 0, w_row0, kb, pol_w);
                            if (p.n_chunks == 2)
                                tma_load_3d(sa + kATileBytes + p.chunk_n * kBlockK * 2, &tmap_w, bar_full + 8 * st, 0,
                                            w_row0 + p.chunk_n, kb, pol_w);
                        }
                    }
                    __syncwarp();
                    st_addr += L.stage_bytes;
                    if (++st == static_cast<uint32_t>(p.n_stages)) { st = 0; st_par ^= 1u; st_addr = smem_base; }
                }
            }
            if (!ok) break;
            ++seq;
            if (leader) {
                tile_next = __shfl_sync(0xffffffffu, tile_next, 0);
                ok = publish(seq, tile_next);
                tile = tile_next;
            } else {
                tile = sched_get(seq);
            }
        }
        if (tile < 0) ok = false;
        if (!ok && lane == 0) {
            // abort path: let the copies already in flight land before the CTA exits
            if (leader) {
                const uint32_t n_out = it < static_cast<uint32_t>(p.n_stages) ? it : static_cast<uint32_t>(p.n_stages);
                for (uint32_t j = 0; j < n_out; ++j) {
                    const uint32_t fill = it - 1 - j;
                    const uint32_t s = fill % p.n_stages;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(bar_full + 8 * s, (fill / p.n_stages) & 1u))
                        if (clock64() - t0 > KVZAP_WAIT_LIMIT_CYCLES / 16) break;
                }
            } else {
                // this CTA's copies complete on the other CTA's barriers: give them a fixed time instead
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000LL) { }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (a pair: its first CTA only)
        if (leader) {
            const uint32_t idesc = kFp8 ? umma_idesc_e4m3_f32(kTileM * kCtas, static_cast<uint32_t>(p.chunk_n))
                                        : umma_idesc_bf16_f32(kTileM * kCtas, static_cast<uint32_t>(p.chunk_n));
            // operand descriptors: constant high word, low word = (address >> 4) | fixed fields
            const uint64_t desc0 = umma_desc_k_major_sw128(smem_base);
            const uint32_t desc_hi = static_cast<uint32_t>(desc0 >> 32);
            const uint32_t desc_lo0 = static_cast<uint32_t>(desc0);
            const uint32_t b_chunk_step = static_cast<uint32_t>(b_rows_chunk * kBlockK * 2) >> 4;
            const uint32_t stage_units = L.stage_bytes >> 4;
            const bool elected = elect_one();               // the same lane issues every MMA and commit
            uint32_t acc_it = 0;
            uint32_t st = 0, st_par = 0, a_lo = desc_lo0;    // ring position, kept incrementally
            bool ok = true;
            for (uint32_t seq = 0; ok; ++seq) {
                const int tile = sched_get(seq);
                if (tile < 0) { ok = false; break; }
                if (tile >= p.n_tiles) break;
                for (int g = 0; g < p.n_groups && ok; ++g, ++acc_it) {
                    const uint32_t buf = acc_it % p.acc_bufs;
                    const uint32_t use = acc_it / p.acc_bufs;
                    // every lane waits (no broadcast needed afterwards); one elected lane issues
                    if (!__all_sync(0xffffffffu, mbar_wait(bar_tempty + 8 * buf, (use & 1u) ^ 1u, abort_flag))) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + buf * p.acc_stride;
                    for (int kb = 0; kb < k_blocks; ++kb) {
                        if (!__all_sync(0xffffffffu, mbar_wait(bar_full + 8 * st, st_par, abort_flag))) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        if (elected) {
                            const uint32_t b_lo = a_lo + (kATileBytes >> 4);
                            if (p.n_chunks == 1)
                                issue_k_block<kPair, 1, kFp8>(d_tmem, a_lo, b_lo, desc_hi, b_chunk_step, p.chunk_n, idesc, kb == 0);
                            else
                                issue_k_block<kPair, 2, kFp8>(d_tmem, a_lo, b_lo, desc_hi, b_chunk_step, p.chunk_n, idesc, kb == 0);
                            // the stage is free (in both CTAs) once these MMAs retire
                            if constexpr (kPair) umma_commit_pair(bar_empty + 8 * st, 3);
                            else umma_commit(bar_empty + 8 * st);
                        }
                        __syncwarp();
                        a_lo += stage_units;
                        if (++st == static_cast<uint32_t>(p.n_stages)) { st = 0; st_par ^= 1u; a_lo = desc_lo0; }
                    }
                    if (ok && elected) {                     // accumulator complete
                        if constexpr (kPair) umma_commit_pair(bar_tfull + 8 * buf, 3);
                        else umma_commit(bar_tfull + 8 * buf);
                    }
                    __syncwarp();
                }
            }
            __syncwarp();
            if (!ok && elected) {
                // abort path: wait (bounded) for the MMAs already issued before TMEM is freed
                if constexpr (kPair) umma_commit_pair(bar_done, 1);
                else umma_commit(bar_done);
                const long long t0 = clock64();
                while (!mbar_try_wait(bar_done, 0))
                    if (clock64() - t0 > KVZAP_WAIT_LIMIT_CYCLES / 16) break;
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int ew = warp - 2;            // 0..7
        const int q = warp & 3;             // TMEM lane quarter this warp may read
        const int hsel = ew >> 2;           // MLP: which half of the group's columns
        const int row = q * 32 + lane;      // token row inside the tile
        const bool active = kMlp || hsel == 0;
        uint32_t acc_it = 0, tile_it = 0, epi_it = 0;
        int cur_layer = -1;
        bool waited = false;
        bool ok = true;
        uint32_t tempty_addr[2] = {bar_tempty, bar_tempty + 8};
        if constexpr (kPair) {
            tempty_addr[0] = map_to_cta(bar_tempty, 0);
            tempty_addr[1] = map_to_cta(bar_tempty + 8, 0);
        }
        if (active) {
            for (uint32_t seq = 0; ok; ++seq, ++tile_it) {
                const int tile = sched_get(seq);
                if (tile < 0) { ok = false; break; }
                if (tile >= p.n_tiles) break;
                const int l_rel = tile / p.tiles_per_layer;
                const int m_tile = (tile - l_rel * p.tiles_per_layer) * kCtas + static_cast<int>(cta_rank);
                const int layer = p.layer0 + l_rel;
                if constexpr (kMlp) {
                    if (layer != cur_layer) {
                        // (re)load this layer's b1 and W2 into shared memory; all epilogue warps have
                        // finished the previous tile's reads once they have all arrived here
                        const int etid = threadIdx.x - 64;
                        if (cur_layer >= 0) {
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar_epi);
                            if (!mbar_wait(bar_epi, epi_it & 1u, abort_flag)) { ok = false; break; }
                            ++epi_it;
                        }
                        const float *w2g = p.w2t + static_cast<int64_t>(layer) * p.n_hidden * kMaxHeads;
                        const float *b1g = p.b1 + static_cast<int64_t>(layer) * p.n_hidden;
                        for (int i = etid; i < p.n_hidden * kMaxHeads; i += kEpiWarps * 32) {
                            const int j = i >> 3, h = i & 7;      // W2[h][j] -> pair slot (j / 2, h), element j % 2
                            w2f[(((j >> 1) * kMaxHeads + h) << 1) + (j & 1)] = __ldg(w2g + i);
                        }
                        for (int i = etid; i < p.n_hidden; i += kEpiWarps * 32) b1s[i] = __ldg(b1g + i);
                        if constexpr (kFp8)
                            for (int i = etid; i < p.n_hidden; i += kEpiWarps * 32)
                                w1s[i] = __ldg(p.w1_scale + static_cast<int64_t>(layer) * p.n_hidden + i);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_epi);
                        if (!mbar_wait(bar_epi, epi_it & 1u, abort_flag)) { ok = false; break; }
                        ++epi_it;
                        cur_layer = layer;
                    }
                }
                float s[kMaxHeads];
                uint64_t acc[kMaxHeads];
#pragma unroll
                for (int h = 0; h < kMaxHeads; ++h) { s[h] = 0.0f; acc[h] = 0ull; }
                float sx = 1.0f;                               // 8-bit inputs: this token's scale
                if constexpr (kFp8) {
                    const int64_t t_row = static_cast<int64_t>(m_tile) * kTileM + row;
                    if (p.x_scale != nullptr && t_row < p.n_tokens) sx = __ldg(p.x_scale + static_cast<int64_t>(l_rel) * p.n_tokens + t_row);
                }
                for (int g = 0; g < p.n_groups; ++g, ++acc_it) {
                    const uint32_t buf = acc_it % p.acc_bufs;
                    const uint32_t use = acc_it / p.acc_bufs;
                    if (!mbar_wait(bar_tfull + 8 * buf, use & 1u, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * p.acc_stride;
                    if constexpr (kMlp) {
                        const int half_w = p.group_w >> 1;
                        const int col0 = hsel * half_w;
                        const int j0 = g * p.group_w + col0;
                        // two register sets: the next 16 columns are in flight while these are processed
                        uint32_t ra[16], rb[16];
                        tmem_ld_x16(t_row + col0, ra);
                        for (int c = 0; c < half_w; c += 32) {
                            tmem_wait_ld();
                            reg_fence16(ra);
                            tmem_ld_x16(t_row + col0 + c + 16, rb);
                            if constexpr (kFp8) mlp_columns_scaled<16>(ra, j0 + c, b1s, w1s, f2_pack(sx, sx), w2p, acc);
                            else mlp_columns<16>(ra, j0 + c, b1s, w2p, acc);
                            tmem_wait_ld();
                            reg_fence16(rb);
                            if (c + 32 < half_w) tmem_ld_x16(t_row + col0 + c + 32, ra);
                            if constexpr (kFp8) mlp_columns_scaled<16>(rb, j0 + c + 16, b1s, w1s, f2_pack(sx, sx), w2p, acc);
                            else mlp_columns<16>(rb, j0 + c + 16, b1s, w2p, acc);
                        }
                    } else {
                        uint32_t r[16];
                        tmem_ld_x16(t_row, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int h = 0; h < kMaxHeads; ++h) {
                            if constexpr (kFp8)
                                s[h] = fmaf(__uint_as_float(r[h]), sx * __ldg(p.w1_scale + layer * p.w_rows + h), __ldg(p.b1 + layer * p.w_rows + h));
                            else
                                s[h] = __uint_as_float(r[h]) + __ldg(p.b1 + layer * p.w_rows + h);
                        }
                    }
                    // this warp is done reading the accumulator buffer
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) {
                        if constexpr (kPair) mbar_arrive_cluster(tempty_addr[buf]);
                        else mbar_arrive(bar_tempty + 8 * buf);
                    }
                }
                if (!ok) break;
                if constexpr (kMlp) {
#pragma unroll
                    for (int h = 0; h < kMaxHeads; ++h) {
                        float lo, hi;
                        f2_unpack(acc[h], lo, hi);
                        s[h] = lo + hi;
                    }
                    // combine the two column halves through `part`; the hsel = 0 warps finish the tile
                    if (hsel == 1) {
                        if (!mbar_wait(bar_pempty, (tile_it & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                        float4 *dst = reinterpret_cast<float4 *>(part + row * kMaxHeads);
                        dst[0] = make_float4(s[0], s[1], s[2], s[3]);
                        dst[1] = make_float4(s[4], s[5], s[6], s[7]);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_pfull);
                    } else {
                        if (!mbar_wait(bar_pfull, tile_it & 1u, abort_flag)) { ok = false; break; }
                        const float4 *src = reinterpret_cast<const float4 *>(part + row * kMaxHeads);
                        const float4 pa = src[0], pb = src[1];
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_pempty);
                        s[0] += pa.x + __ldg(p.b2 + layer * kMaxHeads + 0);
                        s[1] += pa.y + __ldg(p.b2 + layer * kMaxHeads + 1);
                        s[2] += pa.z + __ldg(p.b2 + layer * kMaxHeads + 2);
                        s[3] += pa.w + __ldg(p.b2 + layer * kMaxHeads + 3);
                        s[4] += pb.x + __ldg(p.b2 + layer * kMaxHeads + 4);
                        s[5] += pb.y + __ldg(p.b2 + layer * kMaxHeads + 5);
                        s[6] += pb.z + __ldg(p.b2 + layer * kMaxHeads + 6);
                        s[7] += pb.w + __ldg(p.b2 + layer * kMaxHeads + 7);
                    }
                }
                if (hsel == 0 && m_tile < p.blocks_per_layer) {
                    if (p.wait_before_write && !waited) {
                        // started early on a machine that was not full: the buffers written below may still
                        // be in use by the calls before this one until the kernel ahead has completed
                        griddep_wait();
                        waited = true;
                    }
                    const int64_t t = static_cast<int64_t>(m_tile) * kTileM + row;      // row inside the layer
                    const bool valid = t < p.n_tokens;
                    if (valid && p.scores != nullptr) {
                        float *dst = p.scores + (static_cast<int64_t>(l_rel) * p.n_tokens + t) * p.n_heads;
                        if (p.n_heads == kMaxHeads) {
                            reinterpret_cast<float4 *>(dst)[0] = make_float4(s[0], s[1], s[2], s[3]);
                            reinterpret_cast<float4 *>(dst)[1] = make_float4(s[4], s[5], s[6], s[7]);
                        } else {
#pragma unroll
                            for (int h = 0; h < kMaxHeads; ++h)
                                if (h < p.n_heads) dst[h] = s[h];
                        }
                    }
                    if (p.maskbits != nullptr) {
                        bool in_window = false;
                        if (valid) {
                            int64_t seq_end = p.n_tokens;
                            if (p.cu_seqlens != nullptr && p.n_seqs > 1)
                                seq_end = __ldg(p.cu_seqlens + seq_of_token(p.cu_seqlens, p.n_seqs, t) + 1);
                            in_window = t >= seq_end - static_cast<int64_t>(p.window);
                        }
                        uint32_t my_word = 0;
#pragma unroll
                        for (int h = 0; h < kMaxHeads; ++h) {
                            const bool keep = valid && (in_window ? p.window_keep != 0 : s[h] >= p.tau);
                            const uint32_t word = __ballot_sync(0xffffffffu, keep);
                            if (lane == h) my_word = word;
                        }
                        if (lane < p.n_heads)
                            p.maskbits[(static_cast<int64_t>(l_rel) * p.n_heads + lane) * p.n_words +
                                       static_cast<int64_t>(m_tile) * 4 + q] = my_word;
                    }
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    // a pair: neither CTA leaves (or frees tensor memory) while the other may still read its shared
    // memory, signal its barriers or write its accumulator
    if constexpr (kPair) cluster_sync_all();
    if (threadIdx.x == 0 && *abort_flag) atomicCAS(p.status, 0, 5 /* KVZAP_ERR_TIMEOUT */);
    // If this kernel was allowed to start before the one ahead of it had finished, no CTA leaves
    // before that kernel is complete: kernels then still complete in stream order, and a CTA of the
    // next scoring kernel that finds this SM free knows that everything two launches back is done.
    griddep_wait();      // every thread executes it: a wait by some threads only was seen not to hold the others' CTA back
    if (warp == 1) {
        tc_fence_after_sync();
        if constexpr (kPair) tmem_dealloc_pair(tmem_base, static_cast<uint32_t>(p.tmem_cols));
        else tmem_dealloc(tmem_base, static_cast<uint32_t>(p.tmem_cols));
    }
}

}  // namespace kvzap
