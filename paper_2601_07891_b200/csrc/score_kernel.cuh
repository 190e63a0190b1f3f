// Surrogate scoring on the 5th-generation tensor cores (Method, "KVzap").
//
// One persistent CTA per SM walks 128-token tiles.  Per tile the first layer
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
#pragma once

#include "ptx.cuh"

namespace kvzap {

constexpr int kTileM = 128;            // tokens per tile = UMMA M
constexpr int kBlockK = 64;            // bf16 elements per 128-byte swizzled row
constexpr int kUmmaK = 16;             // K of one tcgen05.mma for 16-bit inputs
constexpr int kATileBytes = kTileM * kBlockK * 2;
constexpr int kMaxStages = 8;
constexpr int kScoreThreads = 320;
constexpr int kMaxHeads = 8;

struct ScoreParams {
    int64_t n_tokens;        // rows (tokens) per layer
    int32_t n_tiles;         // tiles_per_layer * n_layers_call
    int32_t tiles_per_layer;
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
    const float *b1;      // stacked over all layers: MLP [L][n_hidden]; Linear [L][16] (zero padded)
    const float *w2t;     // MLP: [L][n_hidden][8] fp32, heads beyond n_heads are zero
    const float *b2;      // MLP: [L][8]
    float *scores;        // [n_layers_call][n_tokens, n_heads] or nullptr
    uint32_t *maskbits;   // [n_layers_call][n_heads][n_words] or nullptr
    int64_t n_words;      // 32-token words per head and layer (= 4 * tiles_per_layer)
    const int32_t *cu_seqlens;   // [n_seqs + 1] or nullptr (one sequence)
    int32_t n_seqs;
    int32_t window;
    int32_t window_keep;  // 1: tokens inside the window are kept (Algorithm 1); 0: they are left out of the mask
    float tau;
    int32_t *status;      // device status word
};

// Byte offsets inside the dynamic shared memory block (after 1024-byte alignment).
struct ScoreSmemLayout {
    uint32_t stage_bytes, stages_end, w2s, b1s, part, bars, total;
};
__host__ __device__ inline ScoreSmemLayout score_smem_layout(int group_w, int n_stages, int n_hidden)
{
    ScoreSmemLayout L;
    L.stage_bytes = kATileBytes + static_cast<uint32_t>(group_w) * kBlockK * 2;
    L.stages_end = L.stage_bytes * n_stages;
    L.w2s = L.stages_end;
    L.b1s = L.w2s + static_cast<uint32_t>(n_hidden) * kMaxHeads * 4;
    L.part = L.b1s + static_cast<uint32_t>(n_hidden) * 4;
    L.bars = L.part + kTileM * kMaxHeads * 4;
    L.total = L.bars + 256;
    return L;
}

__device__ __forceinline__ float gelu_erf(float z)
{
    return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f));
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

template <bool kMlp>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
             const ScoreParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t *smem = smem_raw + pad;
    const uint32_t smem_base = raw_addr + pad;
    const ScoreSmemLayout L = score_smem_layout(p.group_w, p.n_stages, kMlp ? p.n_hidden : 0);

    float4 *w2s = reinterpret_cast<float4 *>(smem + L.w2s);
    float *b1s = reinterpret_cast<float *>(smem + L.b1s);
    float *part = reinterpret_cast<float *>(smem + L.part);
    const uint32_t bars = smem_base + L.bars;
    const uint32_t bar_full = bars;                      // [kMaxStages] TMA -> MMA
    const uint32_t bar_empty = bars + 8 * kMaxStages;    // [kMaxStages] MMA -> TMA
    const uint32_t bar_tfull = bars + 16 * kMaxStages;   // [2] MMA -> epilogue
    const uint32_t bar_tempty = bar_tfull + 16;          // [2] epilogue -> MMA
    const uint32_t bar_done = bar_tempty + 16;           // [1] abort path only
    const uint32_t bar_pfull = bar_done + 8;             // [1] MLP: second column half -> first
    const uint32_t bar_pempty = bar_pfull + 8;           // [1] MLP: first column half -> second
    const uint32_t bar_epi = bar_pempty + 8;             // [1] MLP: all epilogue warps (weight reload)
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + L.bars + 16 * kMaxStages + 72);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L.bars + 16 * kMaxStages + 76);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    constexpr int kEpiWarps = kMlp ? 8 : 4;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tfull + 8 * b, 1);
            mbar_init(bar_tempty + 8 * b, kEpiWarps);
        }
        mbar_init(bar_done, 1);
        mbar_init(bar_pfull, 4);
        mbar_init(bar_pempty, 4);
        mbar_init(bar_epi, kEpiWarps);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_x);
        prefetch_tensormap(&tmap_w);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), static_cast<uint32_t>(p.tmem_cols));
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    const int k_blocks = p.d_model / kBlockK;
    const uint32_t stage_tx = L.stage_bytes;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        const uint64_t pol_x = l2_policy_evict_first();   // hidden states are streamed once
        const uint64_t pol_w = l2_policy_evict_last();    // weights are re-read by every tile
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
            for (int g = 0; g < p.n_groups && ok; ++g) {
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const uint32_t s = it % p.n_stages;
                    const uint32_t round = it / p.n_stages;
                    int got = 0;
                    if (lane == 0) got = mbar_wait(bar_empty + 8 * s, (round & 1u) ^ 1u, abort_flag) ? 1 : 0;
                    got = __shfl_sync(0xffffffffu, got, 0);
                    if (!got) { ok = false; break; }
                    if (lane == 0) {
                        const uint32_t sa = smem_base + s * L.stage_bytes;
                        mbar_arrive_expect_tx(bar_full + 8 * s, stage_tx);
                        const int l_rel = tile / p.tiles_per_layer;
                        const int m_tile = tile - l_rel * p.tiles_per_layer;
                        const int w_row0 = (p.layer0 + l_rel) * p.w_rows + g * p.group_w;
                        tma_load_3d(sa, &tmap_x, bar_full + 8 * s, kb * kBlockK, m_tile * kTileM, l_rel, pol_x);
                        for (int c = 0; c < p.n_chunks; ++c)
                            tma_load_2d(sa + kATileBytes + c * p.chunk_n * kBlockK * 2, &tmap_w, bar_full + 8 * s,
                                        kb * kBlockK, w_row0 + c * p.chunk_n, pol_w);
                    }
                    __syncwarp();
                }
            }
        }
        if (!ok && lane == 0) {
            // abort path: let the copies already in flight land before the CTA exits
            const uint32_t n_out = it < static_cast<uint32_t>(p.n_stages) ? it : static_cast<uint32_t>(p.n_stages);
            for (uint32_t j = 0; j < n_out; ++j) {
                const uint32_t fill = it - 1 - j;
                const uint32_t s = fill % p.n_stages;
                const long long t0 = clock64();
                while (!mbar_try_wait(bar_full + 8 * s, (fill / p.n_stages) & 1u))
                    if (clock64() - t0 > KVZAP_WAIT_LIMIT_CYCLES / 16) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        const uint32_t idesc = umma_idesc_bf16_f32(kTileM, static_cast<uint32_t>(p.chunk_n));
        uint32_t it = 0, acc_it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x) {
            for (int g = 0; g < p.n_groups && ok; ++g, ++acc_it) {
                const uint32_t buf = acc_it % p.acc_bufs;
                const uint32_t use = acc_it / p.acc_bufs;
                int got = 0;
                if (lane == 0) got = mbar_wait(bar_tempty + 8 * buf, (use & 1u) ^ 1u, abort_flag) ? 1 : 0;
                got = __shfl_sync(0xffffffffu, got, 0);
                if (!got) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * p.acc_stride;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const uint32_t s = it % p.n_stages;
                    const uint32_t round = it / p.n_stages;
                    if (lane == 0) got = mbar_wait(bar_full + 8 * s, round & 1u, abort_flag) ? 1 : 0;
                    got = __shfl_sync(0xffffffffu, got, 0);
                    if (!got) { ok = false; break; }
                    tc_fence_after_sync();
                    if (lane == 0) {
                        const uint32_t sa = smem_base + s * L.stage_bytes;
                        const uint64_t a_desc = umma_desc_k_major_sw128(sa);
#pragma unroll
                        for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                            // advancing K by 16 elements = 32 bytes = 2 descriptor address units
                            for (int c = 0; c < p.n_chunks; ++c) {
                                const uint64_t b_desc =
                                    umma_desc_k_major_sw128(sa + kATileBytes + c * p.chunk_n * kBlockK * 2);
                                umma_bf16(d_tmem + c * p.chunk_n, a_desc + 2 * k, b_desc + 2 * k, idesc,
                                          (kb | k) != 0 ? 1u : 0u);
                            }
                        }
                        umma_commit(bar_empty + 8 * s);          // stage is free once these MMAs retire
                    }
                    __syncwarp();
                }
                if (ok && lane == 0) umma_commit(bar_tfull + 8 * buf);   // accumulator complete
                __syncwarp();
            }
        }
        if (!ok && lane == 0) {
            // abort path: wait (bounded) for the MMAs already issued before TMEM is freed
            umma_commit(bar_done);
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_done, 0))
                if (clock64() - t0 > KVZAP_WAIT_LIMIT_CYCLES / 16) break;
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
        bool ok = true;
        if (active) {
            for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++tile_it) {
                const int l_rel = tile / p.tiles_per_layer;
                const int m_tile = tile - l_rel * p.tiles_per_layer;
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
                        const float4 *w2g = reinterpret_cast<const float4 *>(p.w2t) +
                                            static_cast<int64_t>(layer) * p.n_hidden * 2;
                        const float *b1g = p.b1 + static_cast<int64_t>(layer) * p.n_hidden;
                        for (int i = etid; i < p.n_hidden * 2; i += kEpiWarps * 32) w2s[i] = __ldg(w2g + i);
                        for (int i = etid; i < p.n_hidden; i += kEpiWarps * 32) b1s[i] = __ldg(b1g + i);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_epi);
                        if (!mbar_wait(bar_epi, epi_it & 1u, abort_flag)) { ok = false; break; }
                        ++epi_it;
                        cur_layer = layer;
                    }
                }
                float s[kMaxHeads];
#pragma unroll
                for (int h = 0; h < kMaxHeads; ++h) s[h] = 0.0f;
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
                        for (int c = 0; c < half_w; c += 32) {
                            uint32_t r[32];
                            tmem_ld_x32(t_row + col0 + c, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                const int j = j0 + c + i;
                                const float gz = gelu_erf(__uint_as_float(r[i]) + b1s[j]);
                                const float4 wa = w2s[2 * j], wb = w2s[2 * j + 1];
                                s[0] = fmaf(gz, wa.x, s[0]);
                                s[1] = fmaf(gz, wa.y, s[1]);
                                s[2] = fmaf(gz, wa.z, s[2]);
                                s[3] = fmaf(gz, wa.w, s[3]);
                                s[4] = fmaf(gz, wb.x, s[4]);
                                s[5] = fmaf(gz, wb.y, s[5]);
                                s[6] = fmaf(gz, wb.z, s[6]);
                                s[7] = fmaf(gz, wb.w, s[7]);
                            }
                        }
                    } else {
                        uint32_t r[16];
                        tmem_ld_x16(t_row, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int h = 0; h < kMaxHeads; ++h)
                            s[h] = __uint_as_float(r[h]) + __ldg(p.b1 + layer * p.w_rows + h);
                    }
                    // this warp is done reading the accumulator buffer
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
                }
                if (!ok) break;
                if constexpr (kMlp) {
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
                if (hsel == 0) {
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
    if (threadIdx.x == 0 && *abort_flag) atomicCAS(p.status, 0, 5 /* KVZAP_ERR_TIMEOUT */);
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, static_cast<uint32_t>(p.tmem_cols));
    }
}

}  // namespace kvzap
