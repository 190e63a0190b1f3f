// KVzap-Linear scoring (Method, "KVzap": one linear map from the hidden state to H scores) for SHORT
// inputs: a prompt of a few thousand tokens gives only a few dozen 128-token tiles, and with one CTA
// per tile most SMs would idle while each busy one streams a whole 1 MB tile of hidden states at the
// rate a single SM can pull (the launch then takes ~20 us however fast HBM is).  Here a cluster of
// kLinSplit CTAs shares a tile: CTA r runs the K blocks [r, r+1) * d_model / kLinSplit of the product
// (its quarter of the X tile, its quarter of W), the partial 128 x 8 sums of the others go to the
// cluster's first CTA through distributed shared memory, and after one cluster barrier that CTA adds
// them in rank order plus the bias and writes scores and keep bits.
//
// Warp roles as in score_kernel: warp 0 TMA producer, warp 1 MMA issuer / TMEM owner, warps 2..5
// epilogue (TMEM lane quarter = warp % 4).  The kernel may be placed before the kernel ahead of it in
// the stream has finished: it reads only hidden states and weights, every thread waits for that
// kernel before it exits, and with p.wait_before_write set nothing is written before that wait either
// (the host sets it unless the mask slice and the scores buffer written here are known to be free).
#pragma once

#include "prune_onepass_kernel.cuh"
#include "score_kernel.cuh"

namespace kvzap {

constexpr int kLinSplit = 4;
constexpr int kLinStages = 8;             // pipeline stages; kLinStagesCompact when the compaction runs in the same launch
constexpr int kLinStagesCompact = 2;      // (four CTAs then fit an SM: the launches of the next calls run beside this one;
                                          //  measured per call at 4096 tokens: 8.8 us with 2 stages, 9.9 with 3, 9.6 with 5)
constexpr int kLinThreads = 192;          // producer warp, MMA warp, four epilogue warps
constexpr int kLinMaxTiles = 64;          // tiles of a launch that also compacts (its clusters wait for one another)
constexpr uint32_t kLinBTileBytes = 16 * kBlockK * 2;                 // 16 weight rows (H <= 8, padded) of one K block
constexpr uint32_t kLinStageBytes = kATileBytes + kLinBTileBytes;    // 18 KB, a multiple of 1024
// shared memory after the stages: [kLinSplit - 1][128][8] fp32 partial sums, then barriers and flags
__host__ __device__ constexpr uint32_t lin_xpart_off(int n_stages) { return static_cast<uint32_t>(n_stages) * kLinStageBytes; }
__host__ __device__ constexpr uint32_t lin_bars_off(int n_stages) { return lin_xpart_off(n_stages) + (kLinSplit - 1) * kTileM * kMaxHeads * 4; }
__host__ __device__ constexpr uint32_t lin_smem_bytes(int n_stages) { return lin_bars_off(n_stages) + 256 + 1024; }   // + alignment slack
constexpr uint32_t kLinSmemBytes = lin_smem_bytes(kLinStages);

// The compaction of Algorithm 1 inside the scoring launch (one sequence, dense-ragged output, one layer per
// launch, a grid that is resident at once): the cluster of a tile publishes the tile's kept count per head,
// adds up the counts of the tiles before it, and moves its own tile's kept rows -- each of its four CTAs a
// quarter of the tile's tokens -- through the pipeline stages, which are idle by then.  (Bulk copies, one
// per 256-byte row, were tried for that and moved rows at 2.7 TB/s; 16-byte asynchronous copies do 4+.)
struct LinCompact {
    int32_t enabled;
    int32_t row_bytes;           // 2 * head_dim, a multiple of 16
    const char *K, *V;           // row (h, t) at (h * in_stride_h + t * in_stride_t) * row_bytes
    char *K_out, *V_out;         // [H][n_tokens][D]
    int64_t in_stride_h, in_stride_t;
    int32_t *lengths;            // [H]
    uint64_t *tile_counts;       // [n_tiles][8]: (call number << 32) | rows of head h kept in the tile
    int32_t epoch;               // the call's number, never 0
    int32_t n_stages;
    int64_t wait_limit;
};

// gridDim.x = kLinSplit * p.n_tiles (cluster dimension kLinSplit); p.n_tiles = 128-token tiles over all
// layers of the call, p.tiles_per_layer of them per layer; d_model / 64 divisible by kLinSplit.
__global__ void __launch_bounds__(kLinThreads)
score_linear_split_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                          const ScoreParams p, const LinCompact fc)
{
    __shared__ uint32_t wt_s[kMaxHeads][4];             // compaction: the tile's keep words (head, quarter of the tile)
    __shared__ int32_t run_s[kMaxHeads];                //             rows of head h kept before the tile
    __shared__ int32_t red_s[kLinThreads / 32][kMaxHeads];
    __shared__ int64_t ent_src_s[kMaxHeads * 32], ent_dst_s[kMaxHeads * 32];     // kept rows of this CTA's quarter (byte offsets)
    const int n_st = fc.enabled ? fc.n_stages : kLinStages;
    extern __shared__ uint8_t lin_smem_raw[];
    const uint32_t raw_addr = smem_u32(lin_smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t *smem = lin_smem_raw + pad;
    const uint32_t smem_base = raw_addr + pad;
    const uint32_t xpart_off = lin_xpart_off(n_st), bars_off = lin_bars_off(n_st);
    float *xpart = reinterpret_cast<float *>(smem + xpart_off);
    const uint32_t bars = smem_base + bars_off;
    const uint32_t bar_full = bars;                       // [kLinStages] TMA -> MMA
    const uint32_t bar_empty = bars + 8 * kLinStages;     // [kLinStages] MMA -> TMA
    const uint32_t bar_tfull = bars + 16 * kLinStages;    // MMA -> epilogue
    const uint32_t bar_done = bar_tfull + 8;              // abort path only
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + bars_off + 16 * kLinStages + 16);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + bars_off + 16 * kLinStages + 20);

    griddep_launch_dependents();
    if (p.wait_before_load) griddep_wait();     // caller data is read only after the work ahead in the stream is complete
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();
    const int tile = static_cast<int>(blockIdx.x) / kLinSplit;
    const int l_rel = tile / p.tiles_per_layer;
    const int m_tile = tile - l_rel * p.tiles_per_layer;
    const int layer = p.layer0 + l_rel;
    constexpr uint32_t kTmemCols = 32;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kLinStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_tfull, 1);
        mbar_init(bar_done, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_x);
        prefetch_tensormap(&tmap_w);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const int k_blocks = p.d_model / kBlockK / kLinSplit;      // K blocks of this CTA
    const int kb_first = static_cast<int>(rank) * k_blocks;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        const uint64_t pol_x = l2_policy_evict_first();    // every byte of X is read once
        const uint64_t pol_w = l2_policy_evict_last();     // the weights are shared by all tiles of the layer
        const bool elected = elect_one();
        const int w_row = layer * p.w_rows;
        const int row0 = m_tile * kTileM;
        uint32_t st = 0, st_par = 1, sa = smem_base;
        bool ok = true;
        for (int kb = 0; kb < k_blocks; ++kb) {
            if (!__all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * st, st_par, abort_flag))) {
                ok = false;
                break;
            }
            if (elected) {
                mbar_arrive_expect_tx(bar_full + 8 * st, kLinStageBytes);
                tma_load_3d(sa + kATileBytes, &tmap_w, bar_full + 8 * st, 0, w_row, kb_first + kb, pol_w);
                tma_load_3d(sa, &tmap_x, bar_full + 8 * st, (kb_first + kb) * kBlockK, row0, l_rel, pol_x);
            }
            __syncwarp();
            sa += kLinStageBytes;
            if (++st == static_cast<uint32_t>(n_st)) { st = 0; st_par ^= 1u; sa = smem_base; }
        }
        if (!ok && lane == 0) {
            // abort path: give the copies already in flight a fixed time to land before the CTA exits
            const long long t0 = clock64();
            while (clock64() - t0 < 2000000LL) { }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        const uint32_t idesc = umma_idesc_bf16_f32(kTileM, 16);
        const uint64_t desc0 = umma_desc_k_major_sw128(smem_base);
        const uint32_t desc_hi = static_cast<uint32_t>(desc0 >> 32);
        const uint32_t desc_lo0 = static_cast<uint32_t>(desc0);
        const bool elected = elect_one();
        uint32_t st = 0, st_par = 0, a_lo = desc_lo0;
        bool ok = true;
        for (int kb = 0; kb < k_blocks; ++kb) {
            if (!__all_sync(0xffffffffu, mbar_wait(bar_full + 8 * st, st_par, abort_flag))) {
                ok = false;
                break;
            }
            tc_fence_after_sync();
            if (elected) {
                issue_k_block<false, 1>(tmem_base, a_lo, a_lo + (kATileBytes >> 4), desc_hi, 0, 0, idesc, kb == 0);
                umma_commit(bar_empty + 8 * st);
            }
            __syncwarp();
            a_lo += kLinStageBytes >> 4;
            if (++st == static_cast<uint32_t>(n_st)) { st = 0; st_par ^= 1u; a_lo = desc_lo0; }
        }
        if (ok && elected) umma_commit(bar_tfull);
        __syncwarp();
        if (!ok && elected) {
            umma_commit(bar_done);
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_done, 0))
                if (clock64() - t0 > KVZAP_WAIT_LIMIT_CYCLES / 16) break;
        }
    }

    // ------------------------------------------------------------ epilogue (warps 2..5): one thread per token
    const bool epi = warp >= 2;
    const int q = warp & 3;                 // TMEM lane quarter
    const int row = q * 32 + lane;
    float s[kMaxHeads];
#pragma unroll
    for (int h = 0; h < kMaxHeads; ++h) s[h] = 0.0f;
    if (epi) {
        if (mbar_wait(bar_tfull, 0, abort_flag)) {
            tc_fence_after_sync();
            uint32_t r[16];
            tmem_ld_x16(tmem_base + (static_cast<uint32_t>(q * 32) << 16), r);
            tmem_wait_ld();
#pragma unroll
            for (int h = 0; h < kMaxHeads; ++h) s[h] = __uint_as_float(r[h]);
        }
        if (rank != 0) {
            // the partial sums of this CTA's K range go to the first CTA: xpart[rank - 1][row][8]
            const uint32_t dst = map_to_cta(smem_base + xpart_off + ((rank - 1) * kTileM + row) * kMaxHeads * 4, 0);
            st_shared_cluster_v4(dst, s[0], s[1], s[2], s[3]);
            st_shared_cluster_v4(dst + 16, s[4], s[5], s[6], s[7]);
        }
    }
    tc_fence_before_sync();
    // every thread of every CTA of the cluster arrives here (all waits above are bounded)
    cluster_sync_all();
    if (threadIdx.x == 0 && *abort_flag) atomicCAS(p.status, 0, 5 /* KVZAP_ERR_TIMEOUT */);
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    // nothing has been written so far
    if (fc.enabled) {
        // ------------------------------------------------------------ scoring and compaction in one launch
        if (p.wait_before_write) griddep_wait();           // every thread: outputs may still be in use by the work ahead
        const uint32_t wt_addr = smem_u32(&wt_s[0][0]);
        if (rank == 0 && epi) {
#pragma unroll
            for (int r = 0; r < kLinSplit - 1; ++r) {
                const float4 *src = reinterpret_cast<const float4 *>(xpart + (r * kTileM + row) * kMaxHeads);
                const float4 pa = src[0], pb = src[1];
                s[0] += pa.x; s[1] += pa.y; s[2] += pa.z; s[3] += pa.w;
                s[4] += pb.x; s[5] += pb.y; s[6] += pb.z; s[7] += pb.w;
            }
#pragma unroll
            for (int h = 0; h < kMaxHeads; ++h) s[h] += __ldg(p.b1 + layer * p.w_rows + h);
            const int64_t t = static_cast<int64_t>(m_tile) * kTileM + row;
            const bool valid = t < p.n_tokens;
            if (valid && p.scores != nullptr) {
                float *dst = p.scores + t * p.n_heads;
                if (p.n_heads == kMaxHeads) {
                    reinterpret_cast<float4 *>(dst)[0] = make_float4(s[0], s[1], s[2], s[3]);
                    reinterpret_cast<float4 *>(dst)[1] = make_float4(s[4], s[5], s[6], s[7]);
                } else {
#pragma unroll
                    for (int h = 0; h < kMaxHeads; ++h)
                        if (h < p.n_heads) dst[h] = s[h];
                }
            }
            const bool in_window = valid && t >= p.n_tokens - static_cast<int64_t>(p.window);      // one sequence
            uint32_t my_word = 0;
#pragma unroll
            for (int h = 0; h < kMaxHeads; ++h) {
                const bool keep = valid && (in_window || s[h] >= p.tau);
                const uint32_t word = __ballot_sync(0xffffffffu, keep);
                if (lane == h) my_word = word;
            }
            if (lane < kMaxHeads) {
                if (lane >= p.n_heads || *abort_flag) my_word = 0;      // a pipeline that gave up: nothing is kept, nothing moved
                // the tile's keep words go to all four CTAs of the cluster
#pragma unroll
                for (uint32_t r = 0; r < kLinSplit; ++r)
                    st_shared_cluster_u32(map_to_cta(wt_addr + (lane * 4 + q) * 4, r), my_word);
            }
        }
        cluster_sync_all();
        const uint64_t tag = static_cast<uint64_t>(static_cast<uint32_t>(fc.epoch)) << 32;
        if (rank == 0 && threadIdx.x < kMaxHeads) {
            const int cnt = __popc(wt_s[threadIdx.x][0]) + __popc(wt_s[threadIdx.x][1]) + __popc(wt_s[threadIdx.x][2]) +
                            __popc(wt_s[threadIdx.x][3]);
            st_relaxed_gpu_u64(fc.tile_counts + tile * kMaxHeads + threadIdx.x, tag | static_cast<uint32_t>(cnt));
        }
        // rows kept before this tile: the counts of the tiles before it (every CTA of the cluster adds them up itself)
        {
            int32_t acc[kMaxHeads];
#pragma unroll
            for (int h = 0; h < kMaxHeads; ++h) acc[h] = 0;
            for (int j = threadIdx.x; j < tile; j += kLinThreads) {
                const uint64_t *e = fc.tile_counts + static_cast<int64_t>(j) * kMaxHeads;
                ulonglong2 v[4];
                const long long t_begin = clock64();
                for (;;) {
                    bool all = true;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        v[i] = ld_relaxed_gpu_v2(e + 2 * i);
                        all = all && (v[i].x >> 32) == (tag >> 32) && (v[i].y >> 32) == (tag >> 32);
                    }
                    if (all) break;
                    if (clock64() - t_begin > fc.wait_limit) { *abort_flag = 2; break; }
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[2 * i] += static_cast<int32_t>(static_cast<uint32_t>(v[i].x));
                    acc[2 * i + 1] += static_cast<int32_t>(static_cast<uint32_t>(v[i].y));
                }
            }
#pragma unroll
            for (int h = 0; h < kMaxHeads; ++h) acc[h] = __reduce_add_sync(0xffffffffu, acc[h]);
            if (lane == 0) {
#pragma unroll
                for (int h = 0; h < kMaxHeads; ++h) red_s[warp][h] = acc[h];
            }
            __syncthreads();
            if (threadIdx.x < kMaxHeads) {
                int32_t r = 0;
#pragma unroll
                for (int wv = 0; wv < kLinThreads / 32; ++wv) r += red_s[wv][threadIdx.x];
                run_s[threadIdx.x] = r;
            }
            __syncthreads();
        }
        if (*abort_flag == 2) {                             // a tile before this one never published: nothing is moved
            if (threadIdx.x == 0) atomicCAS(p.status, 0, 5 /* KVZAP_ERR_TIMEOUT */);
            griddep_wait();
            return;
        }
        // this CTA's quarter of the tile: tokens 32 * rank .. + 31, all heads; its kept rows listed by (head, token)
        const int64_t t_q0 = static_cast<int64_t>(m_tile) * kTileM + rank * 32;
        int n_rows = 0;
        for (int h = 0; h < p.n_heads; ++h) n_rows += __popc(wt_s[h][rank]);
        for (int pi = threadIdx.x; pi < p.n_heads * 32; pi += kLinThreads) {
            const int h = pi >> 5, tk = pi & 31;
            const uint32_t w = wt_s[h][rank];
            if ((w >> tk) & 1u) {
                int idx = __popc(w & ((1u << tk) - 1u)), before = 0;
                for (int hh = 0; hh < h; ++hh) idx += __popc(wt_s[hh][rank]);
                for (uint32_t qq = 0; qq < rank; ++qq) before += __popc(wt_s[h][qq]);
                const int64_t n = run_s[h] + before + __popc(w & ((1u << tk) - 1u));          // rank inside head h's list
                ent_src_s[idx] = (h * fc.in_stride_h + (t_q0 + tk) * fc.in_stride_t) * fc.row_bytes;
                ent_dst_s[idx] = (static_cast<int64_t>(h) * p.n_tokens + n) * fc.row_bytes;
            }
        }
        if (rank == 0 && m_tile == p.tiles_per_layer - 1 && threadIdx.x < p.n_heads) {
            const int h = threadIdx.x;
            fc.lengths[h] = run_s[h] + __popc(wt_s[h][0]) + __popc(wt_s[h][1]) + __popc(wt_s[h][2]) + __popc(wt_s[h][3]);
        }
        __syncthreads();
        // rows travel global -> the idle pipeline stages -> global; as many per round as the stages hold
        const int cap = static_cast<int>(static_cast<uint32_t>(n_st) * kLinStageBytes / (2u * fc.row_bytes));
        // as asynchronous 16-byte copies into shared memory (they pass by the L1 and the registers, so the rows of
        // a round are all in flight at once), 16 lanes per row, then ordinary loads from there and stores
        const int group = threadIdx.x >> 4, gl = threadIdx.x & 15;
        for (int c0 = 0; c0 < n_rows; c0 += cap) {
            const int n_chunk = n_rows - c0 < cap ? n_rows - c0 : cap;
            for (int i = group; i < n_chunk; i += kLinThreads / 16) {
                const uint32_t slot = smem_base + static_cast<uint32_t>(i) * 2u * fc.row_bytes;
                const int64_t src = ent_src_s[c0 + i];
                for (uint32_t u = gl * 16u; u < static_cast<uint32_t>(fc.row_bytes); u += 256u) {
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot + u), "l"(fc.K + src + u) : "memory");
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot + fc.row_bytes + u), "l"(fc.V + src + u) : "memory");
                }
            }
            asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
            __syncthreads();
            for (int i = group; i < n_chunk; i += kLinThreads / 16) {
                const uint8_t *slot = smem + static_cast<uint32_t>(i) * 2u * fc.row_bytes;
                const int64_t dst = ent_dst_s[c0 + i];
                for (uint32_t u = gl * 16u; u < static_cast<uint32_t>(fc.row_bytes); u += 256u) {
                    *reinterpret_cast<uint4 *>(fc.K_out + dst + u) = *reinterpret_cast<const uint4 *>(slot + u);
                    *reinterpret_cast<uint4 *>(fc.V_out + dst + u) = *reinterpret_cast<const uint4 *>(slot + fc.row_bytes + u);
                }
            }
            __syncthreads();
        }
        griddep_wait();                                     // this kernel still completes after the one ahead of it
        return;
    }
    // nothing has been written so far
    if (p.wait_before_write || rank != 0 || !epi) {
        griddep_wait();                     // from here on the kernel ahead in the stream has completed
        if (rank != 0 || !epi) return;
    }

    // ------------------------------------------------------------ first CTA: total, scores, keep bits
#pragma unroll
    for (int r = 0; r < kLinSplit - 1; ++r) {
        const float4 *src = reinterpret_cast<const float4 *>(xpart + (r * kTileM + row) * kMaxHeads);
        const float4 pa = src[0], pb = src[1];
        s[0] += pa.x; s[1] += pa.y; s[2] += pa.z; s[3] += pa.w;
        s[4] += pb.x; s[5] += pb.y; s[6] += pb.z; s[7] += pb.w;
    }
#pragma unroll
    for (int h = 0; h < kMaxHeads; ++h) s[h] += __ldg(p.b1 + layer * p.w_rows + h);
    const int64_t t = static_cast<int64_t>(m_tile) * kTileM + row;
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
            p.maskbits[(static_cast<int64_t>(l_rel) * p.n_heads + lane) * p.n_words + static_cast<int64_t>(m_tile) * 4 + q] = my_word;
    }
    griddep_wait();                         // this kernel still completes after the one ahead of it
}

}  // namespace kvzap
