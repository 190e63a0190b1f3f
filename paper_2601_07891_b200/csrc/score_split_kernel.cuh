// MLP surrogate scoring for FEW tokens per layer (the decode step: one new token per sequence,
// Method, "KVzap" and the caption of Algorithm 1), where one 128-token tile per layer would leave
// most SMs idle and every byte of W1 has to come from HBM.
//
// n_split * k_split CTAs share one 128-token tile.  The hidden units are cut into n_split slices of
// Ns = hidden / n_split; a slice is computed by a cluster of k_split CTAs (1 or 2).  With k_split = 2
// each CTA of the pair runs half of the K range (so an X tile is read by two CTAs per slice and every
// byte of W1 exactly once), and the two partial pre-activation tiles are combined before the GELU:
// each CTA sends the half of its accumulator that its partner owns through distributed shared memory
// (into the partner's pipeline stages, idle by then) and finishes the columns it owns itself: bias,
// GELU, its part of the second layer.  The 8 partial sums per token go to the pair's first CTA
// (distributed shared memory, one cluster barrier).
//
// The slices of a tile meet in global memory: the first CTA of every cluster stores its 128 x 8 partial
// sums and counts itself in; the cluster that arrives last adds the parts in slice order (so the sum
// does not depend on who was last) plus b2 and writes the scores (and, if asked for, the keep bits).
// Clusters are kept this small on purpose: 36 layers x 2 slices x 2 CTAs fill the machine at once,
// whereas clusters of four do not all find four free SMs in one GPC and leave a second wave.
//
// Warp roles as in score_kernel: warp 0 TMA producer, warp 1 MMA issuer / TMEM owner, warps 2..9
// epilogue (TMEM lane quarter = warp % 4; the two warps of a quarter take alternate 16-column chunks).
#pragma once

#include "decode_kernels.cuh"
#include "score_kernel.cuh"

namespace kvzap {

// Decode step fused into the scoring launch (enabled != 0): while the MMAs run, the epilogue warps
// of a cluster do the cache update of the cluster's own lists -- 128 sequences x H heads of one layer,
// a quarter per CTA -- exactly as decode_update_kernel does (the token that leaves the window is
// judged by its buffered score, so nothing here needs the new scores); the cluster's first CTA puts
// the new scores into the score buffer at the very end (the last cluster of the tile to arrive).
// Consecutive steps may overlap in time (the next launch starts as SMs become free): `done[cluster]`
// counts the steps a cluster has completed, and a cluster touches the cache only after all clusters of
// its tile have published the number of the step before.  Which step a CTA is working on it learns on the
// device: it draws a ticket from a counter of its own (tile, slice, rank) before it lets the next launch be
// placed, so the CTAs that serve the same slice in consecutive launches draw consecutive numbers whatever the
// host knows -- a captured CUDA graph of steps can be replayed.
struct DecodeFuse {
    int32_t enabled;
    int32_t *ticket;                // [n_layers * tiles_per_layer][4][2]: steps started, per (slice, rank in the cluster)
    CacheView c;
    const uint4 *K_new, *V_new;     // [n_layers_call][B][H][D] bf16
    float tau;
    int32_t *done;                  // [n_layers * tiles_per_layer][n_split]
    int64_t wait_limit;             // cycles a cluster waits for the step before to be published
};

struct SplitSmemLayout {
    uint32_t stage_bytes, stages_end, w2s, b1s, w1s, part, xpart, bars, total;
};
__host__ __device__ inline SplitSmemLayout split_smem_layout(int ns, int n_stages, int n_split)
{
    SplitSmemLayout L;
    L.stage_bytes = kATileBytes + static_cast<uint32_t>(ns) * kBlockK * 2;
    L.stages_end = L.stage_bytes * n_stages;
    L.w2s = L.stages_end;
    L.b1s = L.w2s + static_cast<uint32_t>(ns) * kMaxHeads * 4;
    L.w1s = L.b1s + static_cast<uint32_t>(ns) * 4;            // first-layer row scales (8-bit inputs)
    L.part = L.w1s + static_cast<uint32_t>(ns) * 4;
    L.xpart = L.part + kTileM * kMaxHeads * 4;
    L.bars = L.xpart + static_cast<uint32_t>(n_split) * kTileM * kMaxHeads * 4;
    L.total = L.bars + 256;
    return L;
}

// p.group_w = p.chunk_n = Ns (the MMA's N); p.n_chunks = 1; p.acc_bufs = 1; p.n_tiles = 128-token tiles
// over all layers of the call; cluster dimension k_split, gridDim.x = n_split * k_split * p.n_tiles.
// A CTA ends up owning Ns / k_split hidden units: xpart and the W2 / b1 slices are sized for those.
// kFp8: hidden states and W1 are E4M3 bytes (K blocks of 128 codes, tcgen05.mma kind::f8f6f4); the scales
// x_scale[token] * w1_scale[hidden unit] multiply the summed pre-activation before the bias.
template <bool kFp8>
__global__ void __maxnreg__(128)
score_split_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                   const ScoreParams p, const int n_split, const int k_split, const DecodeFuse f)
{
    constexpr int kElems = kFp8 ? 2 * kBlockK : kBlockK;         // elements per 128-byte K block
    __shared__ int64_t fuse_dst[256];       // fused decode step: page row of the evicted token (-1 = dropped)
    __shared__ int64_t fuse_ring[256];      //                     ring row of the list's current slot (-1 = no list)
    __shared__ int32_t fuse_step;           //                     number of the step this CTA works on (its ticket)
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t *smem = smem_raw + pad;
    const uint32_t smem_base = raw_addr + pad;
    const int ns = p.chunk_n;
    const int n_ctas = n_split * k_split;
    const SplitSmemLayout L = split_smem_layout(ns, p.n_stages, n_ctas);

    ulonglong2 *w2p = reinterpret_cast<ulonglong2 *>(smem + L.w2s);
    float *w2f = reinterpret_cast<float *>(smem + L.w2s);
    float *b1s = reinterpret_cast<float *>(smem + L.b1s);
    float *w1s = reinterpret_cast<float *>(smem + L.w1s);
    float *part = reinterpret_cast<float *>(smem + L.part);
    float *xpart = reinterpret_cast<float *>(smem + L.xpart);
    const uint32_t bars = smem_base + L.bars;
    const uint32_t bar_full = bars;                      // [kMaxStages] TMA -> MMA
    const uint32_t bar_empty = bars + 8 * kMaxStages;    // [kMaxStages] MMA -> TMA
    const uint32_t bar_tfull = bars + 16 * kMaxStages;   // MMA -> epilogue
    const uint32_t bar_done = bar_tfull + 8;             // abort path only
    const uint32_t bar_pfull = bar_done + 8;             // second warp of a lane quarter -> first
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + L.bars + 16 * kMaxStages + 32);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L.bars + 16 * kMaxStages + 36);
    volatile int *last_flag = reinterpret_cast<volatile int *>(smem + L.bars + 16 * kMaxStages + 40);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();            // 0 .. k_split - 1
    const int kh = static_cast<int>(rank);               // which part of the K range
    const int nh = (static_cast<int>(blockIdx.x) / k_split) % n_split;   // which slice of the hidden units
    const int pos = nh * k_split + kh;                   // this CTA among the n_ctas of its tile
    const int tile = static_cast<int>(blockIdx.x) / n_ctas;
    const int l_rel = tile / p.tiles_per_layer;
    const int m_tile = tile - l_rel * p.tiles_per_layer;
    const int layer = p.layer0 + l_rel;
    if (f.enabled) {
        // the step number, drawn before any thread of this CTA lets the next launch be placed: a CTA of that launch
        // starts only after every CTA of this one has passed the instruction below, hence after this draw
        if (threadIdx.x == 0)
            fuse_step = atomicAdd(f.ticket + ((layer * p.tiles_per_layer + m_tile) * 4 + nh) * 2 + kh, 1);
        __syncthreads();
    }
    griddep_launch_dependents();
    // unless the caller vouches for the producers of its inputs, nothing of them is read before the work
    // ahead in the stream has completed (every thread waits: the loads below are issued by several warps)
    if (p.wait_before_load) griddep_wait();
    const int own_n = ns / k_split;                      // accumulator columns this CTA finishes
    const int own_c0 = kh * own_n;                       // the first of them
    const int j_first = nh * ns + own_c0;                // = first hidden unit of this CTA

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_tfull, 1);
        mbar_init(bar_done, 1);
        mbar_init(bar_pfull, 4);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_x);
        prefetch_tensormap(&tmap_w);
    }
    const int k_blocks = p.d_model / kElems / k_split;   // K blocks of this CTA
    const int kb_first = kh * k_blocks;
    const uint64_t pol_x = l2_policy_evict_last();        // the other CTAs of the cluster read the same X tile
    const uint64_t pol_w = l2_policy_evict_first();       // every W1 byte is read once per step
    const int w_row = layer * p.w_rows + nh * ns;
    const int row0 = m_tile * kTileM;
    const int n_pre = k_blocks < p.n_stages ? k_blocks : p.n_stages;
    if (warp == 0) {
        // The first loads go out before the CTA-wide barrier below (TMEM allocation, the other warps): the
        // stages are empty and their barriers were initialised by this warp's lane 0 just above.
        __syncwarp();
        if (elect_one()) {
            for (int kb = 0; kb < n_pre; ++kb) {
                const uint32_t sa = smem_base + kb * L.stage_bytes;
                mbar_arrive_expect_tx(bar_full + 8 * kb, L.stage_bytes);
                tma_load_3d(sa + kATileBytes, &tmap_w, bar_full + 8 * kb, 0, w_row, kb_first + kb, pol_w);
                tma_load_3d(sa, &tmap_x, bar_full + 8 * kb, (kb_first + kb) * kElems, row0, l_rel, pol_x);
            }
        }
        __syncwarp();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), static_cast<uint32_t>(p.tmem_cols));
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (from the stage after those)
        const bool elected = elect_one();
        uint32_t st = n_pre == p.n_stages ? 0u : static_cast<uint32_t>(n_pre);
        uint32_t st_par = n_pre == p.n_stages ? 0u : 1u;
        uint32_t sa = smem_base + st * L.stage_bytes;
        bool ok = true;
        for (int kb = n_pre; kb < k_blocks; ++kb) {
            if (!__all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * st, st_par, abort_flag))) {
                ok = false;
                break;
            }
            if (elected) {
                mbar_arrive_expect_tx(bar_full + 8 * st, L.stage_bytes);
                tma_load_3d(sa + kATileBytes, &tmap_w, bar_full + 8 * st, 0, w_row, kb_first + kb, pol_w);
                tma_load_3d(sa, &tmap_x, bar_full + 8 * st, (kb_first + kb) * kElems, row0, l_rel, pol_x);
            }
            __syncwarp();
            sa += L.stage_bytes;
            if (++st == static_cast<uint32_t>(p.n_stages)) { st = 0; st_par ^= 1u; sa = smem_base; }
        }
        if (!ok && lane == 0) {
            // abort path: give the copies already in flight a fixed time to land before the CTA exits
            const long long t0 = clock64();
            while (clock64() - t0 < 2000000LL) { }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        const uint32_t idesc = kFp8 ? umma_idesc_e4m3_f32(kTileM, static_cast<uint32_t>(ns))
                                    : umma_idesc_bf16_f32(kTileM, static_cast<uint32_t>(ns));
        const uint64_t desc0 = umma_desc_k_major_sw128(smem_base);
        const uint32_t desc_hi = static_cast<uint32_t>(desc0 >> 32);
        const uint32_t desc_lo0 = static_cast<uint32_t>(desc0);
        const uint32_t stage_units = L.stage_bytes >> 4;
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
                issue_k_block<false, 1, kFp8>(tmem_base, a_lo, a_lo + (kATileBytes >> 4), desc_hi, 0, 0, idesc, kb == 0);
                umma_commit(bar_empty + 8 * st);
            }
            __syncwarp();
            a_lo += stage_units;
            if (++st == static_cast<uint32_t>(p.n_stages)) { st = 0; st_par ^= 1u; a_lo = desc_lo0; }
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

    // ------------------------------------------------------------ epilogue (warps 2..9)
    const bool epi = warp >= 2;
    const int q = warp & 3;                 // TMEM lane quarter
    const int hsel = (warp - 2) >> 2;       // which of the two warps of that quarter
    const int row = q * 32 + lane;
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    bool ok = true;
    if (epi) {
        // this CTA's slice of b1 and W2 (pairs of hidden units, see mlp_columns)
        const int etid = threadIdx.x - 64;
        const float *w2g = p.w2t + (static_cast<int64_t>(layer) * p.n_hidden + j_first) * kMaxHeads;
        const float *b1g = p.b1 + static_cast<int64_t>(layer) * p.n_hidden + j_first;
        for (int i = etid; i < own_n * kMaxHeads; i += 256) {
            const int j = i >> 3, h = i & 7;
            w2f[(((j >> 1) * kMaxHeads + h) << 1) + (j & 1)] = __ldg(w2g + i);
        }
        for (int i = etid; i < own_n; i += 256) b1s[i] = __ldg(b1g + i);
        if constexpr (kFp8)
            for (int i = etid; i < own_n; i += 256) w1s[i] = __ldg(p.w1_scale + static_cast<int64_t>(layer) * p.n_hidden + j_first + i);
        named_barrier_sync(1, 256);
        if (f.enabled) {
            // ---- the cache update of this CTA's lists, under the MMAs
            const CacheView &c = f.c;
            const int cid = layer * p.tiles_per_layer + m_tile;
            if (etid < n_split) {
                const long long t0 = clock64();
                const int32_t expect = fuse_step;
                while (ld_acquire_gpu(f.done + cid * n_split + etid) != expect) {
                    if (clock64() - t0 > f.wait_limit) { *abort_flag = 1; break; }
                }
            }
            named_barrier_sync(1, 256);
            const bool go = *abort_flag == 0;
            const int rows_per_cta = kTileM / n_ctas;
            // one thread per list: which row leaves, where it goes, which slot the new token takes
            {
                const int b_loc = pos * rows_per_cta + etid / kMaxHeads, h = etid % kMaxHeads;
                const int64_t b = static_cast<int64_t>(m_tile) * kTileM + b_loc;
                int64_t dst = -1, ring = -1;
                if (go && etid < rows_per_cta * kMaxHeads && b < c.n_seqs && h < c.n_heads && c.active[b] != 0) {
                    const int64_t li = (b * c.n_layers + layer) * c.n_heads + h;
                    // two round trips to memory instead of four: both counters first, then the score of
                    // the slot's old token and the page the prefix ends in, whether or not it will be needed
                    const int32_t n = __ldcg(c.n_tokens + li);
                    const int32_t idx = __ldcg(c.prefix_len + li);
                    const int slot = n % c.window;
                    ring = li * c.window + slot;
                    const int page_i = idx / c.page_tokens, in_page = idx % c.page_tokens;
                    const bool full = n >= c.window;
                    const float s_old = full ? __ldcg(c.score_ring + ring) : 0.0f;
                    const int32_t page_old =
                        full && in_page != 0 && page_i < c.max_pages ? __ldcg(c.page_table + li * c.max_pages + page_i) : -1;
                    if (full && s_old >= f.tau) {
                        int32_t page = -1;
                        if (page_i >= c.max_pages) {
                            atomicCAS(p.status, 0, 4 /* KVZAP_ERR_OOM_PAGES */);
                        } else if (in_page == 0) {
                            page = cache_take_page(c, p.status);
                            if (page >= 0) c.page_table[li * c.max_pages + page_i] = page;
                        } else {
                            page = page_old;
                        }
                        if (page >= 0) {
                            dst = static_cast<int64_t>(page) * c.page_tokens + in_page;
                            c.prefix_len[li] = idx + 1;
                        }
                    }
                    c.n_tokens[li] = n + 1;
                }
                fuse_dst[etid] = dst;
                fuse_ring[etid] = ring;
            }
            named_barrier_sync(1, 256);
            // rows: 16 lanes per list, kLists lists at a time; a lane loads the (old row, new row) pairs of all
            // of them before it stores any of them, so that their round trips to memory overlap
            {
                constexpr int kLists = 2;
                const int grp = etid >> 4, l16 = etid & 15;
                const int n_lists = rows_per_cta * kMaxHeads;
                for (int j0 = grp; j0 < n_lists; j0 += 16 * kLists) {
                    int64_t ring[kLists], dst[kLists], src[kLists];
#pragma unroll
                    for (int i = 0; i < kLists; ++i) {
                        const int j = j0 + 16 * i;
                        ring[i] = j < n_lists ? fuse_ring[j] : -1;
                        dst[i] = j < n_lists ? fuse_dst[j] : -1;
                        const int b_loc = pos * rows_per_cta + j / kMaxHeads, h = j % kMaxHeads;
                        const int64_t b = static_cast<int64_t>(m_tile) * kTileM + b_loc;
                        src[i] = ((static_cast<int64_t>(l_rel) * c.n_seqs + b) * c.n_heads + h) * c.row_units;
                        ring[i] *= c.row_units;           // stays negative where there is no list
                        dst[i] *= c.row_units;
                    }
                    for (int u = l16; u < c.row_units; u += 16) {
                        uint4 ko[kLists], vo[kLists], kn[kLists], vn[kLists];
#pragma unroll
                        for (int i = 0; i < kLists; ++i) {
                            if (ring[i] >= 0 && dst[i] >= 0) {
                                ko[i] = __ldcg(c.k_ring + ring[i] + u);
                                vo[i] = __ldcg(c.v_ring + ring[i] + u);
                            }
                            if (ring[i] >= 0) {
                                kn[i] = __ldg(f.K_new + src[i] + u);
                                vn[i] = __ldg(f.V_new + src[i] + u);
                            }
                        }
#pragma unroll
                        for (int i = 0; i < kLists; ++i) {
                            if (ring[i] >= 0 && dst[i] >= 0) {
                                c.k_pool[dst[i] + u] = ko[i];
                                c.v_pool[dst[i] + u] = vo[i];
                            }
                            if (ring[i] >= 0) {
                                c.k_ring[ring[i] + u] = kn[i];
                                c.v_ring[ring[i] + u] = vn[i];
                            }
                        }
                    }
                }
            }
        }
        ok = mbar_wait(bar_tfull, 0, abort_flag);
        tc_fence_after_sync();
    }
    const int n16 = own_n >> 4;             // 16-column chunks this CTA owns (and as many it sends away)
    float4 *recv = reinterpret_cast<float4 *>(smem);          // [own_n / 4][128 rows] float4, over the idle stages
    if (k_split == 2) {
        // every CTA's MMAs are complete once all have passed this barrier: the stages may be overwritten
        tc_fence_before_sync();
        cluster_sync_all();
        if (epi && ok) {
            const uint32_t partner = rank ^ 1u;
            const int send_c0 = (1 - kh) * own_n;               // the columns the partner owns
            const uint32_t dst0 = map_to_cta(smem_base, partner);
            for (int c = hsel; c < n16; c += 2) {
                uint32_t r[16];
                tmem_ld_x16(t_row + send_c0 + c * 16, r);
                tmem_wait_ld();
                reg_fence16(r);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    st_shared_cluster_v4(dst0 + (static_cast<uint32_t>(c * 4 + i) * kTileM + row) * 16,
                                         __uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                         __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
            }
        }
        cluster_sync_all();                                     // the partner's half has arrived
    }
    if (epi) {
        uint64_t acc[kMaxHeads];
#pragma unroll
        for (int h = 0; h < kMaxHeads; ++h) acc[h] = 0ull;
        if (ok) {
            // the first warp of a lane quarter takes the 16-column chunks 0, 2, 4, ..., the second the odd ones
            uint32_t ra[16], rb[16];
            uint64_t sx2 = 0ull;                                   // 8-bit inputs: this row's token scale, twice
            if constexpr (kFp8) {
                float sx = 1.0f;
                if (p.x_scale != nullptr && row0 + row < p.n_tokens)
                    sx = __ldg(p.x_scale + static_cast<int64_t>(l_rel) * p.n_tokens + row0 + row);
                sx2 = f2_pack(sx, sx);
            }
            int c = hsel;
            if (c < n16) tmem_ld_x16(t_row + own_c0 + c * 16, ra);
            while (c < n16) {
                tmem_wait_ld();
                reg_fence16(ra);
                if (c + 2 < n16) tmem_ld_x16(t_row + own_c0 + (c + 2) * 16, rb);
                if (k_split == 2) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float4 o = recv[(c * 4 + i) * kTileM + row];
                        ra[4 * i] = __float_as_uint(__uint_as_float(ra[4 * i]) + o.x);
                        ra[4 * i + 1] = __float_as_uint(__uint_as_float(ra[4 * i + 1]) + o.y);
                        ra[4 * i + 2] = __float_as_uint(__uint_as_float(ra[4 * i + 2]) + o.z);
                        ra[4 * i + 3] = __float_as_uint(__uint_as_float(ra[4 * i + 3]) + o.w);
                    }
                }
                if constexpr (kFp8) mlp_columns_scaled<16>(ra, c * 16, b1s, w1s, sx2, w2p, acc);
                else mlp_columns<16>(ra, c * 16, b1s, w2p, acc);
                c += 2;
                if (c < n16) {
                    tmem_wait_ld();
                    reg_fence16(rb);
                    if (c + 2 < n16) tmem_ld_x16(t_row + own_c0 + (c + 2) * 16, ra);
                    if (k_split == 2) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float4 o = recv[(c * 4 + i) * kTileM + row];
                            rb[4 * i] = __float_as_uint(__uint_as_float(rb[4 * i]) + o.x);
                            rb[4 * i + 1] = __float_as_uint(__uint_as_float(rb[4 * i + 1]) + o.y);
                            rb[4 * i + 2] = __float_as_uint(__uint_as_float(rb[4 * i + 2]) + o.z);
                            rb[4 * i + 3] = __float_as_uint(__uint_as_float(rb[4 * i + 3]) + o.w);
                        }
                    }
                    if constexpr (kFp8) mlp_columns_scaled<16>(rb, c * 16, b1s, w1s, sx2, w2p, acc);
                    else mlp_columns<16>(rb, c * 16, b1s, w2p, acc);
                    c += 2;
                }
            }
        }
        float s[kMaxHeads];
#pragma unroll
        for (int h = 0; h < kMaxHeads; ++h) {
            float lo, hi;
            f2_unpack(acc[h], lo, hi);
            s[h] = lo + hi;
        }
        if (hsel == 1) {
            float4 *dst = reinterpret_cast<float4 *>(part + row * kMaxHeads);
            dst[0] = make_float4(s[0], s[1], s[2], s[3]);
            dst[1] = make_float4(s[4], s[5], s[6], s[7]);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_pfull);
        } else {
            mbar_wait(bar_pfull, 0, abort_flag);
            const float4 *src = reinterpret_cast<const float4 *>(part + row * kMaxHeads);
            const float4 pa = src[0], pb = src[1];
            s[0] += pa.x; s[1] += pa.y; s[2] += pa.z; s[3] += pa.w;
            s[4] += pb.x; s[5] += pb.y; s[6] += pb.z; s[7] += pb.w;
            // hand this CTA's partial sums to its cluster's first CTA: xpart[rank][row][8]
            const uint32_t dst = map_to_cta(smem_base + L.xpart + (rank * kTileM + row) * kMaxHeads * 4, 0);
            st_shared_cluster_v4(dst, s[0], s[1], s[2], s[3]);
            st_shared_cluster_v4(dst + 16, s[4], s[5], s[6], s[7]);
        }
    }

    tc_fence_before_sync();
    // every thread of every CTA of the cluster arrives here (all waits above are bounded); after it the
    // partial sums of all CTAs are visible in the first CTA's shared memory
    cluster_sync_all();
    if (threadIdx.x == 0 && *abort_flag) atomicCAS(p.status, 0, 5 /* KVZAP_ERR_TIMEOUT */);
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, static_cast<uint32_t>(p.tmem_cols));
    }
    // If this launch was allowed to start before the kernel ahead of it had finished (consecutive decode
    // steps), it still completes after it: every thread waits here.
    griddep_wait();
    if (rank != 0 || warp < 2 || warp >= 6 || m_tile >= p.blocks_per_layer) return;

    // ------------------------------------------------------------ first CTA of the cluster: the slice's sums
    {
        float s[kMaxHeads];
#pragma unroll
        for (int h = 0; h < kMaxHeads; ++h) s[h] = 0.0f;
        for (int r = 0; r < k_split; ++r) {
            const float4 *src = reinterpret_cast<const float4 *>(xpart + (r * kTileM + row) * kMaxHeads);
            const float4 pa = src[0], pb = src[1];
            s[0] += pa.x; s[1] += pa.y; s[2] += pa.z; s[3] += pa.w;
            s[4] += pb.x; s[5] += pb.y; s[6] += pb.z; s[7] += pb.w;
        }
        const int32_t done_i = (layer * p.tiles_per_layer + m_tile) * n_split + nh;
        if (n_split > 1) {
            // the slices meet in global memory; whoever arrives last finishes the tile
            float4 *mine = reinterpret_cast<float4 *>(p.split_part + ((static_cast<int64_t>(tile) * n_split + nh) * kTileM + row) * kMaxHeads);
            __stcg(mine, make_float4(s[0], s[1], s[2], s[3]));
            __stcg(mine + 1, make_float4(s[4], s[5], s[6], s[7]));
            __threadfence();
            named_barrier_sync(2, 128);
            if (threadIdx.x == 64) {
                const uint32_t before = atomicAdd(p.split_arrive + tile, 1u);
                *last_flag = (before + 1u) % static_cast<uint32_t>(n_split) == 0u ? 1 : 0;
                __threadfence();
            }
            named_barrier_sync(2, 128);
            if (*last_flag == 0) {
                // not the last: this cluster's part of the cache update is complete, say so and leave
                if (f.enabled && threadIdx.x == 64 && *abort_flag == 0) st_release_gpu(f.done + done_i, fuse_step + 1);
                return;
            }
#pragma unroll
            for (int h = 0; h < kMaxHeads; ++h) s[h] = 0.0f;
            for (int r = 0; r < n_split; ++r) {
                const float4 *src = reinterpret_cast<const float4 *>(p.split_part + ((static_cast<int64_t>(tile) * n_split + r) * kTileM + row) * kMaxHeads);
                const float4 pa = __ldcg(src), pb = __ldcg(src + 1);
                s[0] += pa.x; s[1] += pa.y; s[2] += pa.z; s[3] += pa.w;
                s[4] += pb.x; s[5] += pb.y; s[6] += pb.z; s[7] += pb.w;
            }
        }
#pragma unroll
        for (int h = 0; h < kMaxHeads; ++h) s[h] += __ldg(p.b2 + layer * kMaxHeads + h);
        const int64_t t = static_cast<int64_t>(m_tile) * kTileM + row;
        const bool valid = t < p.n_tokens;
        if (f.enabled) {
            // the new token's scores go into the slot it took (n_tokens was advanced by the list's CTA)
            const CacheView &c = f.c;
            if (valid && *abort_flag == 0) {
#pragma unroll
                for (int h = 0; h < kMaxHeads; ++h) {
                    if (h < c.n_heads && c.active[t] != 0) {
                        const int64_t li = (t * c.n_layers + layer) * c.n_heads + h;
                        const int slot = (__ldcg(c.n_tokens + li) - 1) % c.window;
                        c.score_ring[li * c.window + slot] = s[h];
                    }
                }
            }
            __threadfence();
            named_barrier_sync(2, 128);
            if (threadIdx.x == 64 && *abort_flag == 0) st_release_gpu(f.done + done_i, fuse_step + 1);
        }
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

}  // namespace kvzap
