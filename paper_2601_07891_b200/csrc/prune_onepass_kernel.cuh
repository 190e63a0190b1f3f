// Algorithm 1 after the scoring step in ONE launch: threshold and window test, per-(sequence, head)
// counts and prefix sums, ordered K/V gather (dense-ragged or paged).  This is the kernel behind
// kvzap_prune_prefill, kvzap_prune_prefill_paged and kvzap_prune_prefill_topk, where the scores are
// given and no scoring kernel runs beside the compaction.
//
// A CTA owns a run of consecutive 128-token blocks and a group of heads (all eight, or four, two, one: see the
// kernel), so a score is read by at most eight CTAs (out of L2 after the first).
//   A. keep bits of its blocks (one warp per 32 tokens, ballot words as everywhere else), kept in shared
//      memory; the CTA's kept count per head is published as eight 64-bit words, each carrying the call's
//      number in its upper half, so a reader knows a word is this call's without any flag or fence and
//      nothing has to be cleared between calls.
//   B. rows kept before the CTA's first token = sum of the counts of all CTAs before it (one poll loop
//      per earlier CTA, all in parallel).  When the sequence in progress at the CTA's first token began
//      inside an earlier CTA's run of blocks, the rows that CTA kept before that start are recounted from
//      the scores (no CTA reads another's mask).  Paged output needs the lengths of ALL lists before any
//      row can be placed: every CTA adds its counts to the lists' lengths (atomics), the CTA that arrives
//      last assigns the pages and publishes a flag that all wait for; the page table is filled by all.
//   C. four blocks at a time: rank of every kept (token, head) by popc and its source and destination as
//      byte offsets, listed in shared memory; then one loop moves whole rows with 16-byte accesses, 16
//      lanes per row, two register sets per lane group so that loads are in flight while the rows before
//      them are stored.
// The grid never exceeds half the CTAs the device holds at once: a CTA that waits for another waits for
// one that is running or about to, and the next call's kernel finds room to do its steps A and B while
// this one moves rows.  Every wait is bounded all the same (status word, KVZAP_ERR_TIMEOUT, nothing
// written).  The scratch of consecutive calls rotates (the host explains the overlap rules).
#pragma once

#include "prune_kernels.cuh"

namespace kvzap {

constexpr int kOpThreads = 256;
constexpr int kOpSmemWords = 256;      // (block, head) pairs of a CTA whose mask words stay in shared memory
// (block, head) pairs whose kept rows are listed together before they are moved (8, 16 or 32).  The list is all the
// shared memory the kernel needs, and the smaller it is the more L1 is left for rows in flight: measured at 128k
// tokens, paged output, a third of the rows kept: 72.5 us per call with 32 pairs, 69.2 with 16, 66.3 with 8.
constexpr int kOpPairs = 8;
constexpr int kOpRing = 16;            // scratch sets used in rotation by consecutive calls
constexpr int kOpRows = 4;             // rows of K and of V per register set of a 16-lane group (two sets in rotation)
// dynamic shared memory: the list of kept rows of kOpPairs (block, head) pairs, rounded up to whole rounds of the move loop
constexpr int kOpFlight = 8;             // rows in flight per 16-lane group of the row mover (asynchronous copies)
constexpr uint32_t kOpListBytes = (kOpPairs * 128 + (kOpThreads / 16) * kOpRows) * 16;
constexpr uint32_t kOpFlightBytes = (kOpThreads / 16) * kOpFlight * 512;   // a slot: 256 bytes of K, 256 of V
constexpr uint32_t kOpDynSmem = kOpListBytes + kOpFlightBytes;

struct PruneParams {
    const float *scores;       // [n_tokens][n_heads]
    const float *tau_list;     // per-list thresholds [n_seqs][n_heads] (fixed-budget selection) or nullptr
    float tau;
    int32_t window;
    int64_t n_tokens, n_blocks, n_words;
    int32_t n_heads, n_seqs;
    const int32_t *cu_seqlens;
    int32_t blocks_per_cta;
    int32_t heads_per_cta;     // 8, 4, 2 or 1
    const uint4 *K, *V;
    uint4 *K_out, *V_out;      // dense-ragged outputs [H][n_tokens][D], or the page pools
    int64_t in_stride_h, in_stride_t;
    int32_t row_units;
    int32_t *lengths;
    int32_t *slot_out;         // write plan [n_tokens][n_heads]: when given, no row is moved; every (token, head) gets its
                               // destination row (inside its list, or the pool row when paged), -1 when dropped
    // paged output (page_tokens > 0)
    int32_t page_tokens, first_page, max_pages;
    int64_t n_pages_pool;
    int32_t *list_page0, *page_table, *n_pages_used;
    int32_t *status;
    // scratch of this call (one of kOpRing sets)
    uint32_t *maskbits;        // [n_heads][n_words]: only the words of a CTA's blocks beyond those shared memory holds go here
    uint64_t *cta_counts;      // [grid][8]: (call number << 32) | rows of head h kept in the CTA's blocks
    int32_t *len_acc;          // paged: [n_seqs * n_heads] list lengths being summed; zero between calls
    uint32_t *arrive;          // paged: CTAs that have added their counts, back to 0 when the last one has
    int32_t *scan_flag;        // paged: the call's number once the page assignment is there
    int32_t epoch;             // the call's number, never 0
    int64_t wait_limit;
    int32_t wait_first;        // 1: wait for the work ahead in the stream before the first load
};

// Spins until *flag == want (acquire); false when the cycle budget runs out.
__device__ __forceinline__ bool wait_flag(const int32_t *flag, int32_t want, int64_t limit)
{
    if (ld_acquire_gpu(flag) == want) return true;
    const long long t0 = clock64();
    while (ld_acquire_gpu(flag) != want)
        if (clock64() - t0 > limit) return false;
    return true;
}

// two 64-bit words in one access; each word by itself is read whole
__device__ __forceinline__ ulonglong2 ld_relaxed_gpu_v2(const uint64_t *p)
{
    ulonglong2 v;
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_gpu_u64(uint64_t *p, uint64_t v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__device__ __forceinline__ int popc4(const uint4 &w) { return __popc(w.x) + __popc(w.y) + __popc(w.z) + __popc(w.w); }

// One token's scores and where it stands in its sequence (lane = token of a 32-token word).
struct TokenScores {
    float s[kMaxHeads];
    int b;                 // the token's sequence, -1 past the end of the input
    bool in_window;
};
__device__ __forceinline__ void load_token(const PruneParams &p, int64_t word, int lane, bool multi, TokenScores &ts)
{
    const int H = p.n_heads;
    const int64_t t = word * 32 + lane;
#pragma unroll
    for (int h = 0; h < kMaxHeads; ++h) ts.s[h] = 0.0f;
    ts.b = -1;
    ts.in_window = false;
    if (t >= p.n_tokens) return;
    const float *src = p.scores + t * H;
    if (H == kMaxHeads) {
        const float4 a = __ldcg(reinterpret_cast<const float4 *>(src));
        const float4 bb = __ldcg(reinterpret_cast<const float4 *>(src) + 1);
        ts.s[0] = a.x; ts.s[1] = a.y; ts.s[2] = a.z; ts.s[3] = a.w;
        ts.s[4] = bb.x; ts.s[5] = bb.y; ts.s[6] = bb.z; ts.s[7] = bb.w;
    } else {
#pragma unroll
        for (int h = 0; h < kMaxHeads; ++h)
            if (h < H) ts.s[h] = __ldcg(src + h);
    }
    int64_t seq_end = p.n_tokens;
    ts.b = 0;
    if (multi) {
        ts.b = seq_of_token(p.cu_seqlens, p.n_seqs, t);
        seq_end = __ldg(p.cu_seqlens + ts.b + 1);
    }
    ts.in_window = t >= seq_end - static_cast<int64_t>(p.window);
}
// Keep bits of the word's 32 tokens (whole warp): lane h returns head h's word.
__device__ __forceinline__ uint32_t keep_word(const PruneParams &p, const TokenScores &ts, int lane)
{
    const int H = p.n_heads;
    const bool valid = ts.b >= 0;
    float tau_h[kMaxHeads];
#pragma unroll
    for (int h = 0; h < kMaxHeads; ++h) tau_h[h] = p.tau;
    if (p.tau_list != nullptr && valid) {
#pragma unroll
        for (int h = 0; h < kMaxHeads; ++h)
            if (h < H) tau_h[h] = __ldcg(p.tau_list + ts.b * H + h);
    }
    uint32_t my_word = 0;
#pragma unroll
    for (int h = 0; h < kMaxHeads; ++h) {
        const bool keep = valid && (ts.in_window || ts.s[h] >= tau_h[h]);
        const uint32_t w = __ballot_sync(0xffffffffu, keep);
        if (lane == h) my_word = w;
    }
    return my_word;
}

// grid (chunks, head groups): CTA (c, g) owns blocks [c * blocks_per_cta, ...) of heads [g * HG, (g + 1) * HG),
// HG = p.heads_per_cta in {8, 4, 2, 1}.  Fewer heads per CTA mean more blocks per CTA for the same grid, so the
// one CTA that holds a sequence's window (all of whose rows are kept) has little more to move than the others.
// Two CTAs per SM (128 registers each): three or four, with fewer rows in flight per thread, moved rows more slowly
// in every case measured (4.4 against 5.6 TB/s at 128k tokens).
template <int kRows>
__global__ void __launch_bounds__(kOpThreads, 2)
prune_onepass_kernel(const PruneParams p)
{
    __shared__ uint4 words_s[kOpSmemWords];             // mask words of the CTA's first blocks: [block][head of the group]
    __shared__ int32_t cnt_s[kMaxHeads];
    __shared__ int32_t red_s[kOpThreads / 32][2 * kMaxHeads];
    __shared__ int32_t part_s[kMaxHeads];
    __shared__ int32_t run_s[kMaxHeads], base_s[kMaxHeads], p0_s[kMaxHeads];
    // kept (token, head) pairs of the blocks in work: byte offsets of the source row and of the destination row
    // (-1: nowhere) inside K / V and the outputs; room for a whole number of rounds of the move loop
    extern __shared__ longlong2 ent_s[];
    __shared__ uint4 wsb_s[kOpPairs];                   // [block of the group in work][head of the group]
    __shared__ int32_t runb_s[kOpPairs + kMaxHeads];    // rows of that head kept before that block; last row: after all of them
    __shared__ int32_t off_s[kOpPairs + 1];
    __shared__ int flag_s;

    griddep_launch_dependents();
    if (p.wait_first) griddep_wait();

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int H = p.n_heads;
    const int HG = p.heads_per_cta;
    const int c = static_cast<int>(blockIdx.x), g = static_cast<int>(blockIdx.y);
    const int h0 = g * HG;
    auto own = [&](int h) -> bool { return h >= h0 && h < h0 + HG && h < H; };
    const int64_t blk0 = static_cast<int64_t>(c) * p.blocks_per_cta;
    const int64_t blk1 = blk0 + p.blocks_per_cta < p.n_blocks ? blk0 + p.blocks_per_cta : p.n_blocks;
    const bool multi = p.cu_seqlens != nullptr && p.n_seqs > 1;
    const bool paged = p.page_tokens > 0;
    const uint64_t tag = static_cast<uint64_t>(static_cast<uint32_t>(p.epoch)) << 32;
    const int smem_blocks = kOpSmemWords / HG;            // blocks whose words stay in shared memory

    if (tid < kMaxHeads) { cnt_s[tid] = 0; part_s[tid] = 0; }
    if (tid == 0) flag_s = 0;
    // the sequences at the CTA's first and last token, and where the first one starts
    const int64_t t0 = blk0 * kBlockTokens;
    const int64_t t_last = (blk1 * kBlockTokens < p.n_tokens ? blk1 * kBlockTokens : p.n_tokens) - 1;
    int b_lo = 0, b_hi = 0;
    int64_t s0 = 0;
    if (multi) {
        b_lo = seq_of_token(p.cu_seqlens, p.n_seqs, t0);
        b_hi = seq_of_token(p.cu_seqlens, p.n_seqs, t_last);
        s0 = p.cu_seqlens[b_lo];
    }
    const int j0 = static_cast<int>((s0 / kBlockTokens) / p.blocks_per_cta);      // the CTA (column) whose blocks hold s0
    __syncthreads();

    // ---------------------------------------------------------------- A: keep bits and counts of the CTA's blocks
    {
        int32_t my_cnt = 0;                                   // lane h: kept rows of head h in the words this warp made
        const int n_w = static_cast<int>(blk1 - blk0) * 4;    // 32-token words of this CTA
        constexpr int kUnroll = 4;                            // words whose scores are in flight together
        for (int w0 = warp; w0 < n_w; w0 += (kOpThreads / 32) * kUnroll) {
            TokenScores ts[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int wl = w0 + u * (kOpThreads / 32);
                if (wl < n_w) load_token(p, blk0 * 4 + wl, lane, multi, ts[u]);
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int wl = w0 + u * (kOpThreads / 32);
                if (wl >= n_w) break;
                const uint32_t my_word = keep_word(p, ts[u], lane);
                const int bl = wl >> 2, q = wl & 3;
                if (own(lane)) {
                    if (bl < smem_blocks) reinterpret_cast<uint32_t *>(&words_s[bl * HG + lane - h0])[q] = my_word;
                    else p.maskbits[static_cast<int64_t>(lane) * p.n_words + blk0 * 4 + wl] = my_word;
                    my_cnt += __popc(my_word);
                }
                if (paged && b_lo != b_hi) {
                    // the CTA's blocks touch several sequences: the lists' lengths are summed word by word, the lanes
                    // of one sequence together
                    const uint32_t same = __match_any_sync(0xffffffffu, ts[u].b);
                    const bool leader = ts[u].b >= 0 && (__ffs(same) - 1) == lane;
#pragma unroll
                    for (int h = 0; h < kMaxHeads; ++h) {
                        const uint32_t wh = __shfl_sync(0xffffffffu, my_word, h);
                        if (leader && own(h) && (wh & same)) atomicAdd(p.len_acc + ts[u].b * H + h, __popc(wh & same));
                    }
                }
            }
        }
        if (own(lane) && my_cnt) atomicAdd(&cnt_s[lane], my_cnt);
        // The sequence in progress at this CTA's first token began inside CTA j0's blocks: the rows CTA j0 kept
        // from that start to the end of its blocks are recounted here (all of them belong to that sequence).
        if (multi && j0 < c) {
            const int64_t end = static_cast<int64_t>(j0 + 1) * p.blocks_per_cta * kBlockTokens;
            int32_t extra = 0;
            for (int64_t word = s0 / 32 + warp; word * 32 < end; word += kOpThreads / 32) {
                TokenScores ts;
                load_token(p, word, lane, multi, ts);
                uint32_t w = keep_word(p, ts, lane);
                if (word * 32 < s0) w &= ~0u << static_cast<int>(s0 - word * 32);       // bits of the sequence before
                extra += __popc(w);
            }
            if (own(lane) && extra) atomicAdd(&part_s[lane], extra);
        }
    }
    __syncthreads();
    if (tid < kMaxHeads && own(tid)) st_relaxed_gpu_u64(p.cta_counts + c * kMaxHeads + tid, tag | static_cast<uint32_t>(cnt_s[tid]));
    if (paged) {
        if (b_lo == b_hi && tid < kMaxHeads && own(tid) && cnt_s[tid]) atomicAdd(p.len_acc + b_lo * H + tid, cnt_s[tid]);
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const uint32_t before = atomicAdd(p.arrive, 1u);
            if (before + 1u == gridDim.x * gridDim.y) {
                *p.arrive = 0u;                               // every CTA of this call has arrived; the set is reused much later
                flag_s = 1;
            }
            __threadfence();
        }
        __syncthreads();
    }

    // ---------------------------------------------------------------- paged: the last CTA assigns the pages
    bool ok = true;
    if (paged) {
        if (flag_s != 0) {
            for (int idx = tid; idx < p.n_seqs * H; idx += kOpThreads) {
                p.lengths[idx] = __ldcg(p.len_acc + idx);
                p.len_acc[idx] = 0;
            }
            __syncthreads();
            assign_pages<kOpThreads>(H, p.n_seqs, p.lengths, p.page_tokens, p.first_page, p.n_pages_pool, p.max_pages,
                                     p.list_page0, p.page_table, p.n_pages_used, nullptr, p.status, 0, nullptr, nullptr,
                                     nullptr, 0);
            __threadfence();
            __syncthreads();
            if (tid == 0) st_release_gpu(p.scan_flag, p.epoch);
        }
        if (tid == 0 && !wait_flag(p.scan_flag, p.epoch, p.wait_limit)) flag_s = -1;
        __syncthreads();
        ok = flag_s >= 0;
        if (ok && tid < H) p0_s[tid] = __ldcg(p.list_page0 + b_lo * H + tid);      // first pages of the lists of the first sequence
        if (ok && __ldcg(p.list_page0) >= 0) {
            // the page table, spread over all CTAs: the n-th page assigned by this call belongs to the last list
            // whose first page is not beyond it (list_page0 is the exclusive scan of the lists' page counts)
            const int32_t used = __ldcg(p.n_pages_used);
            const int n_lists = p.n_seqs * H;
            const int64_t n_ctas = static_cast<int64_t>(gridDim.x) * gridDim.y;
            for (int64_t n = (static_cast<int64_t>(g) * gridDim.x + c) * kOpThreads + tid; n < used; n += n_ctas * kOpThreads) {
                int lo = 0, hi = n_lists;                  // invariant: page0[lo] - first_page <= n, lo < hi
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (__ldcg(p.list_page0 + mid) - p.first_page <= n) lo = mid; else hi = mid;
                }
                const int64_t i = n - (__ldcg(p.list_page0 + lo) - p.first_page);
                p.page_table[static_cast<int64_t>(lo) * p.max_pages + i] = p.first_page + static_cast<int32_t>(n);
            }
        }
    }

    // ---------------------------------------------------------------- B: rows kept before this CTA's first token
    // run_s[h]: kept rows of head h before the current block; base_s[h]: before the start of the sequence that
    // is in progress at the current block's first token
    {
        int32_t acc[2 * kMaxHeads];
#pragma unroll
        for (int i = 0; i < 2 * kMaxHeads; ++i) acc[i] = 0;
        for (int j = tid; j < c && ok; j += kOpThreads) {
            const uint64_t *e = p.cta_counts + static_cast<int64_t>(j) * kMaxHeads;
            uint64_t v[kMaxHeads];
            const long long t_begin = clock64();
            for (;;) {
                bool all = true;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const ulonglong2 x = ld_relaxed_gpu_v2(e + 2 * i);
                    v[2 * i] = x.x;
                    v[2 * i + 1] = x.y;
                }
#pragma unroll
                for (int h = 0; h < kMaxHeads; ++h)
                    if (own(h) && (v[h] >> 32) != (tag >> 32)) all = false;
                if (all) break;
                if (clock64() - t_begin > p.wait_limit) { flag_s = -1; break; }
            }
#pragma unroll
            for (int h = 0; h < kMaxHeads; ++h) {
                const int32_t a = static_cast<int32_t>(static_cast<uint32_t>(v[h]));
                acc[h] += a;
                if (j > j0) acc[kMaxHeads + h] += a;
            }
        }
#pragma unroll
        for (int i = 0; i < 2 * kMaxHeads; ++i) acc[i] = __reduce_add_sync(0xffffffffu, acc[i]);
        if (lane == 0) {
#pragma unroll
            for (int i = 0; i < 2 * kMaxHeads; ++i) red_s[warp][i] = acc[i];
        }
        __syncthreads();
        ok = ok && flag_s >= 0;
        if (tid < kMaxHeads) {
            int32_t r = 0, after = 0;
#pragma unroll
            for (int wv = 0; wv < kOpThreads / 32; ++wv) { r += red_s[wv][tid]; after += red_s[wv][kMaxHeads + tid]; }
            run_s[tid] = r;
            // rows kept before s0 = everything before this CTA, less what lies between s0 and this CTA: the CTAs
            // after j0 in full and CTA j0 from s0 on
            base_s[tid] = !multi ? 0 : (j0 < c ? r - after - part_s[tid] : r);
        }
    }
    if (!ok) {
        if (tid == 0) atomicCAS(p.status, 0, 5 /* KVZAP_ERR_TIMEOUT */);
        griddep_wait();
        return;
    }
    if (c == 0 && p.cu_seqlens != nullptr && !paged)          // empty sequences have no last token to write for them
        for (int i = tid; i < p.n_seqs * H; i += kOpThreads)
            if (own(i % H) && p.cu_seqlens[i / H + 1] == p.cu_seqlens[i / H]) p.lengths[i] = 0;
    __syncthreads();

    // ---------------------------------------------------------------- C: ranks, destinations, row moves
    // kOpPairs (block, head) pairs at a time -- 32 / HG blocks: first the list of all their kept (token, head) pairs,
    // source and destination of each as byte offsets, computed once, in shared memory, ordered by block, head,
    // token; then one long loop that moves the rows.
    const int tok = tid & (kBlockTokens - 1);
    const int half = tid >> 7;                                 // the two threads of a token take alternate (block, head) pairs
    const int group = tid >> 4, gl = tid & 15;
    constexpr int kGroups = kOpThreads / 16;
    constexpr int kStep = kGroups * kRows;
    const int sb_blocks = kOpPairs / HG;
    const int64_t row_bytes = static_cast<int64_t>(p.row_units) * 16;
    const char *Kb = reinterpret_cast<const char *>(p.K), *Vb = reinterpret_cast<const char *>(p.V);
    char *Ko = reinterpret_cast<char *>(p.K_out), *Vo = reinterpret_cast<char *>(p.V_out);
    for (int64_t sb0 = blk0; sb0 < blk1; sb0 += sb_blocks) {
        const int nb = static_cast<int>(blk1 - sb0 < sb_blocks ? blk1 - sb0 : sb_blocks);
        const int64_t sb_start = sb0 * kBlockTokens;
        if (tid < 32) {                                         // one warp; lanes beyond the pairs count nothing
            const int bl = tid / HG, hh = tid % HG, h = h0 + hh;
            uint4 w = make_uint4(0u, 0u, 0u, 0u);
            if (tid < kOpPairs && bl < nb && h < H)
                w = sb0 - blk0 + bl < smem_blocks
                        ? words_s[(sb0 - blk0 + bl) * HG + hh]
                        : __ldcg(reinterpret_cast<const uint4 *>(p.maskbits + static_cast<int64_t>(h) * p.n_words + (sb0 + bl) * 4));
            if (tid < kOpPairs) wsb_s[tid] = w;
            // exclusive offsets of the pairs in the list (one warp), and the rows of the pair's head kept before its block
            const int cnt = popc4(w);
            int incl = cnt, incl_h = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += y;
            }
            for (int o = HG; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, incl_h, o);
                if (lane >= o) incl_h += y;
            }
            if (tid < kOpPairs) {
                off_s[tid] = incl - cnt;
                runb_s[tid] = run_s[h] + incl_h - cnt;
                if (bl == sb_blocks - 1) runb_s[kOpPairs + hh] = run_s[h] + incl_h;
            }
            if (tid == 31) off_s[kOpPairs] = incl;
        }
        __syncthreads();
        // rows of head h0 + hh kept before position x of this group of blocks (sb_start <= x <= its end)
        auto kept_before_local = [&](int hh, int64_t x) -> int32_t {
            const int xb = static_cast<int>((x - sb_start) / kBlockTokens);
            if (xb >= sb_blocks) return runb_s[kOpPairs + hh];
            const uint4 w = wsb_s[xb * HG + hh];
            return runb_s[xb * HG + hh] + popc_below(w.x, w.y, w.z, w.w, static_cast<int>((x - sb_start) % kBlockTokens));
        };
        const int total = off_s[kOpPairs];
        const int padded = (total + kStep - 1) / kStep * kStep;
        for (int i = total + tid; i < padded; i += kOpThreads) ent_s[i] = make_longlong2(0, -1);    // harmless load, no store
        int bl_seq = -1, b = 0;
        int64_t s = 0, e = p.n_tokens;
        for (int pi = half; pi < kOpPairs; pi += 2) {
            const int bl = pi / HG, hh = pi % HG, h = h0 + hh;
            if (bl >= nb || h >= H) continue;
            const int64_t t = sb_start + bl * kBlockTokens + tok;
            if (t >= p.n_tokens) continue;
            if (multi && bl != bl_seq) {
                b = seq_of_token(p.cu_seqlens, p.n_seqs, t);
                s = p.cu_seqlens[b];
                e = p.cu_seqlens[b + 1];
                bl_seq = bl;
            }
            const uint4 w = wsb_s[pi];
            const uint32_t wq = tok < 32 ? w.x : tok < 64 ? w.y : tok < 96 ? w.z : w.w;
            const bool keep = (wq >> (tok & 31)) & 1u;
            const bool last = t + 1 == e && !paged;
            if (!keep && !last) {
                if (p.slot_out != nullptr) p.slot_out[t * H + h] = -1;
                continue;
            }
            const int r = popc_below(w.x, w.y, w.z, w.w, tok);
            int32_t n = runb_s[pi] + r;                       // rank inside list (b,h)
            if (multi) n -= s >= sb_start ? kept_before_local(hh, s) : base_s[h];
            if (keep) {
                int64_t dst;                                    // destination row
                if (paged) {
                    const int32_t p0 = b == b_lo ? p0_s[h] : __ldcg(p.list_page0 + b * H + h);
                    dst = p0 < 0 ? -1 : static_cast<int64_t>(p0) * p.page_tokens + n;
                } else {
                    dst = static_cast<int64_t>(h) * p.n_tokens + s + n;
                }
                if (p.slot_out != nullptr)
                    p.slot_out[t * H + h] = static_cast<int32_t>(paged ? dst : n);
                else
                    ent_s[off_s[pi] + r] =
                        make_longlong2((h * p.in_stride_h + t * p.in_stride_t) * row_bytes, dst < 0 ? -1 : dst * row_bytes);
            } else if (p.slot_out != nullptr) {
                p.slot_out[t * H + h] = -1;
            }
            if (last) p.lengths[b * H + h] = n + (keep ? 1 : 0);
        }
        __syncthreads();
        if (p.slot_out == nullptr && p.row_units <= 16) {
            // Rows of up to 256 bytes: every lane copies its 16 bytes of K and of V asynchronously into the group's
            // ring of kOpFlight slots and stores a row once its copy has landed, so kOpFlight rows per group are on
            // their way at any time and no register holds a row.  A lane reads back only the bytes it copied itself.
            // Exactly kOpFlight copy groups are committed ahead of the row being stored (empty ones at the tail), so
            // the wait is always for all but the newest kOpFlight - 1.
            const bool act = gl < p.row_units;
            const int64_t lane_off = static_cast<int64_t>(gl) * 16;
            char *ring = reinterpret_cast<char *>(ent_s) + kOpListBytes + group * (kOpFlight * 512) + gl * 16;
            const uint32_t ring_a = smem_u32(ring);
            const int n_rows = total > group ? (total - group + kGroups - 1) / kGroups : 0;
            auto issue = [&](int j) {
                if (j < n_rows && act) {
                    const int64_t src = ent_s[group + j * kGroups].x;
                    const uint32_t slot = ring_a + (j % kOpFlight) * 512;
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot), "l"(Kb + src + lane_off) : "memory");
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot + 256u), "l"(Vb + src + lane_off) : "memory");
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
            };
#pragma unroll
            for (int j = 0; j < kOpFlight; ++j) issue(j);
            for (int j = 0; j < n_rows; ++j) {
                asm volatile("cp.async.wait_group %0;" ::"n"(kOpFlight - 1) : "memory");
                const int64_t dst = ent_s[group + j * kGroups].y;
                if (act && dst >= 0) {
                    const char *slot = ring + (j % kOpFlight) * 512;
                    const uint4 kk = *reinterpret_cast<const uint4 *>(slot);
                    const uint4 vv = *reinterpret_cast<const uint4 *>(slot + 256);
                    *reinterpret_cast<uint4 *>(Ko + dst + lane_off) = kk;
                    *reinterpret_cast<uint4 *>(Vo + dst + lane_off) = vv;
                }
                issue(j + kOpFlight);                          // into the slot just read (the stores above needed its data)
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        for (int u0 = gl; u0 < p.row_units && p.slot_out == nullptr && p.row_units > 16; u0 += 16) {
            // longer rows -- two register sets: the loads of one are in flight while the other is stored
            const int64_t lane_off = static_cast<int64_t>(u0) * 16;
            uint4 ka[kRows], va[kRows], kb[kRows], vb[kRows];
            int64_t da[kRows], db[kRows];
            auto load_set = [&](int first, uint4 (&kk)[kRows], uint4 (&vv)[kRows], int64_t (&dd)[kRows]) {
#pragma unroll
                for (int j = 0; j < kRows; ++j) {
                    const longlong2 ent = ent_s[first + j * kGroups];
                    kk[j] = __ldg(reinterpret_cast<const uint4 *>(Kb + ent.x + lane_off));
                    vv[j] = __ldg(reinterpret_cast<const uint4 *>(Vb + ent.x + lane_off));
                    dd[j] = ent.y;
                }
            };
            auto store_set = [&](const uint4 (&kk)[kRows], const uint4 (&vv)[kRows], const int64_t (&dd)[kRows]) {
#pragma unroll
                for (int j = 0; j < kRows; ++j) {
                    if (dd[j] >= 0) {
                        *reinterpret_cast<uint4 *>(Ko + dd[j] + lane_off) = kk[j];
                        *reinterpret_cast<uint4 *>(Vo + dd[j] + lane_off) = vv[j];
                    }
                }
            };
            if (padded > 0) load_set(group, ka, va, da);
            for (int i0 = group; i0 < padded; i0 += 2 * kStep) {
                const bool more = i0 + kStep < padded;
                if (more) load_set(i0 + kStep, kb, vb, db);
                store_set(ka, va, da);
                if (i0 + 2 * kStep < padded) load_set(i0 + 2 * kStep, ka, va, da);
                if (more) store_set(kb, vb, db);
            }
        }
        __syncthreads();
        if (tid < HG && h0 + tid < H) {
            // carried to the next group of blocks: rows kept so far, and rows kept before the start of the
            // sequence that is in progress at its first token
            const int h = h0 + tid;
            const int64_t t_next = sb_start + static_cast<int64_t>(sb_blocks) * kBlockTokens;
            int32_t nbase = 0;
            if (multi && t_next < p.n_tokens) {
                const int64_t s_next = p.cu_seqlens[seq_of_token(p.cu_seqlens, p.n_seqs, t_next)];
                nbase = s_next >= sb_start ? kept_before_local(tid, s_next) : base_s[h];
            }
            run_s[h] = runb_s[kOpPairs + tid];
            base_s[h] = nbase;
        }
        __syncthreads();
    }
    griddep_wait();        // every thread: this kernel completes after the one ahead of it
}

}  // namespace kvzap
