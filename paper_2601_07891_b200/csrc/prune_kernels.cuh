// Threshold/window mask, per-head prefix sums and ordered K/V compaction
// (Algorithm 1: the window, threshold and gather steps).  Everything here is integer / byte work and must
// be bit-exact.
//
// Data flow (all on one stream, no CTA ever waits for another):
//   mask words  [H][n_words]    one keep bit per (head, packed token), 32 tokens per word,
//                               written either by the scoring epilogue or by mask_kernel
//   compact_dense_kernel        the compaction of every entry point that has a context: a CTA owns a
//                               run of 128-token blocks of one head, counts the rows kept before them
//                               straight from the mask words, ranks its kept rows with popc and copies
//                               whole K and V rows with 16-byte accesses to their slot in the (b,h)
//                               list (dense-ragged) or in the list's pages (paged)
//   scan_kernel                 paged output only: lengths[b,h] and the first page of every list
//                               (an exclusive scan over all lists, the one step that needs them all)
//   compact_kernel              the older one-CTA-per-(block, head) compaction behind scan_kernel's
//                               block prefix; still used by the allocation-free entry point
#pragma once

#include "score_kernel.cuh"

namespace kvzap {

constexpr int kBlockTokens = 128;     // tokens per mask block = 4 words (same as the scoring tile)

// ---------------------------------------------------------------------------
// keep[h,t] = in_window(t) || scores[t,h] >= tau, as 32-token ballot words.
// One warp per 32 tokens; 4 warps per CTA = one 128-token block.
// tau_list != nullptr: a threshold per list, tau_list[b * n_heads + h] (fixed-budget selection), instead of tau.
__global__ void __launch_bounds__(128)
mask_kernel(const float *__restrict__ scores, int64_t n_tokens, int n_heads,
            const int32_t *__restrict__ cu_seqlens, int n_seqs, float tau, int window, int window_keep,
            uint32_t *__restrict__ maskbits, int64_t n_words, const float *__restrict__ tau_list)
{
    // may be queued with early start behind the kernels that produce the per-list thresholds
    griddep_launch_dependents();
    griddep_wait();
    const int lane = threadIdx.x & 31;
    const int64_t word = static_cast<int64_t>(blockIdx.x) * 4 + (threadIdx.x >> 5);
    const int64_t t = word * 32 + lane;
    const bool valid = t < n_tokens;
    float s[kMaxHeads], tau_h[kMaxHeads];
#pragma unroll
    for (int h = 0; h < kMaxHeads; ++h) { s[h] = 0.0f; tau_h[h] = tau; }
    bool in_window = false;
    if (valid) {
        const float *src = scores + t * n_heads;
        if (n_heads == kMaxHeads) {
            const float4 a = __ldg(reinterpret_cast<const float4 *>(src));
            const float4 b = __ldg(reinterpret_cast<const float4 *>(src) + 1);
            s[0] = a.x; s[1] = a.y; s[2] = a.z; s[3] = a.w;
            s[4] = b.x; s[5] = b.y; s[6] = b.z; s[7] = b.w;
        } else {
#pragma unroll
            for (int h = 0; h < kMaxHeads; ++h)
                if (h < n_heads) s[h] = __ldg(src + h);
        }
        int64_t seq_end = n_tokens;
        int b = 0;
        if (cu_seqlens != nullptr && n_seqs > 1) {
            b = seq_of_token(cu_seqlens, n_seqs, t);
            seq_end = __ldg(cu_seqlens + b + 1);
        }
        in_window = t >= seq_end - static_cast<int64_t>(window);
        if (tau_list != nullptr) {
            // thresholds written by the kernel ahead in the stream: plain loads
#pragma unroll
            for (int h = 0; h < kMaxHeads; ++h)
                if (h < n_heads) tau_h[h] = __ldcg(tau_list + b * n_heads + h);
        }
    }
    uint32_t my_word = 0;
#pragma unroll
    for (int h = 0; h < kMaxHeads; ++h) {
        const bool keep = valid && (in_window ? window_keep != 0 : s[h] >= tau_h[h]);
        const uint32_t w = __ballot_sync(0xffffffffu, keep);
        if (lane == h) my_word = w;
    }
    if (lane < n_heads) maskbits[static_cast<int64_t>(lane) * n_words + word] = my_word;
}

// Number of kept tokens of head h among packed tokens [0, t), given the block prefix.
__device__ __forceinline__ int32_t kept_before(const uint32_t *__restrict__ maskbits, int64_t n_words,
                                               const int32_t *__restrict__ blockprefix, int64_t n_blocks, int h,
                                               int64_t t)
{
    const int64_t blk = t / kBlockTokens;
    int32_t n = blockprefix[static_cast<int64_t>(h) * (n_blocks + 1) + blk];
    if (blk < n_blocks) {
        const uint32_t *w = maskbits + static_cast<int64_t>(h) * n_words + blk * 4;
        const int r = static_cast<int>(t - blk * kBlockTokens);       // 0..127 bits of this block
        for (int i = 0; i < 4; ++i) {
            const int lo = i * 32;
            if (r >= lo + 32) n += __popc(__ldcg(w + i));
            else if (r > lo) n += __popc(__ldcg(w + i) & ((1u << (r - lo)) - 1u));
        }
    }
    return n;
}

// Where list idx (= b * n_heads + h) of a call lives in the caller's per-list arrays (lengths, page tables): at
// idx itself, or -- appending a batch of prompts to a cache, whose lists are ordered (sequence slot, layer, head) --
// at list_map[b] + h, list_map [n_seqs] naming the list of head 0 of each of the call's sequences.
__device__ __forceinline__ int64_t list_at(const int64_t *__restrict__ list_map, int idx, int n_heads)
{
    return list_map != nullptr ? list_map[idx / n_heads] + idx % n_heads : static_cast<int64_t>(idx);
}

// ---------------------------------------------------------------------------
// Page assignment of the paged output, by all NT threads of one CTA: list idx (= b * n_heads + h) needs
// ceil(lengths[idx] / page_tokens) pages (less those it owns already when appending); list_page0 receives the
// exclusive scan of the needs plus first_page, *n_pages_used the total; a pool or table that is too small
// sets the status word, marks every list with list_page0 = -1 and (append) restores the old lengths.
// fill_table != 0: the page numbers are also entered into page_table here; otherwise the caller does
// that (fill_page_table), e.g. spread over many CTAs.  Arguments as scan_lists.
template <int NT>
__device__ __forceinline__ void
assign_pages(int n_heads, int n_seqs, int32_t *__restrict__ lengths, int page_tokens, int32_t first_page,
             int64_t n_pages_pool, int max_pages, int32_t *__restrict__ list_page0, int32_t *__restrict__ page_table,
             int32_t *__restrict__ n_pages_used, int32_t *__restrict__ page_cursor, int32_t *__restrict__ status, int append,
             int32_t *__restrict__ list_base, const int32_t *__restrict__ free_stack, int32_t *__restrict__ free_top,
             int fill_table, const int64_t *__restrict__ list_map = nullptr)
{
    __shared__ int32_t warp_sums[32];
    __shared__ int32_t carry_s;
    __shared__ int32_t fail_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    auto block_scan = [&](int32_t v, int32_t &total) -> int32_t {   // inclusive scan over the CTA
        int32_t x = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        __syncthreads();
        if (lane == 31) warp_sums[warp] = x;
        __syncthreads();
        if (warp == 0) {
            int32_t w = lane < NT / 32 ? warp_sums[lane] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t y = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += y;
            }
            warp_sums[lane] = w;
        }
        __syncthreads();
        total = warp_sums[31];
        return x + (warp > 0 ? warp_sums[warp - 1] : 0);
    };
    // paged output: exclusive scan of the per-list page counts in (b,h) order
    __syncthreads();
    if (tid == 0) { carry_s = 0; fail_s = 0; }
    __syncthreads();
    const int n_lists = n_heads * n_seqs;
    for (int base = 0; base < n_lists; base += NT) {
        const int idx = base + tid;
        int32_t need = 0;
        if (idx < n_lists) {
            need = (lengths[list_at(list_map, idx, n_heads)] + page_tokens - 1) / page_tokens;
            if (need > max_pages) fail_s = 1;
            if (append) need -= (list_base[idx] + page_tokens - 1) / page_tokens;     // pages the list already owns
        }
        int32_t total;
        const int32_t incl = block_scan(need, total);
        const int32_t carry = carry_s;
        if (idx < n_lists) list_page0[idx] = first_page + carry + incl - need;
        __syncthreads();
        if (tid == 0) carry_s = carry + total;
        __syncthreads();
    }
    const int32_t used = carry_s;
    int32_t n_free = 0;
    if (page_cursor != nullptr && free_top != nullptr) {
        n_free = *free_top;
        if (n_free < 0) n_free = 0;
    }
    const int32_t from_stack = used < n_free ? used : n_free;
    const bool fail = fail_s != 0 || static_cast<int64_t>(first_page) + (used - from_stack) > n_pages_pool;
    if (fail) {
        for (int idx = tid; idx < n_lists; idx += NT) {
            list_page0[idx] = -1;
            if (append) lengths[list_at(list_map, idx, n_heads)] = list_base[idx];
        }
        if (tid == 0) {
            atomicCAS(status, 0, 4 /* KVZAP_ERR_OOM_PAGES */);
            if (n_pages_used != nullptr) *n_pages_used = 0;
        }
        return;
    }
    __syncthreads();      // every thread has read the cursor and the stack height
    if (tid == 0) {
        if (n_pages_used != nullptr) *n_pages_used = used;
        if (page_cursor != nullptr) *page_cursor = first_page + used - from_stack;
        if (from_stack > 0) *free_top = n_free - from_stack;
    }
    __syncthreads();      // list_page0 and lengths of all lists are final
    if (!fill_table) return;
    for (int idx = warp; idx < n_lists; idx += NT / 32) {            // a warp per list
        const int32_t p0 = list_page0[idx];
        const int32_t have = append ? (list_base[idx] + page_tokens - 1) / page_tokens : 0;
        const int64_t li = list_at(list_map, idx, n_heads);
        const int32_t need = (lengths[li] + page_tokens - 1) / page_tokens - have;
        for (int32_t i = lane; i < need; i += 32) {
            const int32_t j = p0 - first_page + i;            // ordinal among the pages assigned by this call
            page_table[li * max_pages + have + i] =
                j < from_stack ? free_stack[n_free - 1 - j] : first_page + (j - from_stack);
        }
    }
}



// ---------------------------------------------------------------------------
// One CTA of NT threads (all of them call it).  blockprefix [H][n_blocks+1], seqbase [H][n_seqs+1] (both nullptr when only the
// lengths and the page assignment are wanted: the lists are then counted directly), lengths [n_seqs][H].
// Paged output (page_tokens > 0): list (b,h) gets
// ceil(len/page_tokens) pages numbered contiguously from first_page in (b,h)
// order; list_page0 [n_seqs*H] receives each list's first page and page_table
// [n_seqs*H][max_pages] its page numbers; *n_pages_used the total.  A pool or
// table that is too small sets the status word and marks every list with
// list_page0 = -1 so that the compaction writes nothing.
// append != 0 (paged only): the lists already hold lengths[] rows in the pages their tables name; the
// kept rows are added behind them.  lengths becomes old + kept (unchanged on failure), only the pages
// beyond the old ones are assigned and entered into the table, and list_base receives the old length.
// With a cursor (a cache's allocator) the new pages are taken from the stack of released pages first
// (free_stack / free_top, may be nullptr), then from the cursor: the pages of a list are then not
// consecutive numbers and the compaction finds them through the table; list_page0 is the ordinal of
// the list's first new page among the pages this call assigns (plus first_page), or -1.
template <int NT>
__device__ __forceinline__ void
scan_lists(const uint32_t *__restrict__ maskbits, int64_t n_words, int64_t n_blocks, int n_heads,
            const int32_t *__restrict__ cu_seqlens, int n_seqs, int64_t n_tokens,
            int32_t *__restrict__ blockprefix, int32_t *__restrict__ seqbase, int32_t *__restrict__ lengths,
            int page_tokens, int32_t first_page, int64_t n_pages_pool, int max_pages,
            int32_t *__restrict__ list_page0, int32_t *__restrict__ page_table, int32_t *__restrict__ n_pages_used,
            int32_t *__restrict__ page_cursor, int32_t *__restrict__ status, int append,
            int32_t *__restrict__ list_base, const int32_t *__restrict__ free_stack, int32_t *__restrict__ free_top,
            const int64_t *__restrict__ list_map = nullptr)
{
    // page_cursor != nullptr: the first page comes from (and the pages used are added to) a device-side
    // allocator cursor instead of the first_page argument
    if (page_tokens > 0 && page_cursor != nullptr) first_page = *page_cursor;
    __shared__ int32_t warp_sums[32];
    __shared__ int32_t carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    auto block_scan = [&](int32_t v, int32_t &total) -> int32_t {   // inclusive scan over the CTA
        int32_t x = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        __syncthreads();
        if (lane == 31) warp_sums[warp] = x;
        __syncthreads();
        if (warp == 0) {
            int32_t w = lane < NT / 32 ? warp_sums[lane] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t y = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += y;
            }
            warp_sums[lane] = w;
        }
        __syncthreads();
        total = warp_sums[31];
        return x + (warp > 0 ? warp_sums[warp - 1] : 0);
    };

    if (blockprefix == nullptr) {
        // Only the lengths are wanted (the compaction counts its own prefixes): every list's kept rows are
        // counted straight from the mask words of its token range, a group of threads per list.
        const int n_lists_all = n_heads * n_seqs;
        int per_list = NT;
        while (per_list > 32 && NT / per_list < n_lists_all) per_list >>= 1;
        const int n_groups = NT / per_list, grp = tid / per_list, gt = tid % per_list;
        __shared__ int32_t group_sum[32];
        for (int idx0 = 0; idx0 < n_lists_all; idx0 += n_groups) {
            if (tid < 32) group_sum[tid] = 0;
            __syncthreads();
            const int idx = idx0 + grp;
            int32_t cnt = 0;
            if (idx < n_lists_all) {
                const int b = idx / n_heads, h = idx % n_heads;
                const int64_t t_lo = cu_seqlens != nullptr ? static_cast<int64_t>(cu_seqlens[b]) : 0;
                const int64_t t_hi = cu_seqlens != nullptr ? static_cast<int64_t>(cu_seqlens[b + 1]) : n_tokens;
                const uint32_t *wh = maskbits + static_cast<int64_t>(h) * n_words;
                for (int64_t wi = t_lo / 32 + gt; wi * 32 < t_hi; wi += per_list) {
                    uint32_t w = __ldcg(wh + wi);
                    if (wi * 32 < t_lo) w &= ~0u << static_cast<int>(t_lo - wi * 32);               // bits below the sequence
                    if (wi * 32 + 32 > t_hi) w &= (1u << static_cast<int>(t_hi - wi * 32)) - 1u;    // bits above it
                    cnt += __popc(w);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
            if (lane == 0 && cnt) atomicAdd(&group_sum[grp], cnt);
            __syncthreads();
            if (gt == 0 && idx < n_lists_all) {
                const int64_t li = list_at(list_map, idx, n_heads);
                const int32_t old = append ? lengths[li] : 0;
                if (append) list_base[idx] = old;
                lengths[li] = old + group_sum[grp];
            }
            __syncthreads();
        }
    } else {
    for (int h = 0; h < n_heads; ++h) {
        if (tid == 0) carry_s = 0;
        __syncthreads();
        for (int64_t base = 0; base < n_blocks; base += NT) {
            const int64_t blk = base + tid;
            int32_t cnt = 0;
            if (blk < n_blocks) {
                const uint4 w = __ldcg(reinterpret_cast<const uint4 *>(maskbits + static_cast<int64_t>(h) * n_words + blk * 4));
                cnt = __popc(w.x) + __popc(w.y) + __popc(w.z) + __popc(w.w);
            }
            int32_t total;
            const int32_t incl = block_scan(cnt, total);
            const int32_t carry = carry_s;
            if (blk < n_blocks) blockprefix[static_cast<int64_t>(h) * (n_blocks + 1) + blk] = carry + incl - cnt;
            __syncthreads();
            if (tid == 0) carry_s = carry + total;
            __syncthreads();
        }
        if (tid == 0) blockprefix[static_cast<int64_t>(h) * (n_blocks + 1) + n_blocks] = carry_s;
    }
    __syncthreads();      // blockprefix written by this CTA is visible to it from here on

    for (int idx = tid; idx < n_heads * (n_seqs + 1); idx += NT) {
        const int h = idx / (n_seqs + 1), b = idx % (n_seqs + 1);
        const int64_t t = cu_seqlens != nullptr ? static_cast<int64_t>(cu_seqlens[b]) : (b == 0 ? 0 : n_tokens);
        seqbase[idx] = kept_before(maskbits, n_words, blockprefix, n_blocks, h, t);
    }
    __syncthreads();
    for (int idx = tid; idx < n_heads * n_seqs; idx += NT) {
        const int b = idx / n_heads, h = idx % n_heads;
        const int64_t li = list_at(list_map, idx, n_heads);
        const int32_t old = append ? lengths[li] : 0;
        if (append) list_base[idx] = old;
        lengths[li] = old + seqbase[h * (n_seqs + 1) + b + 1] - seqbase[h * (n_seqs + 1) + b];
    }
    }
    if (page_tokens <= 0) return;
    __syncthreads();
    assign_pages<NT>(n_heads, n_seqs, lengths, page_tokens, first_page, n_pages_pool, max_pages, list_page0, page_table,
                     n_pages_used, page_cursor, status, append, list_base, free_stack, free_top, 1, list_map);
}

// The page assignment as a kernel of its own: one CTA of 1024 threads (behind the fused scoring kernels
// and for appending to a cache's lists).
__global__ void __launch_bounds__(1024)
scan_kernel(const uint32_t *__restrict__ maskbits, int64_t n_words, int64_t n_blocks, int n_heads,
            const int32_t *__restrict__ cu_seqlens, int n_seqs, int64_t n_tokens,
            int32_t *__restrict__ blockprefix, int32_t *__restrict__ seqbase, int32_t *__restrict__ lengths,
            int page_tokens, int32_t first_page, int64_t n_pages_pool, int max_pages,
            int32_t *__restrict__ list_page0, int32_t *__restrict__ page_table, int32_t *__restrict__ n_pages_used,
            int32_t *__restrict__ page_cursor, int32_t *__restrict__ status, int append,
            int32_t *__restrict__ list_base, const int32_t *__restrict__ free_stack, int32_t *__restrict__ free_top,
            const int64_t *__restrict__ list_map)
{
    // may be placed before the kernel that writes the mask has finished; waits for it here
    griddep_launch_dependents();
    griddep_wait();
    scan_lists<1024>(maskbits, n_words, n_blocks, n_heads, cu_seqlens, n_seqs, n_tokens, blockprefix, seqbase, lengths,
                     page_tokens, first_page, n_pages_pool, max_pages, list_page0, page_table, n_pages_used, page_cursor,
                     status, append, list_base, free_stack, free_top, list_map);
}

// ---------------------------------------------------------------------------
// One CTA per (128-token block, head).  Rows are row_bytes = 2*D bytes, moved
// as 16-byte units by 16-lane groups; up to kRowsInFlight rows of K and of V
// are loaded before any is stored.
constexpr int kCompactThreads = 256;
constexpr int kRowsInFlight = 4;

template <bool kPaged>
__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(const uint4 *__restrict__ K, const uint4 *__restrict__ V, uint4 *__restrict__ K_out,
               uint4 *__restrict__ V_out, const uint32_t *__restrict__ maskbits, int64_t n_words, int64_t n_blocks,
               const int32_t *__restrict__ blockprefix, const int32_t *__restrict__ seqbase,
               const int32_t *__restrict__ cu_seqlens, int n_seqs, int64_t n_tokens, int n_heads, int row_units,
               int page_tokens, const int32_t *__restrict__ list_page0)
{
    __shared__ int32_t src_tok[kBlockTokens];     // packed token index of the i-th kept row of this block
    __shared__ int64_t dst_row[kBlockTokens];     // its destination row (dense: within head h; paged: pool row)
    const int64_t blk = blockIdx.x;
    const int h = blockIdx.y;
    const int tid = threadIdx.x;
    const uint32_t *words = maskbits + static_cast<int64_t>(h) * n_words + blk * 4;
    const uint32_t w0 = words[0], w1 = words[1], w2 = words[2], w3 = words[3];
    const int cnt = __popc(w0) + __popc(w1) + __popc(w2) + __popc(w3);
    if (cnt == 0) return;
    if (tid < kBlockTokens) {
        const int wi = tid >> 5, bit = tid & 31;
        const uint32_t w = wi == 0 ? w0 : wi == 1 ? w1 : wi == 2 ? w2 : w3;
        if ((w >> bit) & 1u) {
            int r = __popc(w & ((1u << bit) - 1u));
            if (wi > 0) r += __popc(w0);
            if (wi > 1) r += __popc(w1);
            if (wi > 2) r += __popc(w2);
            const int64_t t = blk * kBlockTokens + tid;
            const int32_t before = blockprefix[static_cast<int64_t>(h) * (n_blocks + 1) + blk] + r;
            int b = 0;
            int64_t seq_start = 0;
            if (cu_seqlens != nullptr && n_seqs > 1) {
                b = seq_of_token(cu_seqlens, n_seqs, t);
                seq_start = cu_seqlens[b];
            }
            const int64_t n = before - seqbase[h * (n_seqs + 1) + b];     // rank inside list (b,h)
            int64_t dst;
            if constexpr (kPaged) {
                const int32_t p0 = list_page0[b * n_heads + h];
                dst = p0 < 0 ? -1 : (static_cast<int64_t>(p0) + n / page_tokens) * page_tokens + n % page_tokens;
            } else {
                dst = static_cast<int64_t>(h) * n_tokens + seq_start + n;
            }
            src_tok[r] = static_cast<int32_t>(t - blk * kBlockTokens);
            dst_row[r] = dst;
        }
    }
    __syncthreads();

    const int group = tid >> 4, gl = tid & 15;            // 16 groups of 16 lanes
    constexpr int kGroups = kCompactThreads / 16;
    const int64_t head_row0 = static_cast<int64_t>(h) * n_tokens + blk * kBlockTokens;
    for (int i0 = group; i0 < cnt; i0 += kGroups * kRowsInFlight) {
        for (int u0 = gl; u0 < row_units; u0 += 16) {
            uint4 kv[kRowsInFlight], vv[kRowsInFlight];
#pragma unroll
            for (int j = 0; j < kRowsInFlight; ++j) {
                const int i = i0 + j * kGroups;
                if (i < cnt) {
                    const int64_t src = (head_row0 + src_tok[i]) * row_units + u0;
                    kv[j] = __ldg(K + src);
                    vv[j] = __ldg(V + src);
                }
            }
#pragma unroll
            for (int j = 0; j < kRowsInFlight; ++j) {
                const int i = i0 + j * kGroups;
                if (i < cnt) {
                    const int64_t d = dst_row[i];
                    if (d >= 0) {
                        K_out[d * row_units + u0] = kv[j];
                        V_out[d * row_units + u0] = vv[j];
                    }
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------
// Dense-ragged compaction without a separate scan pass.  Grid (chunks, H): a CTA owns
// `blocks_per_cta` consecutive 128-token blocks of one head.  It first counts, straight from the
// mask words, the rows kept before its first block (and before the start of the sequence that is
// in progress there), then walks its blocks keeping a running count, so that every kept row's
// slot in its (sequence, head) list is known without any other CTA's help.  lengths[b,h] is
// written by the thread that handles the last token of sequence b; empty sequences by chunk 0.
constexpr int kDenseThreads = 128;     // = kBlockTokens: one thread ranks one token; small enough to sit beside a scoring CTA
constexpr int kDenseThreadsShort = 256; // short inputs (one block per CTA): twice the rows in flight, one round of row loads

// bits of the block's four words below in-block position r (0..128)
__device__ __forceinline__ int popc_below(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, int r)
{
    int n = 0;
    const uint32_t w[4] = {w0, w1, w2, w3};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int lo = i * 32;
        if (r >= lo + 32) n += __popc(w[i]);
        else if (r > lo) n += __popc(w[i] & ((1u << (r - lo)) - 1u));
    }
    return n;
}

// kThreads = 128, or 256 for short inputs (one block per CTA: all kept rows of the block in flight at once).
// At most 64 registers per thread (eight 128-thread CTAs per SM by registers): two of these CTAs then fit into the
// register-file quarters that the MLP scoring kernel's ten warps leave free, so the compaction of layer
// l runs beside the scoring of layer l + 1 at full width; at 72 registers only one fits and the layer
// period of the fused path grows by ~10 us.
template <int kThreads>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
compact_dense_kernel(const uint4 *__restrict__ K, const uint4 *__restrict__ V, uint4 *__restrict__ K_out,
                     uint4 *__restrict__ V_out, const uint32_t *__restrict__ maskbits, int64_t n_words,
                     int64_t n_blocks, int blocks_per_cta, const int32_t *__restrict__ cu_seqlens, int n_seqs,
                     int64_t n_tokens, int n_heads, int row_units, int32_t *__restrict__ lengths, int page_tokens,
                     const int32_t *__restrict__ list_page0, int64_t in_stride_h, int64_t in_stride_t,
                     const int32_t *__restrict__ list_base, const int32_t *__restrict__ page_table, int max_pages,
                     const int64_t *__restrict__ list_map)
{
    // list_base != nullptr (paged): list (b,h) already holds list_base[] rows; kept rows go behind them,
    // into the pages that page_table [list][max_pages] names (the scan has entered the new ones); the table
    // of list (b,h) is row b * H + h of page_table, or row list_map[b] + h (see list_at).
    // Row (h, t) of the inputs starts at row index h * in_stride_h + t * in_stride_t: (n_tokens, 1) for
    // the head-major cache layout [H][T][D], (1, H) for the K/V projection's own output [T][H][D].
    // page_tokens > 0: paged output.  K_out / V_out are the page pools, list (b,h) starts at page
    // list_page0[b * H + h] (-1 = nothing may be written), and lengths come from the scan kernel.
    const bool paged = page_tokens > 0;
    __shared__ int32_t src_tok[kBlockTokens];
    __shared__ int64_t dst_row[kBlockTokens];
    __shared__ int32_t red[2][kThreads / 32];
    __shared__ int32_t base_next_s;
    const int h = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t blk0 = static_cast<int64_t>(blockIdx.x) * blocks_per_cta;
    const int64_t blk1 = blk0 + blocks_per_cta < n_blocks ? blk0 + blocks_per_cta : n_blocks;
    const bool multi = cu_seqlens != nullptr && n_seqs > 1;
    const uint32_t *words = maskbits + static_cast<int64_t>(h) * n_words;

    // This grid is small enough to be resident all at once: the next kernel in the stream may be
    // placed as soon as it is; the mask itself is read only after the kernel ahead has completed.
    griddep_launch_dependents();
    griddep_wait();

    if (blockIdx.x == 0 && cu_seqlens != nullptr && !paged)   // empty sequences have no last token to write for them
        for (int b = tid; b < n_seqs; b += kThreads)
            if (cu_seqlens[b + 1] == cu_seqlens[b]) lengths[b * n_heads + h] = 0;
    if (blk0 >= n_blocks) return;

    // rows kept before this CTA's first token, and before the start of the sequence in progress there
    const int64_t t0 = blk0 * kBlockTokens;
    int64_t s0 = 0;
    if (multi) s0 = cu_seqlens[seq_of_token(cu_seqlens, n_seqs, t0)];
    int32_t total = 0, before_s0 = 0;
    // the first block's own words are fetched together with the words before it (one round trip, not two)
    uint4 wv_next = __ldcg(reinterpret_cast<const uint4 *>(words + blk0 * 4));
    for (int64_t i = tid; i < blk0 * 4; i += kThreads) {
        const uint32_t w = __ldcg(words + i);     // not a read-only-data load: it must stay behind griddep_wait()
        const int c = __popc(w);
        total += c;
        const int64_t lo = i * 32;
        if (lo + 32 <= s0) before_s0 += c;
        else if (lo < s0) before_s0 += __popc(w & ((1u << static_cast<int>(s0 - lo)) - 1u));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        total += __shfl_xor_sync(0xffffffffu, total, o);
        before_s0 += __shfl_xor_sync(0xffffffffu, before_s0, o);
    }
    if (lane == 0) { red[0][warp] = total; red[1][warp] = before_s0; }
    __syncthreads();
    int32_t running = 0, base_cur = 0;       // kept before the current block / before the sequence in progress at its start
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) { running += red[0][i]; base_cur += red[1][i]; }

    const int group = tid >> 4, gl = tid & 15;
    constexpr int kGroups = kThreads / 16;
    for (int64_t blk = blk0; blk < blk1; ++blk) {
        const uint4 wv = wv_next;
        if (blk + 1 < blk1) wv_next = __ldcg(reinterpret_cast<const uint4 *>(words + (blk + 1) * 4));
        const uint32_t w0 = wv.x, w1 = wv.y, w2 = wv.z, w3 = wv.w;
        const int cnt = __popc(w0) + __popc(w1) + __popc(w2) + __popc(w3);
        const int64_t blk_start = blk * kBlockTokens;
        if (tid < kBlockTokens) {
            const int64_t t = blk_start + tid;
            if (t < n_tokens) {
                int b = 0;
                int64_t s = 0, e = n_tokens;
                if (multi) {
                    b = seq_of_token(cu_seqlens, n_seqs, t);
                    s = cu_seqlens[b];
                    e = cu_seqlens[b + 1];
                }
                // kept rows before the start of this token's sequence
                const int32_t base = s >= blk_start ? running + popc_below(w0, w1, w2, w3, static_cast<int>(s - blk_start))
                                                    : base_cur;
                const int r = popc_below(w0, w1, w2, w3, tid);
                const uint32_t w = tid < 32 ? w0 : tid < 64 ? w1 : tid < 96 ? w2 : w3;
                const bool keep = (w >> (tid & 31)) & 1u;
                if (keep) {
                    src_tok[r] = tid;
                    const int64_t n = running + r - base;                  // rank inside list (b,h)
                    if (paged) {
                        const int32_t p0 = list_page0[b * n_heads + h];
                        if (list_base == nullptr) {
                            dst_row[r] = p0 < 0 ? -1 : (static_cast<int64_t>(p0) + n / page_tokens) * page_tokens + n % page_tokens;
                        } else {
                            const int64_t nn = list_base[b * n_heads + h] + n;
                            if (p0 < 0) {
                                dst_row[r] = -1;
                            } else {
                                const int64_t trow = list_map != nullptr ? list_map[b] + h : static_cast<int64_t>(b * n_heads + h);
                                const int64_t page = __ldcg(page_table + trow * max_pages + nn / page_tokens);
                                dst_row[r] = page * page_tokens + nn % page_tokens;
                            }
                        }
                    } else {
                        dst_row[r] = static_cast<int64_t>(h) * n_tokens + s + n;
                    }
                }
                if (t + 1 == e && !paged) lengths[b * n_heads + h] = running + r + (keep ? 1 : 0) - base;
                if (tid == kBlockTokens - 1 || t + 1 == n_tokens) {
                    // base of the sequence in progress at the next block's first token
                    int32_t nb = base;
                    if (multi && t + 1 == e) nb = running + cnt;      // a new sequence starts exactly there
                    base_next_s = nb;
                }
            }
        }
        __syncthreads();
        const int64_t head_row0 = static_cast<int64_t>(h) * in_stride_h + blk_start * in_stride_t;
        for (int i0 = group; i0 < cnt; i0 += kGroups * kRowsInFlight) {
            for (int u0 = gl; u0 < row_units; u0 += 16) {
                uint4 kv[kRowsInFlight], vv[kRowsInFlight];
#pragma unroll
                for (int j = 0; j < kRowsInFlight; ++j) {
                    const int i = i0 + j * kGroups;
                    if (i < cnt) {
                        const int64_t src = (head_row0 + src_tok[i] * in_stride_t) * row_units + u0;
                        kv[j] = __ldg(K + src);
                        vv[j] = __ldg(V + src);
                    }
                }
#pragma unroll
                for (int j = 0; j < kRowsInFlight; ++j) {
                    const int i = i0 + j * kGroups;
                    if (i < cnt && dst_row[i] >= 0) {
                        const int64_t d = dst_row[i] * row_units + u0;
                        K_out[d] = kv[j];
                        V_out[d] = vv[j];
                    }
                }
            }
        }
        running += cnt;
        base_cur = base_next_s;
        __syncthreads();
    }
}

}  // namespace kvzap
