// Decode-time pruning on a paged, ragged cache (caption of Algorithm 1: decoding
// applies the same rule with a buffer of the scores of the tokens still inside the
// sliding window; contribution list: delayed eviction with a sliding window).
//
// One list per (sequence b, layer l, KV head h), index li = (b * L + l) * H + h:
//   window ring   k_ring / v_ring [li][w][D], score_ring [li][w]: the most recent w tokens,
//                 position p lives in slot p % w
//   prefix        the tokens that left the window with score >= tau, in position order,
//                 stored in pages of page_tokens rows taken from the caller's pool;
//                 page_table [li][max_pages], prefix_len [li]
//   n_tokens [li] tokens appended so far
// A step appends one token per sequence: the token that leaves the window (position
// n - w, found in the very slot the new token will take) is copied to the prefix iff
// its buffered score >= tau, then the new row and its score overwrite the slot.
// Logical cache = prefix ++ window in age order.  Pages come from a bump allocator
// (atomicAdd on one cursor); an exhausted pool or page table sets the status word and
// drops the row instead of writing out of bounds.
#pragma once

#include "ptx.cuh"

namespace kvzap {

struct CacheView {
    int32_t n_seqs, n_layers, n_heads, row_units, window, page_tokens, max_pages;
    int64_t n_pages_pool;
    uint4 *k_ring, *v_ring;
    float *score_ring;
    int32_t *n_tokens, *prefix_len, *page_table, *page_cursor;
    uint4 *k_pool, *v_pool;
};

constexpr int kDecodeThreads = 256;
constexpr int kDecodeLanes = 8;        // lanes that share one list (a 256-byte row = two 16-byte units per lane)

// kDecodeLanes lanes per list; lists of layers [layer0, layer0 + n_layers_call); the grid walks the lists
// with a grid stride.  scores [n_layers_call][B][H] fp32, K_new/V_new [n_layers_call][B][H][D] bf16.
//
// The kernel is launched so that it may be placed while the scoring kernel ahead of it in the stream
// is still running.  With a window, the fate of the token that leaves it depends only on its
// BUFFERED score, so the row traffic (old row to its page, new rows into the ring) needs nothing
// from that kernel and only the new scores wait for it.  `wait_first` != 0 makes the whole kernel
// wait instead: required when the scoring kernel itself was started before the previous step's
// update had finished (two updates must never touch the cache at the same time).
__global__ void __launch_bounds__(kDecodeThreads)
decode_update_kernel(const CacheView c, int layer0, int n_layers_call, const float *__restrict__ scores,
                     const uint4 *__restrict__ K_new, const uint4 *__restrict__ V_new, float tau,
                     int32_t *__restrict__ status, int wait_first)
{
    griddep_launch_dependents();
    const bool rows_first = c.window > 0 && wait_first == 0;
    if (!rows_first) griddep_wait();                     // every thread executes the wait
    const int gl = threadIdx.x % kDecodeLanes;
    const int64_t n_groups = static_cast<int64_t>(n_layers_call) * c.n_seqs * c.n_heads;
    const int64_t group0 = (static_cast<int64_t>(blockIdx.x) * kDecodeThreads + threadIdx.x) / kDecodeLanes;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * (kDecodeThreads / kDecodeLanes);
    const int64_t n_iter = (n_groups + stride - 1) / stride;       // the same for every thread
    for (int64_t it = 0; it < n_iter; ++it) {
        const int64_t group = group0 + it * stride;
        const bool live = group < n_groups;
        // every lane of the warp runs the whole body (the shuffles below need all 32 lanes)
        const int64_t g = live ? group : 0;
        const int l_rel = static_cast<int>(g / (static_cast<int64_t>(c.n_seqs) * c.n_heads));
        const int rem = static_cast<int>(g - static_cast<int64_t>(l_rel) * c.n_seqs * c.n_heads);
        const int b = rem / c.n_heads, h = rem % c.n_heads;
        const int64_t li = (static_cast<int64_t>(b) * c.n_layers + layer0 + l_rel) * c.n_heads + h;
        const int64_t src_row = (static_cast<int64_t>(l_rel) * c.n_seqs + b) * c.n_heads + h;
        const int32_t n = c.n_tokens[li];

        // which row (if any) moves to the prefix now
        bool append = false;
        const uint4 *app_k = nullptr, *app_v = nullptr;
        int slot = 0;
        if (c.window > 0) {
            slot = n % c.window;
            if (n >= c.window) {
                const float s_old = c.score_ring[li * c.window + slot];
                append = s_old >= tau;
                app_k = c.k_ring + (li * c.window + slot) * c.row_units;
                app_v = c.v_ring + (li * c.window + slot) * c.row_units;
            }
        } else {
            append = __ldcg(scores + src_row) >= tau;
            app_k = K_new + src_row * c.row_units;
            app_v = V_new + src_row * c.row_units;
        }
        append = append && live;

        // page for the appended row: lane 0 of the group allocates when the row opens a new page
        const int32_t idx = c.prefix_len[li];
        const int page_i = idx / c.page_tokens, in_page = idx % c.page_tokens;
        int32_t page = -1;
        if (append && gl == 0) {
            if (page_i >= c.max_pages) {
                atomicCAS(status, 0, 4 /* KVZAP_ERR_OOM_PAGES */);
            } else if (in_page == 0) {
                const int32_t got = atomicAdd(c.page_cursor, 1);
                if (got >= c.n_pages_pool) {
                    atomicCAS(status, 0, 4);
                } else {
                    page = got;
                    c.page_table[li * c.max_pages + page_i] = got;
                }
            } else {
                page = c.page_table[li * c.max_pages + page_i];
            }
        }
        page = __shfl_sync(0xffffffffu, page, 0, kDecodeLanes);
        if (append && page >= 0) {
            const int64_t dst = (static_cast<int64_t>(page) * c.page_tokens + in_page) * c.row_units;
            for (int u = gl; u < c.row_units; u += 2 * kDecodeLanes) {       // all loads of a pass before its stores
                const int u2 = u + kDecodeLanes;
                const bool two = u2 < c.row_units;
                const uint4 ka = app_k[u], va = app_v[u];
                uint4 kb = ka, vb = va;
                if (two) { kb = app_k[u2]; vb = app_v[u2]; }
                c.k_pool[dst + u] = ka;
                c.v_pool[dst + u] = va;
                if (two) { c.k_pool[dst + u2] = kb; c.v_pool[dst + u2] = vb; }
            }
            if (gl == 0) c.prefix_len[li] = idx + 1;
        }
        if (live && c.window > 0) {
            // each lane overwrites exactly the 16-byte units it read above, so no lane races another
            const int64_t ring = (li * c.window + slot) * c.row_units;
            const uint4 *kn = K_new + src_row * c.row_units, *vn = V_new + src_row * c.row_units;
            for (int u = gl; u < c.row_units; u += 2 * kDecodeLanes) {
                const int u2 = u + kDecodeLanes;
                const bool two = u2 < c.row_units;
                const uint4 ka = __ldg(kn + u), va = __ldg(vn + u);
                uint4 kb = ka, vb = va;
                if (two) { kb = __ldg(kn + u2); vb = __ldg(vn + u2); }
                c.k_ring[ring + u] = ka;
                c.v_ring[ring + u] = va;
                if (two) { c.k_ring[ring + u2] = kb; c.v_ring[ring + u2] = vb; }
            }
        }
        if (live && gl == 0) {
            c.n_tokens[li] = n + 1;
            if (c.window > 0 && !rows_first) c.score_ring[li * c.window + slot] = __ldcg(scores + src_row);
        }
    }
    if (rows_first) {
        griddep_wait();                                  // every thread; the scoring kernel's output is needed only here
        if (gl == 0) {
            for (int64_t it = 0; it < n_iter; ++it) {
                const int64_t group = group0 + it * stride;
                if (group >= n_groups) break;
                const int l_rel = static_cast<int>(group / (static_cast<int64_t>(c.n_seqs) * c.n_heads));
                const int rem = static_cast<int>(group - static_cast<int64_t>(l_rel) * c.n_seqs * c.n_heads);
                const int b = rem / c.n_heads, h = rem % c.n_heads;
                const int64_t li = (static_cast<int64_t>(b) * c.n_layers + layer0 + l_rel) * c.n_heads + h;
                const int64_t src_row = (static_cast<int64_t>(l_rel) * c.n_seqs + b) * c.n_heads + h;
                const int slot = (c.n_tokens[li] - 1) % c.window;      // the slot this thread filled above
                c.score_ring[li * c.window + slot] = __ldcg(scores + src_row);
            }
        }
    }
}

// A further chunk of m prompt tokens is about to be appended to lists li0 .. li0+H-1 (chunked
// prefill): the tokens of the present window that it pushes out are decided here by their buffered
// scores, oldest first, and the kept ones appended to the list's paged prefix (pages from the
// cache's cursor), exactly as m decode steps would have done.  One warp per list; n_tokens is left
// as it is (tokens_add_kernel advances it once the chunk's own rows are in place).
__global__ void __launch_bounds__(32)
chunk_evict_kernel(const CacheView c, int64_t li0, int64_t m, float tau, int32_t *__restrict__ status)
{
    const int64_t li = li0 + blockIdx.x;
    const int lane = threadIdx.x;
    const int64_t n_old = c.n_tokens[li];
    const int64_t in_ring = n_old < c.window ? n_old : c.window;
    const int64_t first = n_old - in_ring;                         // oldest position still in the window
    int64_t exit_end = n_old + m - c.window;                       // positions below it leave the window
    if (exit_end > n_old) exit_end = n_old;
    const int64_t n_exit = exit_end > first ? exit_end - first : 0;
    int64_t len = c.prefix_len[li];
    int32_t *table = c.page_table + li * c.max_pages;
    for (int64_t base = 0; base < n_exit; base += 32) {
        const int64_t pos = first + base + lane;
        const bool valid = base + lane < n_exit;
        const int64_t slot = li * c.window + pos % c.window;
        const bool keep = valid && c.score_ring[slot] >= tau;
        const uint32_t kept = __ballot_sync(0xffffffffu, keep);
        const int cnt = __popc(kept);
        const int64_t have = (len + c.page_tokens - 1) / c.page_tokens;
        const int64_t want = (len + cnt + c.page_tokens - 1) / c.page_tokens;
        int ok = 1;
        if (lane == 0 && want > have) {
            if (want > c.max_pages) ok = 0;
            else {
                const int32_t got = atomicAdd(c.page_cursor, static_cast<int32_t>(want - have));
                if (static_cast<int64_t>(got) + (want - have) > c.n_pages_pool) ok = 0;
                else for (int64_t i = have; i < want; ++i) table[i] = got + static_cast<int32_t>(i - have);
            }
            if (!ok) atomicCAS(status, 0, 4 /* KVZAP_ERR_OOM_PAGES */);
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;                                            // what was appended so far stays valid
        __syncwarp();
        if (keep) {
            const int64_t nn = len + __popc(kept & ((1u << lane) - 1u));
            const int64_t page = *(volatile int32_t *)(table + nn / c.page_tokens);
            const int64_t dst = (page * c.page_tokens + nn % c.page_tokens) * c.row_units;
            for (int u = 0; u < c.row_units; ++u) {
                c.k_pool[dst + u] = c.k_ring[slot * c.row_units + u];
                c.v_pool[dst + u] = c.v_ring[slot * c.row_units + u];
            }
        }
        len += cnt;
    }
    if (lane == 0) c.prefix_len[li] = static_cast<int32_t>(len);
}

// The last min(m, w) tokens of a chunk of m (rows of K, V [H][m][D], scores [m][H]) go into the window
// rings of lists li0 .. li0+H-1 at the slots of their absolute positions n_tokens + chunk index.
__global__ void __launch_bounds__(256)
ring_append_kernel(const CacheView c, int64_t li0, const float *__restrict__ scores, const uint4 *__restrict__ K,
                   const uint4 *__restrict__ V, int64_t m)
{
    const int h = blockIdx.y;
    const int64_t li = li0 + h;
    const int64_t n_old = c.n_tokens[li];
    const int64_t n_win = m < c.window ? m : c.window;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_win * c.row_units;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t j = i / c.row_units;
        const int u = static_cast<int>(i % c.row_units);
        const int64_t ci = m - n_win + j;                      // index inside the chunk
        const int64_t slot = li * c.window + (n_old + ci) % c.window;
        const int64_t src = (static_cast<int64_t>(h) * m + ci) * c.row_units + u;
        c.k_ring[slot * c.row_units + u] = K[src];
        c.v_ring[slot * c.row_units + u] = V[src];
        if (u == 0) c.score_ring[slot] = scores[ci * c.n_heads + h];
    }
}

__global__ void tokens_add_kernel(const CacheView c, int64_t li0, int64_t m)
{
    if (threadIdx.x < c.n_heads) c.n_tokens[li0 + threadIdx.x] += static_cast<int32_t>(m);
}

// lengths[li] = prefix_len + min(n_tokens, w)
__global__ void cache_lengths_kernel(const CacheView c, int32_t *__restrict__ lengths)
{
    const int64_t li = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t n_lists = static_cast<int64_t>(c.n_seqs) * c.n_layers * c.n_heads;
    if (li < n_lists) lengths[li] = c.prefix_len[li] + min(c.n_tokens[li], c.window);
}

// Linearises one list (prefix pages, then the window oldest first) into K_out/V_out [capacity][D].
__global__ void __launch_bounds__(256)
cache_export_kernel(const CacheView c, int64_t li, uint4 *__restrict__ K_out, uint4 *__restrict__ V_out,
                    int64_t capacity_rows, int32_t *__restrict__ n_rows)
{
    const int32_t n_prefix = c.prefix_len[li];
    const int32_t n = c.n_tokens[li];
    const int32_t n_win = min(n, c.window);
    const int64_t total = static_cast<int64_t>(n_prefix) + n_win;
    if (threadIdx.x == 0 && blockIdx.x == 0) *n_rows = static_cast<int32_t>(total);
    const int64_t rows = total < capacity_rows ? total : capacity_rows;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < rows * c.row_units;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t r = i / c.row_units;
        const int u = static_cast<int>(i % c.row_units);
        int64_t src;
        const uint4 *ksrc, *vsrc;
        if (r < n_prefix) {
            const int32_t page = c.page_table[li * c.max_pages + r / c.page_tokens];
            src = (static_cast<int64_t>(page) * c.page_tokens + r % c.page_tokens) * c.row_units + u;
            ksrc = c.k_pool;
            vsrc = c.v_pool;
        } else {
            const int64_t pos = static_cast<int64_t>(n) - n_win + (r - n_prefix);
            src = (li * c.window + pos % c.window) * c.row_units + u;
            ksrc = c.k_ring;
            vsrc = c.v_ring;
        }
        K_out[i] = ksrc[src];
        V_out[i] = vsrc[src];
    }
}

}  // namespace kvzap
