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
    // pages given back by released sequences: a stack; a new page is taken from it before the cursor moves on
    int32_t *free_stack;      // [n_pages_pool]
    int32_t *free_top;        // entries on the stack
    // 0 for a slot whose sequence has been released and that has not been given a new prompt: decode steps
    // leave its lists alone
    uint8_t *active;          // [n_seqs]
};

// One more page for a list: a released one if the stack has any, else the next never-used page of the
// pool; -1 (and the status word) when neither is left.  Kernels that take pages never release any, so the
// stack only shrinks while they run: an index handed out by the atomic below is stable.
__device__ __forceinline__ int32_t cache_take_page(const CacheView &c, int32_t *status)
{
    if (__ldcg(c.free_top) > 0) {                       // the usual case, an empty stack, costs one load
        const int32_t top = atomicSub(c.free_top, 1);
        if (top > 0) return c.free_stack[top - 1];
        atomicAdd(c.free_top, 1);                       // someone else took the last one
    }
    const int32_t got = atomicAdd(c.page_cursor, 1);
    if (got >= c.n_pages_pool) {
        atomicCAS(status, 0, 4 /* KVZAP_ERR_OOM_PAGES */);
        return -1;
    }
    return got;
}

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
        const bool in_range = group < n_groups;
        // every lane of the warp runs the whole body (the shuffles below need all 32 lanes)
        const int64_t g = in_range ? group : 0;
        const int l_rel = static_cast<int>(g / (static_cast<int64_t>(c.n_seqs) * c.n_heads));
        const int rem = static_cast<int>(g - static_cast<int64_t>(l_rel) * c.n_seqs * c.n_heads);
        const int b = rem / c.n_heads, h = rem % c.n_heads;
        const int64_t li = (static_cast<int64_t>(b) * c.n_layers + layer0 + l_rel) * c.n_heads + h;
        const int64_t src_row = (static_cast<int64_t>(l_rel) * c.n_seqs + b) * c.n_heads + h;
        const int32_t n = c.n_tokens[li];
        const bool live = in_range && c.active[b] != 0;

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
                page = cache_take_page(c, status);
                if (page >= 0) c.page_table[li * c.max_pages + page_i] = page;
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
                if (c.active[b] == 0) continue;
                const int slot = (c.n_tokens[li] - 1) % c.window;      // the slot this thread filled above
                c.score_ring[li * c.window + slot] = __ldcg(scores + src_row);
            }
        }
    }
}

// Chunked prefill, the window side of one chunk of m prompt tokens appended to lists li0 .. li0+H-1
// (one CTA per list), after the chunk has been scored:
//   1. the tokens of the present window that the chunk pushes out (positions below n_old + m - w) are
//      decided by their buffered scores, oldest first, and the kept ones appended to the list's paged
//      prefix (pages from the cache's cursor) -- what m decode steps would have done;
//   2. the chunk's last min(m, w) tokens (rows of K, V [H][m][D], scores [m][H]) take the ring slots of
//      their absolute positions n_old + chunk index;
//   3. n_tokens advances by m.
// The chunk's own tokens before its last w are appended to the prefix afterwards by the compaction.
// A batch of prompts in one launch (grid (H, n_seqs)): sequence b's chunk is tokens cu_seqlens[b] .. cu_seqlens[b+1]
// of the packed buffers (K, V [H][n_total][D], scores [n_total][H]) and its lists start at list_map[b];
// list_map == nullptr: one sequence, lists li0 .. li0+H-1, m = n_total tokens.
__global__ void __launch_bounds__(256)
chunk_ring_kernel(const CacheView c, int64_t li0, const float *__restrict__ scores, const uint4 *__restrict__ K,
                  const uint4 *__restrict__ V, int64_t n_total, float tau, int32_t *__restrict__ status,
                  const int64_t *__restrict__ list_map, const int32_t *__restrict__ cu_seqlens)
{
    __shared__ int64_t exit_src[128];       // ring row of an exiting token
    __shared__ int64_t exit_dst[128];       // its pool row, -1 = dropped
    __shared__ int64_t len_s;
    __shared__ int ok_s;
    const int h = blockIdx.x;
    const int64_t li = (list_map != nullptr ? list_map[blockIdx.y] : li0) + h;
    const int64_t tok0 = list_map != nullptr ? static_cast<int64_t>(cu_seqlens[blockIdx.y]) : 0;
    const int64_t m = list_map != nullptr ? static_cast<int64_t>(cu_seqlens[blockIdx.y + 1]) - tok0 : n_total;
    if (m <= 0) return;                     // an empty chunk leaves its lists as they are
    K += tok0 * c.row_units;                // row (h, i) of the chunk is row h * n_total + tok0 + i of the buffers
    V += tok0 * c.row_units;
    scores += tok0 * c.n_heads;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t n_old = c.n_tokens[li];
    const int64_t in_ring = n_old < c.window ? n_old : c.window;
    const int64_t first = n_old - in_ring;                         // oldest position still in the window
    int64_t exit_end = n_old + m - c.window;                       // positions below it leave the window
    if (exit_end > n_old) exit_end = n_old;
    const int64_t n_exit = exit_end > first ? exit_end - first : 0;
    int32_t *table = c.page_table + li * c.max_pages;
    if (tid == 0) { len_s = c.prefix_len[li]; ok_s = 1; }
    __syncthreads();
    for (int64_t base = 0; base < n_exit && ok_s; base += 128) {
        if (warp == 0) {
            int64_t len = len_s;
            for (int i = lane; i < 128; i += 32) exit_dst[i] = -1;     // nothing is copied unless it is decided below
            float sc4[4];                                              // the buffered scores of the batch, loaded together
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int64_t pos = first + base + 32 * j + lane;
                sc4[j] = base + 32 * j + lane < n_exit ? c.score_ring[li * c.window + pos % c.window] : 0.0f;
            }
            __syncwarp();
#pragma unroll
            for (int sub = 0; sub < 128; sub += 32) {
                if (base + sub >= n_exit) break;
                const int64_t pos = first + base + sub + lane;
                const bool valid = base + sub + lane < n_exit;
                const int64_t slot = li * c.window + pos % c.window;
                const bool keep = valid && sc4[sub >> 5] >= tau;
                const uint32_t kept = __ballot_sync(0xffffffffu, keep);
                const int cnt = __popc(kept);
                const int64_t have = (len + c.page_tokens - 1) / c.page_tokens;
                const int64_t want = (len + cnt + c.page_tokens - 1) / c.page_tokens;
                int ok = 1;
                if (lane == 0 && want > have) {
                    if (want > c.max_pages) {
                        ok = 0;
                        atomicCAS(status, 0, 4 /* KVZAP_ERR_OOM_PAGES */);
                    } else {
                        for (int64_t i = have; i < want && ok; ++i) {
                            const int32_t page = cache_take_page(c, status);
                            if (page < 0) ok = 0;
                            else table[i] = page;
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                __syncwarp();
                if (valid) {
                    int64_t dst = -1;
                    if (keep && ok) {
                        const int64_t nn = len + __popc(kept & ((1u << lane) - 1u));
                        const int64_t page = *(volatile int32_t *)(table + nn / c.page_tokens);
                        dst = page * c.page_tokens + nn % c.page_tokens;
                    }
                    exit_src[sub + lane] = slot;
                    exit_dst[sub + lane] = dst;
                }
                if (!ok) { if (lane == 0) ok_s = 0; break; }       // what was appended so far stays valid
                len += cnt;
            }
            if (lane == 0) len_s = len;
        }
        __syncthreads();
        // rows of this batch of exits: 16 lanes per row
        const int64_t n_batch = n_exit - base < 128 ? n_exit - base : 128;
        for (int64_t i0 = tid >> 4; i0 < n_batch; i0 += 64) {     // four rows per lane group in flight
            for (int u = tid & 15; u < c.row_units; u += 16) {
                uint4 kr[4], vr[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t i = i0 + 16 * j;
                    if (i < n_batch && exit_dst[i] >= 0) {
                        kr[j] = c.k_ring[exit_src[i] * c.row_units + u];
                        vr[j] = c.v_ring[exit_src[i] * c.row_units + u];
                    }
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t i = i0 + 16 * j;
                    if (i < n_batch && exit_dst[i] >= 0) {
                        c.k_pool[exit_dst[i] * c.row_units + u] = kr[j];
                        c.v_pool[exit_dst[i] * c.row_units + u] = vr[j];
                    }
                }
            }
        }
        __syncthreads();
    }
    // the chunk's last min(m, w) tokens into the ring (the slots they take were read above)
    const int64_t n_win = m < c.window ? m : c.window;
    for (int64_t i0 = tid; i0 < n_win * c.row_units; i0 += 4 * 256) {     // four units per thread in flight
        uint4 kr[4], vr[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t i = i0 + 256 * j;
            if (i < n_win * c.row_units) {
                const int64_t src = (static_cast<int64_t>(h) * n_total + m - n_win + i / c.row_units) * c.row_units + i % c.row_units;
                kr[j] = __ldg(K + src);
                vr[j] = __ldg(V + src);
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t i = i0 + 256 * j;
            if (i < n_win * c.row_units) {
                const int64_t ci = m - n_win + i / c.row_units;        // index inside the chunk
                const int u = static_cast<int>(i % c.row_units);
                const int64_t slot = li * c.window + (n_old + ci) % c.window;
                c.k_ring[slot * c.row_units + u] = kr[j];
                c.v_ring[slot * c.row_units + u] = vr[j];
                if (u == 0) c.score_ring[slot] = scores[ci * c.n_heads + h];
            }
        }
    }
    if (tid == 0) {
        c.prefix_len[li] = static_cast<int32_t>(len_s);
        c.n_tokens[li] = static_cast<int32_t>(n_old + m);
        if (h == 0) c.active[li / (static_cast<int64_t>(c.n_layers) * c.n_heads)] = 1;     // the slot holds a sequence again
    }
}

// A sequence has ended: the pages of all its lists (L x H of them, one warp each) go onto the stack of
// released pages and the lists become empty.  Runs alone on the stream (it is the one kernel that adds
// to the stack).
__global__ void __launch_bounds__(32)
release_seq_kernel(const CacheView c, int32_t seq)
{
    const int64_t li = static_cast<int64_t>(seq) * c.n_layers * c.n_heads + blockIdx.x;
    const int lane = threadIdx.x;
    const int32_t n_pages = (c.prefix_len[li] + c.page_tokens - 1) / c.page_tokens;
    int32_t base = 0;
    if (lane == 0 && n_pages > 0) base = atomicAdd(c.free_top, n_pages);
    base = __shfl_sync(0xffffffffu, base, 0);
    for (int32_t i = lane; i < n_pages; i += 32) c.free_stack[base + i] = c.page_table[li * c.max_pages + i];
    __syncwarp();
    if (lane == 0) {
        c.prefix_len[li] = 0;
        c.n_tokens[li] = 0;
        if (blockIdx.x == 0) c.active[seq] = 0;
    }
}

// no window: only the token count advances
__global__ void tokens_add_kernel(const CacheView c, int64_t li0, int64_t m, const int64_t *__restrict__ list_map,
                                  const int32_t *__restrict__ cu_seqlens)
{
    if (list_map != nullptr) {              // one block per sequence of a batch
        li0 = list_map[blockIdx.x];
        m = cu_seqlens[blockIdx.x + 1] - cu_seqlens[blockIdx.x];
        if (m <= 0) return;
    }
    if (threadIdx.x < c.n_heads) c.n_tokens[li0 + threadIdx.x] += static_cast<int32_t>(m);
    if (threadIdx.x == 0) c.active[li0 / (static_cast<int64_t>(c.n_layers) * c.n_heads)] = 1;
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
