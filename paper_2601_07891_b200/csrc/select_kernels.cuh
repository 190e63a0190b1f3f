// Fixed-budget selection (Ablations, "Threshold-based pruning": top-k per head, or per layer as in
// AdaKV, the alternatives thresholding is compared with).  Both are reduced to the path that already
// exists: find the cut value tau*[b,h] -- the k-th largest candidate score of list (b,h), or the
// (H*k)-th largest over all heads of sequence b -- and then run the usual window + threshold mask and
// compaction with that per-list threshold.  Candidates are the positions outside the window; scores
// equal to the cut value are all kept; NaN scores are never candidates.
//
// The cut value comes from a radix select over order-preserving 32-bit keys, 8 bits per pass:
// pass p histograms the byte p (from the top) of every candidate key that matches the bytes already
// fixed.  Histograms of all four passes live in global memory (zeroed by the host before the first
// pass); each CTA re-derives the bytes fixed so far from the earlier passes' histograms (at most three
// 256-bin scans), so a pass is one launch and no kernel ever waits for another.
#pragma once

#include "score_kernel.cuh"

namespace kvzap {

constexpr int kSelectThreads = 256;      // 8 warps: warp i derives the state of head i

// larger score <-> larger key; -0 sorts below +0, NaN is never turned into a key
__device__ __forceinline__ uint32_t score_key(float v)
{
    const uint32_t u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_score(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Whole warp: walking the 256 bins from the top, the bin that holds the k-th key (k >= 1); `above` =
// keys in higher bins.  Returns 256 when all bins together hold fewer than k keys.
__device__ __forceinline__ uint32_t select_bin(const uint32_t *hist, uint32_t k, uint32_t &above, int lane)
{
    uint32_t c[8], mine = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        c[i] = __ldcg(hist + 8 * lane + i);
        mine += c[i];
    }
    uint32_t incl = mine;                 // becomes the count in this lane's bins and all higher lanes'
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_down_sync(0xffffffffu, incl, o);
        if (lane + o < 32) incl += y;
    }
    const uint32_t higher = incl - mine;
    uint32_t bin = 256u, ab = 0u;
    if (higher < k && k <= incl) {
        uint32_t run = higher;
#pragma unroll
        for (int i = 7; i >= 0; --i) {
            if (bin == 256u) {
                if (run + c[i] >= k) { bin = 8u * lane + i; ab = run; }
                else run += c[i];
            }
        }
    }
    const uint32_t found = __ballot_sync(0xffffffffu, bin != 256u);
    if (found == 0u) { above = 0u; return 256u; }
    const int src = __ffs(found) - 1;
    above = __shfl_sync(0xffffffffu, ab, src);
    return __shfl_sync(0xffffffffu, bin, src);
}

struct SelectState {
    uint32_t prefix;      // the key bytes fixed by the passes before `pass`
    uint32_t k_rem;       // rank still to find among the keys that share them
    int dead;             // 1: fewer candidates than the budget (cut value -inf), nothing to histogram
};

// Whole warp: state of one (sequence, head-or-layer) selection before pass `pass`.
// hist points at [pass][...][256] for this selection with `pass_stride` words between passes.
__device__ __forceinline__ SelectState select_state(const uint32_t *hist, int64_t pass_stride, int pass, uint32_t k, int lane)
{
    SelectState s{0u, k, 0};
    for (int q = 0; q < pass; ++q) {
        uint32_t above;
        const uint32_t bin = select_bin(hist + q * pass_stride, s.k_rem, above, lane);
        if (bin == 256u) { s.dead = 1; break; }
        s.prefix = (s.prefix << 8) | bin;
        s.k_rem -= above;
    }
    return s;
}

__device__ __forceinline__ uint32_t select_budget(float keep_ratio, int64_t n_cand, int per_layer, int n_heads, bool &too_many)
{
    const double k = ceil(static_cast<double>(keep_ratio) * static_cast<double>(n_cand));
    const double total = per_layer ? k * n_heads : k;
    too_many = total > 4294967295.0;
    return too_many ? 0xffffffffu : static_cast<uint32_t>(total);
}

// grid (ceil(n_tokens / 256), n_seqs); hist [4][n_seqs][n_sel][256], n_sel = per_layer ? 1 : n_heads
__global__ void __launch_bounds__(kSelectThreads)
select_hist_kernel(const float *__restrict__ scores, int64_t n_tokens, int n_heads, const int32_t *__restrict__ cu_seqlens,
                   int n_seqs, int window, float keep_ratio, int per_layer, int pass, uint32_t *__restrict__ hist)
{
    __shared__ uint32_t sh[kMaxHeads][256];
    __shared__ uint32_t s_prefix[kMaxHeads];
    __shared__ int s_dead[kMaxHeads];
    // the launches of one selection are queued with early start: each lets the next be placed at once and
    // waits here, every thread, for the one ahead (its histograms, or the scores) to be complete
    griddep_launch_dependents();
    griddep_wait();
    const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t t0 = cu_seqlens ? cu_seqlens[b] : 0, t1 = cu_seqlens ? cu_seqlens[b + 1] : n_tokens;
    const int64_t n_cand = t1 - t0 - window > 0 ? t1 - t0 - window : 0;
    const int64_t c0 = static_cast<int64_t>(blockIdx.x) * kSelectThreads;
    if (c0 >= n_cand) return;
    bool too_many;
    const uint32_t k = select_budget(keep_ratio, n_cand, per_layer, n_heads, too_many);
    if (k == 0u) return;                                  // the cut value is +inf whatever the scores
    const int n_sel = per_layer ? 1 : n_heads;
    const int64_t pass_stride = static_cast<int64_t>(n_seqs) * n_sel * 256;
    for (int i = tid; i < kMaxHeads * 256; i += kSelectThreads) (&sh[0][0])[i] = 0u;
    if (warp < n_sel) {
        const SelectState s = select_state(hist + (static_cast<int64_t>(b) * n_sel + warp) * 256, pass_stride, pass, k, lane);
        if (lane == 0) { s_prefix[warp] = s.prefix; s_dead[warp] = s.dead; }
    }
    __syncthreads();
    if (c0 + tid < n_cand) {
        const float *row = scores + (t0 + c0 + tid) * n_heads;
        for (int h = 0; h < n_heads; ++h) {
            const int hs = per_layer ? 0 : h;
            const float v = __ldcg(row + h);
            if (s_dead[hs] || v != v) continue;
            const uint32_t key = score_key(v);
            if (pass == 0 || (key >> (32 - 8 * pass)) == s_prefix[hs])
                atomicAdd(&sh[hs][(key >> (24 - 8 * pass)) & 255u], 1u);
        }
    }
    __syncthreads();
    uint32_t *out = hist + pass * pass_stride + static_cast<int64_t>(b) * n_sel * 256;
    for (int i = tid; i < n_sel * 256; i += kSelectThreads) {
        const uint32_t v = sh[i >> 8][i & 255];
        if (v) atomicAdd(out + i, v);
    }
}

// grid n_seqs; writes the cut values tau_list [n_seqs][n_heads]
__global__ void __launch_bounds__(kSelectThreads)
select_finish_kernel(int64_t n_tokens, int n_heads, const int32_t *__restrict__ cu_seqlens, int n_seqs, int window,
                     float keep_ratio, int per_layer, const uint32_t *__restrict__ hist, float *__restrict__ tau_list,
                     int32_t *__restrict__ status)
{
    griddep_launch_dependents();
    griddep_wait();
    const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t t0 = cu_seqlens ? cu_seqlens[b] : 0, t1 = cu_seqlens ? cu_seqlens[b + 1] : n_tokens;
    const int64_t n_cand = t1 - t0 - window > 0 ? t1 - t0 - window : 0;
    bool too_many;
    const uint32_t k = select_budget(keep_ratio, n_cand, per_layer, n_heads, too_many);
    if (too_many && threadIdx.x == 0) atomicCAS(status, 0, 2 /* KVZAP_ERR_UNSUPPORTED */);
    const int n_sel = per_layer ? 1 : n_heads;
    if (warp >= n_sel) return;
    float tau = INFINITY;
    if (k > 0u) {
        const int64_t pass_stride = static_cast<int64_t>(n_seqs) * n_sel * 256;
        const SelectState s = select_state(hist + (static_cast<int64_t>(b) * n_sel + warp) * 256, pass_stride, 4, k, lane);
        tau = s.dead ? -INFINITY : key_score(s.prefix);
    }
    if (per_layer) {
        for (int h = lane; h < n_heads; h += 32) tau_list[b * n_heads + h] = tau;
    } else if (lane == 0) {
        tau_list[b * n_heads + warp] = tau;
    }
}

}  // namespace kvzap
