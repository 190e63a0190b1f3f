// Attention of the new token over the pruned cache (Introduction, Criterion 3; Discussion,
// "Implementation Challenges": per-head list lengths differ, so the attention kernel has to take
// variable-length lists).  One CTA per (sequence, layer, KV head) list; the G query heads that share
// the KV head (grouped-query attention) are processed together, so every K and V row is read from
// HBM exactly once per step.  The kernel is bound by those reads.
//
// A list is its paged prefix (prefix_len rows in pages of page_tokens rows) plus the valid slots of
// its window ring; softmax attention does not depend on the order of the rows, so the two parts are
// simply walked one after the other in tiles of 16 rows.  Warp w of the CTA takes tiles w, w + W,
// w + 2W, ... with its own online-softmax state and its own ring of shared-memory stages: lane 0
// issues the TMA loads of a tile (K and V, 128-byte swizzle, two 64-element halves per row when
// D = 128) onto the stage's mbarrier, the warp waits for it, and nothing is shared between warps
// until the end, when the partial (max, sum, output) triples are merged through shared memory.
// When a call has too few lists to keep every SM busy to the end (one layer of a moderate batch, or
// a few long sequences), each list is cut into n_parts equal runs of tiles, one CTA each; the parts
// leave their triples in global memory and the part that arrives last (a counter per list) merges
// them in part order, so the result does not depend on which one that was.
//
// Math per tile, on the warp-level tensor-core path (the work is HBM-bound; 16-row MMAs are enough):
//   S[16 x 16]  = Q[16 x D] K^T      m16n8k16, Q rows 0..G-1 real, the rest zero
//   P           = exp2(S * scale * log2(e) - running max), rows beyond the list's end masked
//   O[16 x D]  += P[16 x 16] V
// Rows of a partly filled tile that lie past the end are excluded from the softmax, and their V
// rows are zeroed in shared memory first (stale pool memory may hold NaN bit patterns).
//
// 8-bit rows (Related work, "Quantization": pruning and quantisation of the cache compose).  A cache whose
// rows are D E4M3 codes followed by a 16-byte trailer (the row's fp32 scale, then 12 unused bytes) is walked
// by the same kernel with kFp8 = true: a tile is 16 whole rows, contiguous in memory, brought in by one
// unswizzled TMA box of full 128-byte lines per K and V, the codes are widened to f16 in registers (one exact conversion per pair) and the MMAs take f16
// operands.  Everything that is not a code is kept inside f16's range by factors applied around the MMAs: a
// query row is divided by the power of two of its largest element (exact; bf16's mantissa fits f16's) and the
// K row scales join that factor on the logits, logit = scale * 2^e * ks_i * (q 2^-e . K8_i); P is multiplied by
// vs_i / vref, vref the largest V scale met so far (the accumulator is rescaled when it grows, together with the
// online softmax's own rescaling, and multiplied by vref at the end), so the second operand lies in [0, 1] and
// is rounded to f16 (11 bits) where the bf16 path rounds P to 8.  The MMA's summation index and the
// output columns may be numbered freely as long as both operands agree, so each lane reads whole 16- or 32-byte
// pieces of a row: for Q K^T lane (n, c) owns bytes [c D/4, (c+1) D/4) of K rows n and n + 8, k-step ks taking
// four of them; the second product is computed transposed, O^T += V^T P^T (P, as the softmax leaves it, is the
// B operand; no accumulator row is wasted on the padding of the query heads to 16), lane (n', c) owning bytes
// [n' D/8, (n'+1) D/8) of V rows 2c, 2c+1, 2c+8, 2c+9.  With rows 144 (or 80) bytes apart these reads have no
// bank conflicts.  Four CTAs fit an SM (128 registers, 56 KB of stages).
#pragma once

#include <cuda_fp16.h>

#include "decode_kernels.cuh"
#include "ptx.cuh"

namespace kvzap {

constexpr int kAttnWarps = 4;
constexpr int kAttnStages = 3;
constexpr int kAttnTileRows = 16;
constexpr int kAttnThreads = kAttnWarps * 32;
constexpr int kAttnMaxGroup = 8;                 // query heads per KV head (rows 0..7 of the 16-row MMA)
constexpr uint32_t kAttnHalfBytes = kAttnTileRows * 128;   // 16 rows x 64 bf16

struct AttnParams {
    CacheView c;
    int32_t layer0, n_layers_call;
    int32_t group;              // G = query heads per KV head, 1..8
    float scale_log2e;          // softmax scale times log2(e)
    const uint16_t *q;          // [n_layers_call][B][H * G][D] bf16
    uint16_t *out;              // same shape
    int32_t *status;
    int32_t n_parts;            // CTAs per list (1 = the CTA writes the output itself)
    float *part_scratch;        // n_parts > 1: [list][part] { m[8], l[8], O[8][D] }
    uint32_t *part_arrive;      // n_parts > 1: [list] parts that have stored their triple; back to 0 after the launch
};

constexpr int kAttnTrailerBytes = 16;            // 8-bit rows: fp32 scale + 12 unused bytes behind the codes
__host__ __device__ constexpr uint32_t attn_stage_bytes(int head_dim, bool fp8 = false)
{
    return fp8 ? 2u * kAttnTileRows * (head_dim + kAttnTrailerBytes) : 2u * (head_dim / 64) * kAttnHalfBytes;
}
__host__ __device__ constexpr uint32_t attn_smem_bytes(int head_dim, bool fp8 = false)
{
    return kAttnWarps * kAttnStages * attn_stage_bytes(head_dim, fp8) + (fp8 ? 128u : 1024u) /* alignment */ + 256u /* barriers */;
}

// four E4M3 codes (a 32-bit word, lowest byte first) -> two packed f16 pairs (exact: f16 holds every E4M3 value)
__device__ __forceinline__ void e4m3x4_to_f16(uint32_t w, uint32_t &lo, uint32_t &hi)
{
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.rn.f16x2.e4m3x2 %0, a;\n\tcvt.rn.f16x2.e4m3x2 %1, b;\n\t}"
        : "=r"(lo), "=r"(hi) : "r"(w));
}
__device__ __forceinline__ float bf16_lo(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t pair) { return __uint_as_float(pair & 0xffff0000u); }

template <int kD, bool kFp8>
__global__ void __launch_bounds__(kAttnThreads, kFp8 ? 4 : 1)
decode_attn_kernel(const __grid_constant__ CUtensorMap tmap_kpool, const __grid_constant__ CUtensorMap tmap_vpool,
                   const __grid_constant__ CUtensorMap tmap_kring, const __grid_constant__ CUtensorMap tmap_vring,
                   const AttnParams p)
{
    constexpr int kHalves = kD / 64;
    constexpr uint32_t kStageBytes = attn_stage_bytes(kD, kFp8);
    constexpr int kRowBytes8 = kD + kAttnTrailerBytes;              // 8-bit rows
    constexpr uint32_t kTileBytes8 = kAttnTileRows * kRowBytes8;
    // accumulator tiles: 16 x 8 pieces of O (rows = query heads, half of them unused) for bf16 rows,
    // 16 x 8 pieces of O^T (rows = elements, columns = query heads) for 8-bit rows
    constexpr int kNTiles = kFp8 ? kD / 16 : kD / 8;
    constexpr uint32_t kAlign = kFp8 ? 128u : 1024u;            // swizzled tiles need 1024-byte alignment
    extern __shared__ uint8_t attn_smem_raw[];
    const uint32_t raw_addr = smem_u32(attn_smem_raw);
    const uint32_t pad = (kAlign - (raw_addr & (kAlign - 1u))) & (kAlign - 1u);
    uint8_t *smem = attn_smem_raw + pad;
    const uint32_t smem_base = raw_addr + pad;
    const uint32_t bars = smem_base + kAttnWarps * kAttnStages * kStageBytes;      // [warp][stage] mbarriers
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kAttnWarps * kAttnStages * kStageBytes + 8 * kAttnWarps * kAttnStages);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const CacheView &c = p.c;
    const int H = c.n_heads, B = c.n_seqs;
    const int list = blockIdx.x / p.n_parts, part = blockIdx.x % p.n_parts;
    const int h = list % H, b = (list / H) % B, l_rel = list / (H * B);
    const int layer = p.layer0 + l_rel;
    const int64_t li = (static_cast<int64_t>(b) * c.n_layers + layer) * H + h;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kAttnWarps * kAttnStages; ++i) mbar_init(bars + 8 * i, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_kpool);
        prefetch_tensormap(&tmap_vpool);
        prefetch_tensormap(&tmap_kring);
        prefetch_tensormap(&tmap_vring);
    }
    __syncthreads();

    const int32_t n_total = __ldcg(c.n_tokens + li);
    const int32_t n_prefix = __ldcg(c.prefix_len + li);
    const int32_t n_ring = c.window > 0 ? (n_total < c.window ? n_total : c.window) : 0;
    const int tiles_per_page = c.page_tokens / kAttnTileRows;
    const int n_pt = (n_prefix + kAttnTileRows - 1) / kAttnTileRows;
    const int n_rt = (n_ring + kAttnTileRows - 1) / kAttnTileRows;
    const int n_tiles_list = n_pt + n_rt;
    // this CTA's run of the list's tiles
    const int t_begin = static_cast<int>(static_cast<int64_t>(n_tiles_list) * part / p.n_parts);
    const int n_tiles = static_cast<int>(static_cast<int64_t>(n_tiles_list) * (part + 1) / p.n_parts);
    const int32_t *pages = c.page_table + li * c.max_pages;

    // the query rows of this KV head as A fragments: row g = lane / 4 (real for g < G), two packed
    // elements at columns 16 ks + 2 (lane % 4) and the same + 8
    const int g = lane >> 2, qc = (lane & 3) * 2;
    const int Hq = H * p.group;
    uint32_t qa[kD / 16][2];
    {
        const uint16_t *qrow = p.q + ((static_cast<int64_t>(l_rel) * B + b) * Hq + h * p.group + g) * kD;
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
            qa[ks][0] = qa[ks][1] = 0u;
            if (g < p.group) {
                if constexpr (kFp8) {      // summation index renumbered: this lane's k-step ks covers columns c D/4 + 4 ks ..+3
                    qa[ks][0] = __ldg(reinterpret_cast<const uint32_t *>(qrow + (lane & 3) * (kD / 4) + ks * 4));
                    qa[ks][1] = __ldg(reinterpret_cast<const uint32_t *>(qrow + (lane & 3) * (kD / 4) + ks * 4 + 2));
                } else {
                    qa[ks][0] = __ldg(reinterpret_cast<const uint32_t *>(qrow + ks * 16 + qc));
                    qa[ks][1] = __ldg(reinterpret_cast<const uint32_t *>(qrow + ks * 16 + 8 + qc));
                }
            }
        }
    }

    float logit_scale = p.scale_log2e;     // 8-bit rows: times the power of two taken out of this lane's query row
    if constexpr (kFp8) {
        float qmax = 0.0f;
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks)
            qmax = fmaxf(fmaxf(qmax, fmaxf(fabsf(bf16_lo(qa[ks][0])), fabsf(bf16_hi(qa[ks][0])))),
                         fmaxf(fabsf(bf16_lo(qa[ks][1])), fabsf(bf16_hi(qa[ks][1]))));
        qmax = fmaxf(qmax, __shfl_xor_sync(0xffffffffu, qmax, 1));
        qmax = fmaxf(qmax, __shfl_xor_sync(0xffffffffu, qmax, 2));       // the four lanes of a row hold all its elements
        uint32_t e = __float_as_uint(qmax) >> 23;                        // biased exponent (qmax >= 0)
        e = e > 253u ? 253u : e;
        const float down = __uint_as_float((254u - e) << 23);            // 2^-(e - 127)
        logit_scale *= __uint_as_float(e << 23);                         // 2^(e - 127); zero for a zero row
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
            qa[ks][0] = pack_f16x2(bf16_lo(qa[ks][0]) * down, bf16_hi(qa[ks][0]) * down);
            qa[ks][1] = pack_f16x2(bf16_lo(qa[ks][1]) * down, bf16_hi(qa[ks][1]) * down);
        }
    }

    float o[kNTiles][4];
#pragma unroll
    for (int i = 0; i < kNTiles; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.0f;
    float m_run = -INFINITY, l_run = 0.0f;
    float vref = 0.0f;                     // 8-bit rows: the largest V scale met so far; o is in units of it

    const uint32_t my_stages = smem_base + warp * kAttnStages * kStageBytes;
    const uint32_t my_bars = bars + 8 * warp * kAttnStages;
    const uint64_t policy = l2_policy_evict_first();

    // first row (in its tensor map) of tile t of this list; needs the page number for prefix tiles
    auto tile_row = [&](int t) -> int32_t {
        if (t < n_pt) {
            const int32_t page = __ldcg(pages + t / tiles_per_page);
            return page * c.page_tokens + (t % tiles_per_page) * kAttnTileRows;
        }
        return static_cast<int32_t>(li * c.window) + (t - n_pt) * kAttnTileRows;
    };
    auto issue = [&](int t, int32_t row, int stage) {
        const uint32_t dst = my_stages + stage * kStageBytes;
        const uint32_t bar = my_bars + 8 * stage;
        const bool prefix = t < n_pt;
        mbar_arrive_expect_tx(bar, kStageBytes);
        if constexpr (kFp8) {
            // a tile of 8-bit rows is one contiguous piece of memory: coordinates (0, 0, tile)
            tma_load_3d(dst, prefix ? &tmap_kpool : &tmap_kring, bar, 0, 0, row / kAttnTileRows, policy);
            tma_load_3d(dst + kTileBytes8, prefix ? &tmap_vpool : &tmap_vring, bar, 0, 0, row / kAttnTileRows, policy);
        } else {
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) {
                tma_load_2d(dst + hf * kAttnHalfBytes, prefix ? &tmap_kpool : &tmap_kring, bar, hf * 64, row, policy);
                tma_load_2d(dst + (kHalves + hf) * kAttnHalfBytes, prefix ? &tmap_vpool : &tmap_vring, bar, hf * 64, row, policy);
            }
        }
    };

    // prologue: fill the stages; row_next belongs to the first tile not yet issued
    int t_issue = t_begin + warp;
    for (int s = 0; s < kAttnStages && t_issue < n_tiles; ++s, t_issue += kAttnWarps) {
        const int32_t row = tile_row(t_issue);
        if (lane == 0) issue(t_issue, row, s);
    }
    int32_t row_next = t_issue < n_tiles ? tile_row(t_issue) : 0;

    bool ok = true;
    int stage = 0;
    uint32_t parity = 0;
    for (int t = t_begin + warp; t < n_tiles; t += kAttnWarps) {
        if (!__all_sync(0xffffffffu, mbar_wait(my_bars + 8 * stage, parity, abort_flag))) {
            ok = false;
            break;
        }
        const uint32_t sK = my_stages + stage * kStageBytes;
        const uint32_t sV = sK + (kFp8 ? kTileBytes8 : kHalves * kAttnHalfBytes);
        const int valid = t < n_pt ? n_prefix - t * kAttnTileRows : n_ring - (t - n_pt) * kAttnTileRows;   // >= 1
        if (valid < kAttnTileRows) {
            // zero the V rows past the end of the list (8-bit rows: codes and scale)
            if constexpr (kFp8) {
                const int n_units = (kAttnTileRows - valid) * (kRowBytes8 / 16);
                for (int i = lane; i < n_units; i += 32)
                    *reinterpret_cast<uint4 *>(smem + (sV - smem_base) + valid * kRowBytes8 + i * 16) = make_uint4(0u, 0u, 0u, 0u);
            } else {
                const int n_units = (kAttnTileRows - valid) * kHalves * 8;
                for (int i = lane; i < n_units; i += 32) {
                    const int r = valid + i / (kHalves * 8), rem = i % (kHalves * 8);
                    *reinterpret_cast<uint4 *>(smem + (sV - smem_base) + (rem >> 3) * kAttnHalfBytes + r * 128 + ((rem & 7) << 4)) =
                        make_uint4(0u, 0u, 0u, 0u);
                }
            }
            fence_proxy_async_smem();
            __syncwarp();
        }

        // ---- S = Q K^T: two 8-row column tiles
        float s0[4] = {0.0f, 0.0f, 0.0f, 0.0f}, s1[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        if constexpr (kFp8) {
            // rows n = lane / 4 and n + 8 of the tile, this lane's D/4 bytes of each
            const uint8_t *kt = smem + (sK - smem_base);
            const uint32_t *r0 = reinterpret_cast<const uint32_t *>(kt + g * kRowBytes8 + (lane & 3) * (kD / 4));
            const uint32_t *r1 = reinterpret_cast<const uint32_t *>(kt + (g + 8) * kRowBytes8 + (lane & 3) * (kD / 4));
            uint32_t w0[kD / 16], w1[kD / 16];
#pragma unroll
            for (int i = 0; i < kD / 64; ++i) {
                const uint4 a = reinterpret_cast<const uint4 *>(r0)[i], b = reinterpret_cast<const uint4 *>(r1)[i];
                w0[4 * i] = a.x; w0[4 * i + 1] = a.y; w0[4 * i + 2] = a.z; w0[4 * i + 3] = a.w;
                w1[4 * i] = b.x; w1[4 * i + 1] = b.y; w1[4 * i + 2] = b.z; w1[4 * i + 3] = b.w;
            }
#pragma unroll
            for (int ks = 0; ks < kD / 16; ++ks) {
                uint32_t k0, k1, k2, k3;
                e4m3x4_to_f16(w0[ks], k0, k1);
                e4m3x4_to_f16(w1[ks], k2, k3);
                mma_f16_16816(s0, qa[ks][0], 0u, qa[ks][1], 0u, k0, k1);
                mma_f16_16816(s1, qa[ks][0], 0u, qa[ks][1], 0u, k2, k3);
            }
            // the K rows' scales: this lane holds columns (rows of the tile) qc, qc + 1 of both column tiles
            s0[0] *= *reinterpret_cast<const float *>(kt + qc * kRowBytes8 + kD);
            s0[1] *= *reinterpret_cast<const float *>(kt + (qc + 1) * kRowBytes8 + kD);
            s1[0] *= *reinterpret_cast<const float *>(kt + (8 + qc) * kRowBytes8 + kD);
            s1[1] *= *reinterpret_cast<const float *>(kt + (9 + qc) * kRowBytes8 + kD);
        } else {
            const int mi = lane >> 3, r8 = lane & 7;
            const int krow = (mi >> 1) * 8 + r8;
#pragma unroll
            for (int ks = 0; ks < kD / 16; ++ks) {
                const int chunk = 2 * ks + (mi & 1);
                const uint32_t addr = sK + (chunk >> 3) * kAttnHalfBytes + krow * 128 + (((chunk & 7) ^ (krow & 7)) << 4);
                uint32_t k0, k1, k2, k3;
                ldmatrix_x4(addr, k0, k1, k2, k3);
                mma_bf16_16816(s0, qa[ks][0], 0u, qa[ks][1], 0u, k0, k1);
                mma_bf16_16816(s1, qa[ks][0], 0u, qa[ks][1], 0u, k2, k3);
            }
        }
        // ---- online softmax for row g: this lane holds columns qc, qc + 1 of both column tiles
        float v00 = s0[0] * logit_scale, v01 = s0[1] * logit_scale;
        float v10 = s1[0] * logit_scale, v11 = s1[1] * logit_scale;
        if (valid < kAttnTileRows) {
            if (qc >= valid) v00 = -INFINITY;
            if (qc + 1 >= valid) v01 = -INFINITY;
            if (8 + qc >= valid) v10 = -INFINITY;
            if (9 + qc >= valid) v11 = -INFINITY;
        }
        float mx = fmaxf(fmaxf(v00, v01), fmaxf(v10, v11));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);             // finite: row 0 of a tile is always valid
        const float alpha = fast_ex2(m_run - m_new);      // 0 on the first tile
        const float p00 = fast_ex2(v00 - m_new), p01 = fast_ex2(v01 - m_new);
        const float p10 = fast_ex2(v10 - m_new), p11 = fast_ex2(v11 - m_new);
        l_run = l_run * alpha + ((p00 + p01) + (p10 + p11));
        m_run = m_new;
        uint32_t pa0, pa2;
        if constexpr (kFp8) {
            // the V rows' scales (zero for rows past the end), relative to the largest one so far
            const uint8_t *vt = smem + (sV - smem_base);
            const float vs00 = *reinterpret_cast<const float *>(vt + qc * kRowBytes8 + kD);
            const float vs01 = *reinterpret_cast<const float *>(vt + (qc + 1) * kRowBytes8 + kD);
            const float vs10 = *reinterpret_cast<const float *>(vt + (8 + qc) * kRowBytes8 + kD);
            const float vs11 = *reinterpret_cast<const float *>(vt + (9 + qc) * kRowBytes8 + kD);
            float vmax = fmaxf(fmaxf(fabsf(vs00), fabsf(vs01)), fmaxf(fabsf(vs10), fabsf(vs11)));
            vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, 1));
            vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, 2));
            const float vref_new = fmaxf(vref, vmax);
            const float rinv = vref_new > 0.0f ? 1.0f / vref_new : 0.0f;
            const float alpha_o = alpha * (vref * rinv);
            vref = vref_new;
            // the accumulator tiles hold O^T: this lane's columns are query heads qc and qc + 1
            const float a_lo = __shfl_sync(0xffffffffu, alpha_o, qc * 4), a_hi = __shfl_sync(0xffffffffu, alpha_o, qc * 4 + 4);
#pragma unroll
            for (int i = 0; i < kNTiles; ++i) { o[i][0] *= a_lo; o[i][1] *= a_hi; o[i][2] *= a_lo; o[i][3] *= a_hi; }
            pa0 = pack_f16x2(p00 * (vs00 * rinv), p01 * (vs01 * rinv));
            pa2 = pack_f16x2(p10 * (vs10 * rinv), p11 * (vs11 * rinv));
        } else {
#pragma unroll
            for (int i = 0; i < kNTiles; ++i) { o[i][0] *= alpha; o[i][1] *= alpha; }
            pa0 = pack_bf16x2(p00, p01);
            pa2 = pack_bf16x2(p10, p11);
        }

        // ---- O += P V: two 8-column output tiles per ldmatrix
        if constexpr (kFp8) {
            // O^T[D x 8] += V^T[D x 16] P^T[16 x 8]: P as it comes out of the softmax is the B operand (k = row of the
            // tile, n = query head), V^T is the A operand.  V rows 2c, 2c+1 (k = 2c, 2c+1) and 2c+8, 2c+9 of the tile,
            // this lane's D/8 bytes of each; accumulator tile i takes bytes 2i (MMA rows 0..7) and 2i+1 (rows 8..15)
            const uint8_t *vt = smem + (sV - smem_base) + g * (kD / 8);
            uint32_t ra[kD / 32], rb[kD / 32], rc[kD / 32], rd[kD / 32];
            if constexpr (kD == 128) {
                const uint4 a = *reinterpret_cast<const uint4 *>(vt + qc * kRowBytes8);
                const uint4 b = *reinterpret_cast<const uint4 *>(vt + (qc + 1) * kRowBytes8);
                const uint4 cc = *reinterpret_cast<const uint4 *>(vt + (qc + 8) * kRowBytes8);
                const uint4 d = *reinterpret_cast<const uint4 *>(vt + (qc + 9) * kRowBytes8);
                ra[0] = a.x; ra[1] = a.y; ra[2] = a.z; ra[3] = a.w;
                rb[0] = b.x; rb[1] = b.y; rb[2] = b.z; rb[3] = b.w;
                rc[0] = cc.x; rc[1] = cc.y; rc[2] = cc.z; rc[3] = cc.w;
                rd[0] = d.x; rd[1] = d.y; rd[2] = d.z; rd[3] = d.w;
            } else {
                const uint2 a = *reinterpret_cast<const uint2 *>(vt + qc * kRowBytes8);
                const uint2 b = *reinterpret_cast<const uint2 *>(vt + (qc + 1) * kRowBytes8);
                const uint2 cc = *reinterpret_cast<const uint2 *>(vt + (qc + 8) * kRowBytes8);
                const uint2 d = *reinterpret_cast<const uint2 *>(vt + (qc + 9) * kRowBytes8);
                ra[0] = a.x; ra[1] = a.y; rb[0] = b.x; rb[1] = b.y;
                rc[0] = cc.x; rc[1] = cc.y; rd[0] = d.x; rd[1] = d.y;
            }
#pragma unroll
            for (int i = 0; i < kNTiles; ++i) {
                const uint32_t sel = (i & 1) ? 0x7362u : 0x5140u;       // bytes k, k+1 of both rows, interleaved (k = 0 or 2)
                uint32_t a0, a1, a2, a3;
                e4m3x4_to_f16(__byte_perm(ra[i >> 1], rb[i >> 1], sel), a0, a1);
                e4m3x4_to_f16(__byte_perm(rc[i >> 1], rd[i >> 1], sel), a2, a3);
                mma_f16_16816(o[i], a0, a1, a2, a3, pa0, pa2);
            }
        } else {
            const int mi = lane >> 3, r8 = lane & 7;
            const int krow = (mi & 1) * 8 + r8;
#pragma unroll
            for (int ndp = 0; ndp < kD / 16; ++ndp) {
                const int chunk = 2 * ndp + (mi >> 1);
                const uint32_t addr = sV + (chunk >> 3) * kAttnHalfBytes + krow * 128 + (((chunk & 7) ^ (krow & 7)) << 4);
                uint32_t v0, v1, v2, v3;
                ldmatrix_x4_trans(addr, v0, v1, v2, v3);
                mma_bf16_16816(o[2 * ndp], pa0, 0u, pa2, 0u, v0, v1);
                mma_bf16_16816(o[2 * ndp + 1], pa0, 0u, pa2, 0u, v2, v3);
            }
        }
        __syncwarp();                                     // all lanes are done with this stage
        if (t_issue < n_tiles) {
            if (lane == 0) issue(t_issue, row_next, stage);
            t_issue += kAttnWarps;
            row_next = t_issue < n_tiles ? tile_row(t_issue) : 0;
        }
        if (++stage == kAttnStages) { stage = 0; parity ^= 1u; }
    }
    if (!ok) {
        // a wait ran out: report it, give the copies already in flight a fixed time to land, merge nothing
        if (lane == 0) {
            atomicCAS(p.status, 0, 5 /* KVZAP_ERR_TIMEOUT */);
            const long long t0 = clock64();
            while (clock64() - t0 < 2000000LL) { }
        }
        __syncwarp();
    }

    // ---- merge the warps' partial results: [warp] { m[8], l[8], O[8][kD] } in the warp's own stages
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    {
        float *mine = reinterpret_cast<float *>(smem + warp * kAttnStages * kStageBytes);
        if ((lane & 3) == 0) { mine[g] = m_run; mine[8 + g] = l_run; }
#pragma unroll
        for (int i = 0; i < kNTiles; ++i) {
            if constexpr (kFp8) {           // O^T: rows are elements g D/8 + 2i (+1), columns query heads qc, qc+1; back from units of vref
                mine[16 + qc * kD + g * (kD / 8) + 2 * i] = o[i][0] * vref;
                mine[16 + (qc + 1) * kD + g * (kD / 8) + 2 * i] = o[i][1] * vref;
                mine[16 + qc * kD + g * (kD / 8) + 2 * i + 1] = o[i][2] * vref;
                mine[16 + (qc + 1) * kD + g * (kD / 8) + 2 * i + 1] = o[i][3] * vref;
            } else {
                mine[16 + g * kD + i * 8 + qc] = o[i][0];
                mine[16 + g * kD + i * 8 + qc + 1] = o[i][1];
            }
        }
    }
    __syncthreads();
    const bool failed = *abort_flag != 0;
    const int64_t out_row0 = (static_cast<int64_t>(l_rel) * B + b) * Hq + h * p.group;
    float *unit = p.n_parts > 1 ? p.part_scratch + (static_cast<int64_t>(list) * p.n_parts + part) * (16 + kAttnMaxGroup * kD) : nullptr;
    for (int idx = threadIdx.x; idx < p.group * kD; idx += kAttnThreads) {
        const int gq = idx / kD, d = idx % kD;
        float m_all = -INFINITY;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w)
            m_all = fmaxf(m_all, reinterpret_cast<const float *>(smem + w * kAttnStages * kStageBytes)[gq]);
        float num = 0.0f, den = 0.0f;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) {
            const float *wp = reinterpret_cast<const float *>(smem + w * kAttnStages * kStageBytes);
            if (wp[gq] > -INFINITY) {                       // a warp that saw no tile contributes nothing
                const float f = fast_ex2(wp[gq] - m_all);
                num += wp[16 + gq * kD + d] * f;
                den += wp[8 + gq] * f;
            }
        }
        if (p.n_parts == 1) {
            const float r = (den > 0.0f && !failed) ? num / den : 0.0f;      // an empty list gives zeros
            p.out[(out_row0 + gq) * kD + d] = static_cast<uint16_t>(pack_bf16x2(r, 0.0f) & 0xffffu);
        } else {
            __stcg(unit + 16 + gq * kD + d, num);
            if (d == 0) {
                __stcg(unit + gq, failed ? -INFINITY : m_all);
                __stcg(unit + 8 + gq, failed ? 0.0f : den);
            }
        }
    }
    if (p.n_parts == 1) return;

    // ---- several CTAs per list: the one that arrives last merges all parts, in part order
    __shared__ int last_s;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t before = atomicAdd(p.part_arrive + list, 1u);
        last_s = before + 1u == static_cast<uint32_t>(p.n_parts);
        if (last_s) p.part_arrive[list] = 0u;               // ready for the next launch
        __threadfence();
    }
    __syncthreads();
    if (!last_s) return;
    const float *units = p.part_scratch + static_cast<int64_t>(list) * p.n_parts * (16 + kAttnMaxGroup * kD);
    constexpr int kBatch = 8;               // parts whose values are loaded together (independent loads in flight)
    constexpr int kUnit = 16 + kAttnMaxGroup * kD;
    for (int idx = threadIdx.x; idx < p.group * kD; idx += kAttnThreads) {
        const int gq = idx / kD, d = idx % kD;
        float m_all = -INFINITY;
        for (int i0 = 0; i0 < p.n_parts; i0 += kBatch) {
            float mv[kBatch];
#pragma unroll
            for (int j = 0; j < kBatch; ++j) mv[j] = i0 + j < p.n_parts ? __ldcg(units + (i0 + j) * kUnit + gq) : -INFINITY;
#pragma unroll
            for (int j = 0; j < kBatch; ++j) m_all = fmaxf(m_all, mv[j]);
        }
        float num = 0.0f, den = 0.0f;
        for (int i0 = 0; i0 < p.n_parts; i0 += kBatch) {
            float mv[kBatch], nv[kBatch], dv[kBatch];
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const bool in = i0 + j < p.n_parts;
                const float *u = units + (i0 + j) * kUnit;
                mv[j] = in ? __ldcg(u + gq) : -INFINITY;
                nv[j] = in ? __ldcg(u + 16 + gq * kD + d) : 0.0f;      // a part without tiles stored zeros
                dv[j] = in ? __ldcg(u + 8 + gq) : 0.0f;
            }
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {                          // summed in part order
                const float f = mv[j] > -INFINITY ? fast_ex2(mv[j] - m_all) : 0.0f;
                num += nv[j] * f;
                den += dv[j] * f;
            }
        }
        const float r = den > 0.0f ? num / den : 0.0f;
        p.out[(out_row0 + gq) * kD + d] = static_cast<uint16_t>(pack_bf16x2(r, 0.0f) & 0xffffu);
    }
}

}  // namespace kvzap
