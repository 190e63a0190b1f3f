/*
 * KVzap CPU oracle -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, obviously-correct restatement of what the KVzap pruning path
 * computes, written from the paper's definition (Method section, "KVzap";
 * Algorithm 1 / Listing 1; Experiments, "KVzap training"; Appendix B).
 * It shares no code, header, table or helper with the CUDA library and is
 * only ever called by the tests, the smoke check and the benchmark's
 * cpu_baseline / reference legs.
 *
 * Arithmetic: every bf16 input is widened exactly to double; products and
 * sums are carried in double in the index order of the definition; one
 * rounding to fp32 at the end.  OpenMP only splits the independent token /
 * head loops across cores.
 *
 * All matrices are row-major.  bf16 values are passed as raw uint16_t bit
 * patterns.  Weight matrices are stored [out, in].
 *
 * Parity pins (tests/test_oracle_*.py): exact rational brute force on tiny
 * inputs, one-hot / zero weights, torch-fp64 library composition, GELU
 * identities, the paper's parameter totals and overhead table, mask and
 * compaction invariants, decode == prefill-on-concatenation.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* exact widening of a bf16 bit pattern (upper half of an IEEE fp32) */
static double bf16_to_double(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int kvzap_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* GELU as used by the MLP surrogate (Experiments, "KVzap training": one hidden
 * layer followed by a GELU).  Exact form: x * Phi(x), Phi the standard normal CDF. */
double kvzap_oracle_gelu(double x)
{
    return 0.5 * x * (1.0 + erf(x / sqrt(2.0)));
}

/*
 * KVzap-Linear (Method, "KVzap"): a per-layer linear map from the hidden state
 * h_t in R^{D_h} to H scores, applied independently at each position t.
 *   scores[t,h] = b[h] + sum_k X[t,k] * W[h,k]
 * X [T,Dh] bf16, W [H,Dh] bf16, b [H] fp32 or NULL (= 0), scores [T,H] fp32.
 */
void kvzap_oracle_score_linear(const uint16_t *X, int64_t T, int Dh,
                               const uint16_t *W, const float *b, int H,
                               float *scores)
{
    int64_t t;
#pragma omp parallel for schedule(static)
    for (t = 0; t < T; ++t) {
        for (int h = 0; h < H; ++h) {
            double acc = b ? (double)b[h] : 0.0;
            for (int k = 0; k < Dh; ++k)
                acc += bf16_to_double(X[t * Dh + k]) * bf16_to_double(W[(int64_t)h * Dh + k]);
            scores[t * H + h] = (float)acc;
        }
    }
}

/*
 * KVzap-MLP (Method, "KVzap"; Experiments, "KVzap training"; Appendix B):
 * two linear layers W1 in R^{D_h x N1}, W2 in R^{N1 x H} with a GELU between.
 *   z[j]        = b1[j] + sum_k X[t,k] * W1[j,k]
 *   g[j]        = GELU(z[j])
 *   scores[t,h] = b2[h] + sum_j g[j] * W2[h,j]
 * W1 [N1,Dh] bf16, b1 [N1] fp32|NULL, W2 [H,N1] bf16, b2 [H] fp32|NULL.
 * Returns 0, or -1 if scratch memory could not be allocated.
 */
int kvzap_oracle_score_mlp(const uint16_t *X, int64_t T, int Dh,
                           const uint16_t *W1, const float *b1, int N1,
                           const uint16_t *W2, const float *b2, int H,
                           float *scores)
{
    /* widen the weights once; W1 is kept as [Dh][N1] so that the hidden units,
     * which are independent sums, sit next to each other in memory */
    double *w1 = (double *)malloc(sizeof(double) * (size_t)Dh * (size_t)N1);
    double *w2 = (double *)malloc(sizeof(double) * (size_t)H * (size_t)N1);
    if (!w1 || !w2) { free(w1); free(w2); return -1; }
    for (int j = 0; j < N1; ++j)
        for (int k = 0; k < Dh; ++k)
            w1[(size_t)k * N1 + j] = bf16_to_double(W1[(size_t)j * Dh + k]);
    for (int h = 0; h < H; ++h)
        for (int j = 0; j < N1; ++j)
            w2[(size_t)h * N1 + j] = bf16_to_double(W2[(size_t)h * N1 + j]);

    int failed = 0;
#pragma omp parallel
    {
        double *z = (double *)malloc(sizeof(double) * (size_t)N1);
        if (!z) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
            int64_t t;
#pragma omp for schedule(static)
            for (t = 0; t < T; ++t) {
                for (int j = 0; j < N1; ++j) z[j] = b1 ? (double)b1[j] : 0.0;
                /* each z[j] accumulates its products in increasing k */
                for (int k = 0; k < Dh; ++k) {
                    const double x = bf16_to_double(X[t * Dh + k]);
                    const double *row = w1 + (size_t)k * N1;
                    for (int j = 0; j < N1; ++j) z[j] += x * row[j];
                }
                for (int j = 0; j < N1; ++j) z[j] = kvzap_oracle_gelu(z[j]);
                for (int h = 0; h < H; ++h) {
                    double acc = b2 ? (double)b2[h] : 0.0;
                    for (int j = 0; j < N1; ++j) acc += z[j] * w2[(size_t)h * N1 + j];
                    scores[t * H + h] = (float)acc;
                }
            }
        }
        free(z);
    }
    free(w1);
    free(w2);
    return failed ? -1 : 0;
}

/*
 * Window + threshold (Algorithm 1: the last `window` positions are forced to
 * +inf, then positions with score >= threshold are kept; Method, "KVzap":
 * pairs whose score falls below tau are discarded; the most recent w tokens
 * are always kept).
 *   keep[h, t] = (t_in_seq >= T_b - w) || (scores[t,h] >= tau)
 * The window is per sequence: sequence b owns packed rows
 * [cu_seqlens[b], cu_seqlens[b+1]).  w = 0 protects nothing; T_b <= w keeps all.
 * The comparison is an ordinary fp32 >= (NaN compares false).
 * scores [T_total,H] fp32; keep [H,T_total] bytes (0/1).
 */
void kvzap_oracle_keep_mask(const float *scores, const int32_t *cu_seqlens, int B,
                            int H, float tau, int w, uint8_t *keep)
{
    const int64_t T_total = cu_seqlens[B];
    for (int b = 0; b < B; ++b) {
        const int64_t t0 = cu_seqlens[b], t1 = cu_seqlens[b + 1];
        const int64_t Tb = t1 - t0;
        for (int h = 0; h < H; ++h) {
            for (int64_t t = t0; t < t1; ++t) {
                const int in_window = (t - t0) >= Tb - (int64_t)w;
                const int above = scores[t * H + h] >= tau;
                keep[(int64_t)h * T_total + t] = (uint8_t)(in_window || above);
            }
        }
    }
}

/*
 * Fixed-budget selection: the alternative that the ablation compares
 * thresholding with (Ablations, "Threshold-based pruning": fixed-ratio top-k
 * selection per head, or per layer as in AdaKV).  The paper only names the two
 * variants; the reading used here: for sequence b the candidates are the
 * positions outside the window, n_cand = max(T_b - w, 0), and the budget is
 * k = ceil(keep_ratio * n_cand) rows per head (computed in double).
 *   per head  (per_layer = 0): list (b,h) keeps its k highest-scoring candidates;
 *   per layer (per_layer = 1): the H*k highest of all H*n_cand candidate scores of
 *                              the sequence are kept, whichever heads they fall on.
 * Both are stated through a cut value: tau_out[b,h] = the k-th largest candidate
 * score of the list (per layer: the (H*k)-th largest over all heads, the same
 * for every h), and keep = in_window || score >= tau_out[b,h].  Scores equal to
 * the cut value are all kept, so ties may take a list past its budget; NaN
 * scores are never candidates; k = 0 gives +inf; fewer than k (non-NaN)
 * candidates give -inf.  The window rule is that of kvzap_oracle_keep_mask.
 * scores [T_total,H] fp32; keep [H,T_total] bytes; tau_out [B,H] fp32.
 * Returns 0, or -1 without memory.
 */
static int cmp_float_desc(const void *a, const void *b)
{
    const float x = *(const float *)a, y = *(const float *)b;
    return (x < y) - (x > y);
}

int kvzap_oracle_topk_mask(const float *scores, const int32_t *cu_seqlens, int B, int H, int w,
                           double keep_ratio, int per_layer, uint8_t *keep, float *tau_out)
{
    const int64_t T_total = cu_seqlens[B];
    float *buf = (float *)malloc(sizeof(float) * (size_t)(T_total > 0 ? T_total : 1) * (size_t)H);
    if (!buf) return -1;
    for (int b = 0; b < B; ++b) {
        const int64_t t0 = cu_seqlens[b], t1 = cu_seqlens[b + 1];
        const int64_t Tb = t1 - t0;
        const int64_t n_cand = Tb - w > 0 ? Tb - w : 0;
        const int64_t k = (int64_t)ceil(keep_ratio * (double)n_cand);
        for (int h = 0; h < H; ++h) {
            if (per_layer && h > 0) {
                tau_out[b * H + h] = tau_out[b * H];
                continue;
            }
            /* the candidate scores of this list (of all heads for the per-layer budget), NaN left out */
            int64_t n = 0;
            for (int64_t t = t0; t < t0 + n_cand; ++t)
                for (int hh = (per_layer ? 0 : h); hh < (per_layer ? H : h + 1); ++hh) {
                    const float v = scores[t * H + hh];
                    if (v == v) buf[n++] = v;
                }
            const int64_t want = per_layer ? k * H : k;
            float tau;
            if (want <= 0) tau = INFINITY;
            else if (n < want) tau = -INFINITY;
            else {
                qsort(buf, (size_t)n, sizeof(float), cmp_float_desc);
                tau = buf[want - 1];
            }
            tau_out[b * H + h] = tau;
        }
        for (int h = 0; h < H; ++h)
            for (int64_t t = t0; t < t1; ++t) {
                const int in_window = (t - t0) >= Tb - (int64_t)w;
                keep[(int64_t)h * T_total + t] = (uint8_t)(in_window || scores[t * H + h] >= tau_out[b * H + h]);
            }
    }
    free(buf);
    return 0;
}

/*
 * Per-(sequence, head) ordered compaction (Algorithm 1: keys[indices],
 * values[indices]; contribution list: per-head compression).
 * For each (b,h) walk the sequence's positions in order and copy row t of K
 * and of V, bytes verbatim, to output slot n++ of that (b,h) list.
 * K,V,K_out,V_out [H,T_total,D] bf16; list (b,h) starts at packed row
 * cu_seqlens[b] of head h in the outputs.  Rows past lengths[b,h] are not
 * written.  lengths [B,H] int32.
 */
void kvzap_oracle_compact(const uint16_t *K, const uint16_t *V, const uint8_t *keep,
                          const int32_t *cu_seqlens, int B, int H, int D,
                          uint16_t *K_out, uint16_t *V_out, int32_t *lengths)
{
    const int64_t T_total = cu_seqlens[B];
    const size_t row_bytes = sizeof(uint16_t) * (size_t)D;
    int bh;
#pragma omp parallel for schedule(static)
    for (bh = 0; bh < B * H; ++bh) {
        const int b = bh / H, h = bh % H;
        const int64_t t0 = cu_seqlens[b], t1 = cu_seqlens[b + 1];
        int64_t n = 0;
        for (int64_t t = t0; t < t1; ++t) {
            if (!keep[(int64_t)h * T_total + t]) continue;
            const int64_t src = ((int64_t)h * T_total + t) * D;
            const int64_t dst = ((int64_t)h * T_total + t0 + n) * D;
            memcpy(K_out + dst, K + src, row_bytes);
            memcpy(V_out + dst, V + src, row_bytes);
            ++n;
        }
        lengths[b * H + h] = (int32_t)n;
    }
}

/*
 * Paged variant of the same compaction.  The paper gives no page format
 * (Discussion, "Implementation Challenges": non-uniform per-head lengths need
 * paged kernels with variable-length blocks), so the reading used here is:
 * a page holds page_tokens rows of K (and a page of the same index in the V
 * pool holds the matching V rows); list (b,h) owns ceil(len/page_tokens)
 * pages, numbered contiguously from first_page in (b,h) order.
 * K_pool,V_pool [n_pages_pool, page_tokens, D] bf16;
 * page_table [B*H, max_pages_per_list] int32 (unused entries left untouched);
 * n_pages_used = total pages assigned.  Returns 0, or -1 if the pool or the
 * table is too small (nothing is then written).
 */
int kvzap_oracle_compact_paged(const uint16_t *K, const uint16_t *V, const uint8_t *keep,
                               const int32_t *cu_seqlens, int B, int H, int D,
                               int page_tokens, int32_t first_page, int64_t n_pages_pool,
                               int max_pages_per_list,
                               uint16_t *K_pool, uint16_t *V_pool, int32_t *page_table,
                               int32_t *lengths, int32_t *n_pages_used)
{
    const int64_t T_total = cu_seqlens[B];
    const size_t row_bytes = sizeof(uint16_t) * (size_t)D;
    /* pass 1: lengths and the page budget */
    int64_t pages = 0;
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            int64_t n = 0;
            for (int64_t t = cu_seqlens[b]; t < cu_seqlens[b + 1]; ++t)
                n += keep[(int64_t)h * T_total + t] ? 1 : 0;
            lengths[b * H + h] = (int32_t)n;
            const int64_t need = (n + page_tokens - 1) / page_tokens;
            if (need > max_pages_per_list) return -1;
            pages += need;
        }
    if ((int64_t)first_page + pages > n_pages_pool) return -1;
    /* pass 2: assign pages in (b,h) order and copy rows */
    int64_t cursor = first_page;
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            const int list = b * H + h;
            const int64_t need = ((int64_t)lengths[list] + page_tokens - 1) / page_tokens;
            for (int64_t p = 0; p < need; ++p)
                page_table[(int64_t)list * max_pages_per_list + p] = (int32_t)(cursor + p);
            int64_t n = 0;
            for (int64_t t = cu_seqlens[b]; t < cu_seqlens[b + 1]; ++t) {
                if (!keep[(int64_t)h * T_total + t]) continue;
                const int64_t page = cursor + n / page_tokens;
                const int64_t dst = (page * page_tokens + n % page_tokens) * D;
                const int64_t src = ((int64_t)h * T_total + t) * D;
                memcpy(K_pool + dst, K + src, row_bytes);
                memcpy(V_pool + dst, V + src, row_bytes);
                ++n;
            }
            cursor += need;
        }
    *n_pages_used = (int32_t)pages;
    return 0;
}

/*
 * The same two compactions with K and V given as the key/value projection
 * writes them, [T_total, H, D] (Discussion, "Implementation Challenges":
 * the surrogate needs only hidden states, so pruning may run before
 * attention, i.e. before a head-major cache exists).  Row (t,h) of the input
 * is at element (t*H + h)*D; outputs, lengths and page numbering are exactly
 * those of kvzap_oracle_compact / kvzap_oracle_compact_paged.
 */
void kvzap_oracle_compact_write(const uint16_t *K_proj, const uint16_t *V_proj, const uint8_t *keep,
                                const int32_t *cu_seqlens, int B, int H, int D,
                                uint16_t *K_out, uint16_t *V_out, int32_t *lengths)
{
    const int64_t T_total = cu_seqlens[B];
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            int64_t n = 0;
            for (int64_t t = cu_seqlens[b]; t < cu_seqlens[b + 1]; ++t) {
                if (!keep[(int64_t)h * T_total + t]) continue;
                const uint16_t *k_row = K_proj + (t * H + h) * (int64_t)D;
                const uint16_t *v_row = V_proj + (t * H + h) * (int64_t)D;
                uint16_t *k_dst = K_out + ((int64_t)h * T_total + cu_seqlens[b] + n) * D;
                uint16_t *v_dst = V_out + ((int64_t)h * T_total + cu_seqlens[b] + n) * D;
                for (int d = 0; d < D; ++d) {
                    k_dst[d] = k_row[d];
                    v_dst[d] = v_row[d];
                }
                ++n;
            }
            lengths[b * H + h] = (int32_t)n;
        }
}

int kvzap_oracle_compact_write_paged(const uint16_t *K_proj, const uint16_t *V_proj, const uint8_t *keep,
                                     const int32_t *cu_seqlens, int B, int H, int D,
                                     int page_tokens, int32_t first_page, int64_t n_pages_pool,
                                     int max_pages_per_list,
                                     uint16_t *K_pool, uint16_t *V_pool, int32_t *page_table,
                                     int32_t *lengths, int32_t *n_pages_used)
{
    const int64_t T_total = cu_seqlens[B];
    int64_t pages = 0;
    for (int list = 0; list < B * H; ++list) {
        const int b = list / H, h = list % H;
        int64_t n = 0;
        for (int64_t t = cu_seqlens[b]; t < cu_seqlens[b + 1]; ++t)
            if (keep[(int64_t)h * T_total + t]) ++n;
        lengths[list] = (int32_t)n;
        const int64_t need = (n + page_tokens - 1) / page_tokens;
        if (need > max_pages_per_list) return -1;
        pages += need;
    }
    if ((int64_t)first_page + pages > n_pages_pool) return -1;
    int64_t next_page = first_page;            /* first page of the list being filled */
    for (int list = 0; list < B * H; ++list) {
        const int b = list / H, h = list % H;
        int64_t n = 0;
        for (int64_t t = cu_seqlens[b]; t < cu_seqlens[b + 1]; ++t) {
            if (!keep[(int64_t)h * T_total + t]) continue;
            const int64_t page = next_page + n / page_tokens;
            if (n % page_tokens == 0) page_table[(int64_t)list * max_pages_per_list + n / page_tokens] = (int32_t)page;
            const int64_t slot = page * page_tokens + n % page_tokens;
            for (int d = 0; d < D; ++d) {
                K_pool[slot * D + d] = K_proj[(t * H + h) * (int64_t)D + d];
                V_pool[slot * D + d] = V_proj[(t * H + h) * (int64_t)D + d];
            }
            ++n;
        }
        next_page += (n + page_tokens - 1) / page_tokens;
    }
    *n_pages_used = (int32_t)pages;
    return 0;
}

/*
 * The consumer of the pruned cache: attention of ONE new token over ONE
 * (sequence, layer, KV head) list of whatever length pruning left
 * (Criterion 3 of the introduction and Discussion, "Implementation
 * Challenges": per-head lengths differ, so the attention kernel must take
 * variable-length lists).  The paper prints no formula of its own; this is
 * the ordinary scaled dot-product softmax attention it refers to:
 *   a[g,i]  = scale * sum_d q[g,d] * K[i,d]
 *   p[g,i]  = exp(a[g,i]) / sum_j exp(a[g,j])
 *   out[g]  = sum_i p[g,i] * V[i]
 * for the G query heads g that share the KV head (grouped-query attention).
 * q [G,D] bf16, K,V [n,D] bf16 (the list's rows, any order: the result does
 * not depend on it), out [G,D] fp32 (one rounding from double).  n = 0 gives
 * zeros.  The largest a[g,.] is subtracted before exp, which changes nothing
 * mathematically and keeps exp in range.  Returns 0, or -1 without memory.
 */
int kvzap_oracle_attention(const uint16_t *q, int G, const uint16_t *K, const uint16_t *V,
                           int64_t n, int D, double scale, float *out)
{
    double *a = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    double *acc = (double *)malloc(sizeof(double) * (size_t)D);
    if (!a || !acc) { free(a); free(acc); return -1; }
    for (int g = 0; g < G; ++g) {
        double a_max = -INFINITY;
        for (int64_t i = 0; i < n; ++i) {
            double dot = 0.0;
            for (int d = 0; d < D; ++d)
                dot += bf16_to_double(q[(int64_t)g * D + d]) * bf16_to_double(K[i * D + d]);
            a[i] = scale * dot;
            if (a[i] > a_max) a_max = a[i];
        }
        double denom = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            a[i] = exp(a[i] - a_max);
            denom += a[i];
        }
        for (int d = 0; d < D; ++d) acc[d] = 0.0;
        for (int64_t i = 0; i < n; ++i)
            for (int d = 0; d < D; ++d)
                acc[d] += a[i] * bf16_to_double(V[i * D + d]);
        for (int d = 0; d < D; ++d)
            out[(int64_t)g * D + d] = n > 0 ? (float)(acc[d] / denom) : 0.0f;
    }
    free(a);
    free(acc);
    return 0;
}

/*
 * Closed forms of Appendix B (per token, per layer).
 *   C        = 4 D_h (H_Q D + H D) + 6 D_h D_int      linear-projection FLOPs of a layer
 *   C_MLP    = 2 D_h (D_h/8) + 2 (D_h/8) H = D_h/4 (D_h + H)
 *   C_Linear = 2 D_h H
 */
double kvzap_oracle_layer_flops(int H_Q, int H, int D, int Dh, int D_int)
{
    return 4.0 * Dh * ((double)H_Q * D + (double)H * D) + 6.0 * (double)Dh * D_int;
}

double kvzap_oracle_mlp_flops(int Dh, int N1, int H)
{
    return 2.0 * (double)Dh * N1 + 2.0 * (double)N1 * H;
}

double kvzap_oracle_linear_flops(int Dh, int H)
{
    return 2.0 * (double)Dh * H;
}

/* parameter count of one layer's surrogate, biases included; N1 = 0 means Linear */
int64_t kvzap_oracle_param_count(int Dh, int N1, int H)
{
    if (N1 == 0) return (int64_t)Dh * H + H;
    return (int64_t)Dh * N1 + N1 + (int64_t)N1 * H + H;
}

/*
 * Write plan (Discussion, "Implementation Challenges": since the surrogate
 * needs only hidden states, pruning can be applied before attention, i.e. before
 * the keys and values are stored).  Instead of moving rows, the plan tells
 * whoever produces K and V where each row belongs:
 *   slot[t,h] = n, the number of kept positions of list (b,h) before t, if keep[h,t]
 *             = -1 if the pair is dropped
 * so that writing row t of head h to row cu_seqlens[b] + slot of head h gives
 * exactly kvzap_oracle_compact's output.  Paged (page_tokens > 0): the page
 * assignment is that of kvzap_oracle_compact_paged and the slot is the pool row,
 *   slot[t,h] = (first page of list (b,h) + n / page_tokens) * page_tokens + n % page_tokens.
 * slot [T_total,H] int32; lengths [B,H]; page_table / n_pages_used as in
 * kvzap_oracle_compact_paged (ignored when page_tokens == 0).
 * Returns 0, or -1 if the pool or the table is too small (slot is then all -1).
 */
int kvzap_oracle_plan(const uint8_t *keep, const int32_t *cu_seqlens, int B, int H,
                      int page_tokens, int32_t first_page, int64_t n_pages_pool, int max_pages_per_list,
                      int32_t *slot, int32_t *page_table, int32_t *lengths, int32_t *n_pages_used)
{
    const int64_t T_total = cu_seqlens[B];
    for (int64_t i = 0; i < T_total * H; ++i) slot[i] = -1;
    int64_t pages = 0;
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            int64_t n = 0;
            for (int64_t t = cu_seqlens[b]; t < cu_seqlens[b + 1]; ++t)
                n += keep[(int64_t)h * T_total + t] ? 1 : 0;
            lengths[b * H + h] = (int32_t)n;
            if (page_tokens > 0) {
                const int64_t need = (n + page_tokens - 1) / page_tokens;
                if (need > max_pages_per_list) return -1;
                pages += need;
            }
        }
    if (page_tokens > 0 && (int64_t)first_page + pages > n_pages_pool) return -1;
    int64_t cursor = first_page;
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            const int list = b * H + h;
            int64_t n = 0;
            for (int64_t t = cu_seqlens[b]; t < cu_seqlens[b + 1]; ++t) {
                if (!keep[(int64_t)h * T_total + t]) continue;
                if (page_tokens > 0)
                    slot[t * H + h] = (int32_t)((cursor + n / page_tokens) * page_tokens + n % page_tokens);
                else
                    slot[t * H + h] = (int32_t)n;
                ++n;
            }
            if (page_tokens > 0) {
                const int64_t need = (n + page_tokens - 1) / page_tokens;
                int32_t *row = page_table + (int64_t)list * max_pages_per_list;
                for (int64_t i = 0; i < need; ++i) row[i] = (int32_t)(cursor + i);
                cursor += need;
            }
        }
    if (page_tokens > 0) *n_pages_used = (int32_t)pages;
    return 0;
}

/*
 * 8-bit floating point inputs (Related work, "Quantization": pruning composes
 * with quantisation of the cache; the paper fixes no format).  The reading
 * used here is the OCP 8-bit format E4M3 in its finite variant: 1 sign bit,
 * 4 exponent bits with bias 7, 3 mantissa bits; exponent field 0 holds the
 * subnormals m/8 * 2^-6; there are no infinities; only S.1111.111 is NaN, so
 * the largest magnitude is 1.75 * 2^8 = 448.  Exact widening to double:
 */
double kvzap_oracle_e4m3_to_double(uint8_t bits)
{
    const int sign = bits >> 7, e = (bits >> 3) & 15, m = bits & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/*
 * KVzap-Linear on quantised inputs: hidden states X8 [T,Dh] and weights W8 [H,Dh]
 * as E4M3 bytes, with one fp32 scale per token (x_scale [T], NULL = 1) and one
 * per output row (w_scale [H], NULL = 1) -- the usual per-token / per-channel
 * scaling; the paper gives none.
 *   scores[t,h] = b[h] + x_scale[t] * w_scale[h] * sum_k X8[t,k] * W8[h,k]
 */
void kvzap_oracle_score_linear_fp8(const uint8_t *X8, const float *x_scale, int64_t T, int Dh,
                                   const uint8_t *W8, const float *w_scale, const float *b, int H,
                                   float *scores)
{
    int64_t t;
#pragma omp parallel for schedule(static)
    for (t = 0; t < T; ++t) {
        for (int h = 0; h < H; ++h) {
            double acc = 0.0;
            for (int k = 0; k < Dh; ++k)
                acc += kvzap_oracle_e4m3_to_double(X8[t * Dh + k]) * kvzap_oracle_e4m3_to_double(W8[(int64_t)h * Dh + k]);
            const double sx = x_scale ? (double)x_scale[t] : 1.0, sw = w_scale ? (double)w_scale[h] : 1.0;
            scores[t * H + h] = (float)((b ? (double)b[h] : 0.0) + sx * sw * acc);
        }
    }
}

/*
 * KVzap-MLP on quantised inputs: the first layer as above (X8, W18 [N1,Dh] E4M3,
 * x_scale [T], w1_scale [N1]); GELU and the second layer (W2 [H,N1] bf16) unchanged.
 *   z[j] = b1[j] + x_scale[t] * w1_scale[j] * sum_k X8[t,k] * W18[j,k]
 *   scores[t,h] = b2[h] + sum_j GELU(z[j]) * W2[h,j]
 * Returns 0, or -1 without memory.
 */
int kvzap_oracle_score_mlp_fp8(const uint8_t *X8, const float *x_scale, int64_t T, int Dh,
                               const uint8_t *W18, const float *w1_scale, const float *b1, int N1,
                               const uint16_t *W2, const float *b2, int H, float *scores)
{
    double *w1 = (double *)malloc(sizeof(double) * (size_t)Dh * (size_t)N1);
    if (!w1) return -1;
    for (int j = 0; j < N1; ++j)
        for (int k = 0; k < Dh; ++k)
            w1[(size_t)k * N1 + j] = kvzap_oracle_e4m3_to_double(W18[(size_t)j * Dh + k]);
    int failed = 0;
#pragma omp parallel
    {
        double *z = (double *)malloc(sizeof(double) * (size_t)N1);
        if (!z) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
            int64_t t;
#pragma omp for schedule(static)
            for (t = 0; t < T; ++t) {
                for (int j = 0; j < N1; ++j) z[j] = 0.0;
                for (int k = 0; k < Dh; ++k) {
                    const double x = kvzap_oracle_e4m3_to_double(X8[t * Dh + k]);
                    const double *row = w1 + (size_t)k * N1;
                    for (int j = 0; j < N1; ++j) z[j] += x * row[j];
                }
                const double sx = x_scale ? (double)x_scale[t] : 1.0;
                for (int j = 0; j < N1; ++j) {
                    const double sw = w1_scale ? (double)w1_scale[j] : 1.0;
                    z[j] = kvzap_oracle_gelu((b1 ? (double)b1[j] : 0.0) + sx * sw * z[j]);
                }
                for (int h = 0; h < H; ++h) {
                    double sum = 0.0;
                    for (int j = 0; j < N1; ++j) sum += z[j] * bf16_to_double(W2[(size_t)h * N1 + j]);
                    scores[t * H + h] = (float)((b2 ? (double)b2[h] : 0.0) + sum);
                }
            }
        }
        free(z);
    }
    free(w1);
    return failed ? -1 : 0;
}

/*
 * kvzap_oracle_attention over a list whose rows are stored quantised (Related
 * work, "Quantization"): K8, V8 [n,D] E4M3 bytes with one fp32 scale per row
 * (k_scale, v_scale [n], NULL = 1), so that row i stands for k_scale[i] * K8[i]
 * and v_scale[i] * V8[i]; q [G,D] stays bf16.
 *   a[g,i] = scale * k_scale[i] * sum_d q[g,d] * K8[i,d]
 *   out[g] = sum_i softmax_i(a[g,.]) * v_scale[i] * V8[i]
 * Returns 0, or -1 without memory.
 */
int kvzap_oracle_attention_fp8(const uint16_t *q, int G, const uint8_t *K8, const float *k_scale,
                               const uint8_t *V8, const float *v_scale, int64_t n, int D, double scale,
                               float *out)
{
    double *a = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    double *acc = (double *)malloc(sizeof(double) * (size_t)D);
    if (!a || !acc) { free(a); free(acc); return -1; }
    for (int g = 0; g < G; ++g) {
        double a_max = -INFINITY;
        for (int64_t i = 0; i < n; ++i) {
            double dot = 0.0;
            for (int d = 0; d < D; ++d)
                dot += bf16_to_double(q[(int64_t)g * D + d]) * kvzap_oracle_e4m3_to_double(K8[i * D + d]);
            a[i] = scale * (k_scale ? (double)k_scale[i] : 1.0) * dot;
            if (a[i] > a_max) a_max = a[i];
        }
        double denom = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            a[i] = exp(a[i] - a_max);
            denom += a[i];
        }
        for (int d = 0; d < D; ++d) acc[d] = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            const double sv = v_scale ? (double)v_scale[i] : 1.0;
            for (int d = 0; d < D; ++d)
                acc[d] += a[i] * sv * kvzap_oracle_e4m3_to_double(V8[i * D + d]);
        }
        for (int d = 0; d < D; ++d) {
            const double o = n > 0 ? acc[d] / denom : 0.0;
            out[(int64_t)g * D + d] = (float)o;
        }
    }
    free(a);
    free(acc);
    return 0;
}
