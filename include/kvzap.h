/*
 * kvzap.h -- C ABI of the KVzap pruning hot path for NVIDIA B200 (sm_100a).
 *
 * KVzap (Method section, "KVzap"; Algorithm 1) prunes a transformer layer's
 * KV cache per KV head: a small per-layer surrogate (a linear map, or a
 * two-layer MLP with a GELU) turns each token's hidden state into one
 * log-importance score per KV head; a key/value pair is discarded when its
 * score is below a fixed threshold tau, except that the most recent w tokens
 * are always kept; the kept keys and values of every (sequence, head) are
 * gathered, in token order, into a list whose length differs from head to
 * head.
 *
 * General conventions
 *   - Every tensor argument is a DEVICE pointer owned by the caller, unless a
 *     comment says "host".  The library owns only its context (a private
 *     copy of the surrogate weights and a few MB of scratch).
 *   - bf16 tensors are passed as `const void*` (raw 16-bit patterns),
 *     row-major, innermost dimension last.  Pointers must be 16-byte aligned.
 *   - `stream` is a cudaStream_t passed as `void*` (NULL = default stream).
 *     Calls enqueue work on it and return without synchronising.  A context
 *     must not be used from two streams at the same time: its scratch is
 *     shared by all calls.
 *   - Work of consecutive calls on one stream may overlap on the GPU: the kernels
 *     are launched so that a scoring kernel can start on SMs that the previous
 *     call's kernels have already left, and the compaction of one call runs
 *     beside the scoring kernel of the next.  This is invisible to stream
 *     order: every output of a call is complete before any later operation on
 *     the stream (a copy, another library's kernel, an event) starts.
 *     By default a call's first kernel still waits, before it reads any caller
 *     data, until everything ahead of it in the stream has completed; so any
 *     producer of the inputs is safe, including library kernels that signal
 *     "dependents may start" before their last store (only launch latency is
 *     overlapped then).  KVZAP_FLAG_TRUSTED_PRODUCERS in kvzap_config.flags
 *     drops that wait and gives the full overlap; the caller then guarantees:
 *     (1) inputs of a call (hidden states, K, V) are complete in stream order
 *     before the PREVIOUS kvzap call on that stream was enqueued, or are
 *     produced by an ordinary kernel or copy enqueued between the two calls
 *     that does not itself signal early.  (2) Passing the same scores buffer
 *     to two consecutive calls is allowed in either mode; the library then
 *     launches the second call's scoring kernel without overlap of its stores.
 *   - Stream capture (CUDA graphs): kvzap_decode_step(_fp8) and kvzap_decode_attention(_fp8) may be captured
 *     and replayed.  The other calls rotate scratch sets and counters on the host from call to call and must
 *     be enqueued, not captured.
 *   - Errors the host can see (bad argument, unsupported shape) return at once
 *     and launch nothing.  Conditions only the device can see set a status
 *     word that kvzap_poll_status() reads; kernels never trap and every
 *     device-side wait is bounded.
 *   - Token packing: a batch of B sequences is passed packed along the token
 *     axis; `cu_seqlens` (device, int32 [B+1], cu_seqlens[0] = 0,
 *     cu_seqlens[B] = n_tokens) gives each sequence's rows.  NULL means one
 *     sequence of n_tokens.
 */
#ifndef KVZAP_H_
#define KVZAP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    KVZAP_OK = 0,
    KVZAP_ERR_INVALID_ARG = 1,   /* null pointer, negative size, out-of-range layer, ...        */
    KVZAP_ERR_UNSUPPORTED = 2,   /* shape outside the limits listed at kvzap_create             */
    KVZAP_ERR_CUDA = 3,          /* a CUDA runtime/driver call failed; see kvzap_last_error     */
    KVZAP_ERR_OOM_PAGES = 4,     /* device side: page pool or page table exhausted              */
    KVZAP_ERR_TIMEOUT = 5,       /* device side: a bounded wait inside a kernel expired         */
    KVZAP_ERR_STATE = 6          /* call order violated, e.g. scoring a layer without weights   */
} kvzap_status;

typedef struct kvzap_ctx kvzap_ctx;

/*
 * Shapes of one model's surrogate and cache (Experiments, "KVzap training":
 * input size D_h, one hidden layer of width D_h/8 for the MLP, H outputs;
 * Introduction: cache of shape (2, L, H, T, D)).
 */
typedef struct {
    int32_t d_model;      /* D_h; multiple of 64, 64..16384                                     */
    int32_t hidden;       /* 0 = KVzap-Linear; else MLP hidden width N1: multiple of 64 up to
                             512, or a multiple of 128 up to 1024                               */
    int32_t n_kv_heads;   /* H, 1..8                                                            */
    int32_t head_dim;     /* D; multiple of 8 (rows are whole 16-byte units), 8..1024           */
    int32_t n_layers;     /* L >= 1: number of per-layer surrogates held by the context         */
    int32_t device;       /* CUDA device ordinal                                                */
    int64_t max_tokens;   /* largest n_tokens any call will pass (sizes the scratch)            */
    int32_t max_seqs;     /* largest number of sequences in one call (>= 1)                     */
    int32_t flags;        /* 0, or KVZAP_FLAG_* values or-ed together                           */
} kvzap_config;

/* The caller vouches for whatever produces the inputs of its calls (see "Work of consecutive calls"
 * above): kernels of a call may read caller data before the work ahead in the stream has completed. */
#define KVZAP_FLAG_TRUSTED_PRODUCERS 1

/* Creates a context on cfg->device (allocates weights storage and scratch with
 * cudaMalloc; synchronous).  *out is NULL on failure. */
kvzap_status kvzap_create(kvzap_ctx **out, const kvzap_config *cfg);

/* Synchronises the device, frees everything the context owns.  NULL is allowed. */
kvzap_status kvzap_destroy(kvzap_ctx *ctx);

/* Message of the last failing call on this context ("" if none).  The string is
 * owned by the context and valid until the next call on it.  With ctx == NULL
 * returns the message of the last failing kvzap_create of this process. */
const char *kvzap_last_error(const kvzap_ctx *ctx);

/*
 * Installs one layer's surrogate (Method, "KVzap": a linear layer or a
 * two-layer MLP; Appendix B: W1 in R^{D_h x D_h/8}, W2 in R^{D_h/8 x H}).
 * Matrices are bf16, stored [out, in] row-major, 16-byte aligned; biases are fp32, NULL = zero.
 *   KVzap-Linear (cfg.hidden == 0): W1 [H, d_model], b1 [H]; W2 and b2 must be NULL.
 *   KVzap-MLP:                      W1 [hidden, d_model], b1 [hidden],
 *                                   W2 [H, hidden],       b2 [H].
 * The context keeps its own repacked copy (copy kernels run on `stream`); the
 * caller's buffers may be freed once that stream work has completed.
 */
kvzap_status kvzap_set_weights(kvzap_ctx *ctx, int32_t layer,
                               const void *W1, const float *b1,
                               const void *W2, const float *b2, void *stream);

/*
 * Surrogate scoring (Method, "KVzap"; Algorithm 1, the scoring step): maps each
 * hidden state h_t to H scores, independently per position.
 *   Linear: scores[t,h] = b1[h] + sum_k hidden[t,k] W1[h,k]
 *   MLP:    scores[t,h] = b2[h] + sum_j GELU(b1[j] + sum_k hidden[t,k] W1[j,k]) W2[h,j]
 * GELU is the exact (erf) form.  bf16 products are accumulated in fp32.
 *   hidden [n_tokens, d_model] bf16 (in)   scores [n_tokens, H] fp32 (out)
 * n_tokens may be 0 (nothing is launched) and need not be a multiple of anything.
 */
kvzap_status kvzap_score(kvzap_ctx *ctx, int32_t layer, const void *hidden, int64_t n_tokens,
                         float *scores, void *stream);

/*
 * 8-bit floating point inputs (Related work, "Quantization": pruning composes with quantisation; the paper
 * fixes no format).  Format used here: OCP E4M3 in its finite variant (1 sign, 4 exponent bits with bias 7, 3
 * mantissa bits, no infinities, S.1111.111 = NaN), one fp32 scale per token for the hidden states and one per
 * output row for the first-layer weights -- a value stands for scale * E4M3(byte).  The first layer then runs
 * on the tensor cores' 8-bit path (twice the bf16 rate, half the bytes per hidden state):
 *   Linear: scores[t,h] = b1[h] + x_scale[t] * w1_scale[h] * sum_k X8[t,k] W8[h,k]
 *   MLP:    z[j] = b1[j] + x_scale[t] * w1_scale[j] * sum_k X8[t,k] W8[j,k];  scores as kvzap_score from z
 * kvzap_set_weights_fp8: W1_e4m3 [rows, d_model] bytes (rows = H or hidden), w1_scale [rows] fp32 (NULL = 1),
 * b1, W2 (bf16), b2 as in kvzap_set_weights.  A layer holds either kind of weights; the calls of the other
 * kind return KVZAP_ERR_STATE for it.  d_model must be a multiple of 128 (else KVZAP_ERR_UNSUPPORTED).
 * kvzap_score_fp8 / kvzap_prefill_fused_fp8: hidden_e4m3 [n_tokens, d_model] bytes (device, 16-byte aligned),
 * x_scale [n_tokens] fp32 (device, NULL = 1); everything else as kvzap_score / kvzap_prefill_fused (K and V stay
 * bf16 rows, or any rows of head_dim * 2 bytes: the compaction copies bytes).
 */
kvzap_status kvzap_set_weights_fp8(kvzap_ctx *ctx, int32_t layer, const void *W1_e4m3, const float *w1_scale,
                                   const float *b1, const void *W2, const float *b2, void *stream);
kvzap_status kvzap_score_fp8(kvzap_ctx *ctx, int32_t layer, const void *hidden_e4m3, const float *x_scale,
                             int64_t n_tokens, float *scores, void *stream);
kvzap_status kvzap_prefill_fused_fp8(kvzap_ctx *ctx, int32_t layer, const void *hidden_e4m3, const float *x_scale,
                                     const void *K, const void *V,
                                     const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                     float tau, int32_t w,
                                     void *K_out, void *V_out, int32_t *lengths,
                                     float *scores_out, void *stream);

/* The same into pages (arguments as kvzap_prefill_fused_paged, hidden states and x_scale as above). */
kvzap_status kvzap_prefill_fused_paged_fp8(kvzap_ctx *ctx, int32_t layer, const void *hidden_e4m3, const float *x_scale,
                                           const void *K, const void *V, const int32_t *cu_seqlens, int32_t n_seqs,
                                           int64_t n_tokens, float tau, int32_t w, void *K_pool, void *V_pool,
                                           int64_t n_pages_pool, int32_t page_tokens, int32_t first_page, int32_t *page_table,
                                           int32_t max_pages_per_list, int32_t *lengths, int32_t *n_pages_used,
                                           float *scores_out, void *stream);

/*
 * Threshold + sliding window + per-(sequence, head) ordered compaction
 * (Algorithm 1, the steps after scoring; Method, "KVzap": pairs whose score falls below tau
 * are discarded, the most recent w tokens are kept).
 *   keep[b,h,t] = (t >= T_b - w) || (scores[t,h] >= tau)        (fp32 compare; NaN is not kept)
 * with t counted inside sequence b of length T_b.  w = 0 protects nothing;
 * T_b <= w keeps the whole sequence.
 *   K, V         [H, n_tokens, D] bf16 (in)    packed sequences along the token axis
 *   scores       [n_tokens, H] fp32 (in)
 *   K_out, V_out [H, n_tokens, D] bf16 (out)   list (b,h) occupies rows
 *                cu_seqlens[b] .. cu_seqlens[b] + lengths[b,h] - 1 of head h, in token order,
 *                rows copied bit for bit; all other rows are left untouched.
 *   lengths      [n_seqs, H] int32 (out)
 * K_out/V_out must not overlap K/V.  tau may be any fp32 (+-inf included); w >= 0.
 */
kvzap_status kvzap_prune_prefill(kvzap_ctx *ctx, const void *K, const void *V, const float *scores,
                                 const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                 float tau, int32_t w,
                                 void *K_out, void *V_out, int32_t *lengths, void *stream);

/*
 * Algorithm 1 in one call: kvzap_score on `hidden` with the threshold and
 * window test fused into the scoring kernel's epilogue, then the compaction of
 * kvzap_prune_prefill.  `scores_out` ([n_tokens, H] fp32) may be NULL when the
 * caller does not need the scores.  Other arguments as above.
 */
kvzap_status kvzap_prefill_fused(kvzap_ctx *ctx, int32_t layer, const void *hidden,
                                 const void *K, const void *V,
                                 const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                 float tau, int32_t w,
                                 void *K_out, void *V_out, int32_t *lengths,
                                 float *scores_out, void *stream);

/*
 * kvzap_prefill_fused for callers whose tensors live in HOST memory (pinned
 * memory recommended).  Every pointer argument, cu_seqlens included, is a HOST
 * pointer with the same shapes as above.  The call copies the inputs into
 * device staging buffers owned by the context (allocated at the first call,
 * sized for max_tokens), runs Algorithm 1 on the device, synchronises
 * `stream`, and copies back lengths, the scores (if scores_out != NULL) and,
 * for every (sequence, head) list, exactly its lengths[b,h] kept rows into the
 * same positions of K_out / V_out; other rows of the host outputs are left
 * untouched.  Returns after the results are in host memory.
 */
kvzap_status kvzap_prefill_fused_host(kvzap_ctx *ctx, int32_t layer, const void *hidden,
                                      const void *K, const void *V,
                                      const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                      float tau, int32_t w,
                                      void *K_out, void *V_out, int32_t *lengths,
                                      float *scores_out, void *stream);

/*
 * The same for a run of layers, with the copies overlapped: while layer l is scored and compacted and its
 * kept rows travel back, layer l + 1 is already being copied in (two staging sets, a copy stream in each
 * direction; kernels on `stream`).  hidden, K, V, K_out, V_out, lengths, scores_out (NULL, or entries NULL,
 * when the scores are not wanted) are HOST arrays of layer_end - layer_begin HOST pointers, one per layer,
 * each with the shapes of kvzap_prefill_fused_host; cu_seqlens is shared by all layers.
 * page_tokens == 0: dense-ragged output as above.  page_tokens > 0: paged output as
 * kvzap_prefill_fused_paged -- K_out[i] / V_out[i] are the host page pools [n_pages_pool, page_tokens, D] of
 * layer i, first_page (host int32 [n_layers], NULL = all 0), page_table[i] (host int32
 * [n_seqs*H, max_pages_per_list]) and n_pages_used[i] (host int32 [1]) as there; only the pages a layer
 * used are copied back.  Pinned host memory is needed for the overlap (pageable memory works, serially).
 * Returns after every layer's results are in host memory.
 */
kvzap_status kvzap_prefill_layers_host(kvzap_ctx *ctx, int32_t layer_begin, int32_t layer_end,
                                       const void *const *hidden, const void *const *K, const void *const *V,
                                       const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                       float tau, int32_t w,
                                       void *const *K_out, void *const *V_out, int32_t *const *lengths,
                                       float *const *scores_out,
                                       int32_t page_tokens, int64_t n_pages_pool, const int32_t *first_page,
                                       int32_t *const *page_table, int32_t max_pages_per_list,
                                       int32_t *const *n_pages_used, void *stream);

/*
 * Paged output of the same pruning (Discussion, "Implementation Challenges":
 * per-head lengths differ, so the pruned cache needs paged kernels with
 * variable-length blocks; the paper fixes no page format, this one is ours).
 * A page holds page_tokens rows; page p of the K pool and page p of the V pool
 * hold matching rows.  List (b,h) receives ceil(lengths[b,h] / page_tokens)
 * pages, numbered contiguously from first_page in (b,h) order (list index
 * b*H + h), and its rows fill them in token order.
 *   K_pool, V_pool [n_pages_pool, page_tokens, D] bf16 (out; caller-owned)
 *   page_table     [n_seqs*H, max_pages_per_list] int32 (out): page numbers of each list; entries
 *                  beyond a list's page count are left untouched
 *   lengths        [n_seqs, H] int32 (out)
 *   n_pages_used   [1] int32 (out, device): pages assigned by this call
 * If the pool (first_page + pages needed > n_pages_pool) or the table (a list
 * needs more than max_pages_per_list) is too small, nothing is copied,
 * *n_pages_used = 0, lengths are still written, and the status word is set to
 * KVZAP_ERR_OOM_PAGES (kvzap_poll_status).
 */
kvzap_status kvzap_prune_prefill_paged(kvzap_ctx *ctx, const void *K, const void *V, const float *scores,
                                       const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                       float tau, int32_t w,
                                       void *K_pool, void *V_pool, int64_t n_pages_pool, int32_t page_tokens,
                                       int32_t first_page, int32_t *page_table, int32_t max_pages_per_list,
                                       int32_t *lengths, int32_t *n_pages_used, void *stream);

/* kvzap_prefill_fused with the paged output above. */
kvzap_status kvzap_prefill_fused_paged(kvzap_ctx *ctx, int32_t layer, const void *hidden,
                                       const void *K, const void *V,
                                       const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                       float tau, int32_t w,
                                       void *K_pool, void *V_pool, int64_t n_pages_pool, int32_t page_tokens,
                                       int32_t first_page, int32_t *page_table, int32_t max_pages_per_list,
                                       int32_t *lengths, int32_t *n_pages_used,
                                       float *scores_out, void *stream);

/* kvzap_prefill_fused_paged for HOST tensors (every pointer, the pools, the page table and n_pages_used
 * included, is a host pointer); see kvzap_prefill_fused_host and kvzap_prefill_layers_host. */
kvzap_status kvzap_prefill_fused_paged_host(kvzap_ctx *ctx, int32_t layer, const void *hidden,
                                            const void *K, const void *V,
                                            const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                            float tau, int32_t w,
                                            void *K_pool, void *V_pool, int64_t n_pages_pool, int32_t page_tokens,
                                            int32_t first_page, int32_t *page_table, int32_t max_pages_per_list,
                                            int32_t *lengths, int32_t *n_pages_used,
                                            float *scores_out, void *stream);

/*
 * Fixed-budget selection instead of a threshold (Ablations, "Threshold-based
 * pruning": the top-k alternatives the paper compares thresholding with, per
 * head or per layer as in AdaKV).  For sequence b the candidates are the
 * positions outside the window, n_cand = max(T_b - w, 0), and the budget is
 * k = ceil(keep_ratio * n_cand) rows per head:
 *   per_layer = 0: list (b,h) keeps its k highest-scoring candidates;
 *   per_layer = 1: the H*k highest of all candidate scores of sequence b are kept,
 *                  whichever heads they fall on (heads share one budget).
 * The call finds the cut value tau[b,h] (the k-th largest candidate score; per
 * layer the (H*k)-th largest over all heads, the same for every h) and then
 * prunes exactly as kvzap_prune_prefill does with that threshold for list (b,h):
 * scores equal to the cut value are all kept (ties may exceed the budget), NaN
 * scores are never candidates, k = 0 gives tau = +inf, fewer than k candidates
 * that are numbers give tau = -inf.  The window is always kept.
 *   keep_ratio in [0, 1];  tau_out [n_seqs, H] fp32 (device) or NULL: the cut values used
 * Other arguments, outputs and errors as kvzap_prune_prefill.
 */
kvzap_status kvzap_prune_prefill_topk(kvzap_ctx *ctx, const void *K, const void *V, const float *scores,
                                      const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                      float keep_ratio, int32_t w, int32_t per_layer,
                                      void *K_out, void *V_out, int32_t *lengths, float *tau_out, void *stream);

/*
 * Pruning on the write side (Discussion, "Implementation Challenges": the
 * surrogate needs only hidden states, so pruning can run before attention).
 * Same operation and outputs as kvzap_prefill_fused / kvzap_prefill_fused_paged,
 * but K and V are taken as the key/value projection leaves them, one token
 * after the other:
 *   K_proj, V_proj [n_tokens, H, D] bf16 (device, 16-byte aligned, caller-owned)
 * so a caller never has to build the dense head-major cache [H, n_tokens, D]:
 * rows that are dropped are never read, rows that are kept are read once and
 * written once, straight into list (b,h).  All other arguments, the outputs,
 * the empty-input behaviour and the errors are those of the calls named above.
 */
kvzap_status kvzap_prefill_write(kvzap_ctx *ctx, int32_t layer, const void *hidden,
                                 const void *K_proj, const void *V_proj,
                                 const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                 float tau, int32_t w,
                                 void *K_out, void *V_out, int32_t *lengths,
                                 float *scores_out, void *stream);
kvzap_status kvzap_prefill_write_paged(kvzap_ctx *ctx, int32_t layer, const void *hidden,
                                       const void *K_proj, const void *V_proj,
                                       const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                       float tau, int32_t w,
                                       void *K_pool, void *V_pool, int64_t n_pages_pool, int32_t page_tokens,
                                       int32_t first_page, int32_t *page_table, int32_t max_pages_per_list,
                                       int32_t *lengths, int32_t *n_pages_used,
                                       float *scores_out, void *stream);

/*
 * Pruning on the write side without any copy: a write plan (Discussion, "Implementation Challenges": the
 * surrogate needs only hidden states, so "pruning could also be applied before attention" -- here, before
 * the keys and values are stored at all).  Scores the hidden states, applies threshold and window, and
 * instead of moving rows tells the producer of K and V where every (token, head) pair belongs:
 *   slot [n_tokens, H] int32 (out): the pair's destination row, or -1 if it is dropped.
 *     page_tokens == 0: the row inside list (b,h), i.e. the number of kept positions of the list before the
 *                       token; in the dense-ragged layout of kvzap_prune_prefill the producer writes the pair
 *                       to row cu_seqlens[b] + slot of head h;
 *     page_tokens  > 0: the row of the page pools, pages assigned exactly as by kvzap_prune_prefill_paged
 *                       (page_table, n_pages_used, first_page, n_pages_pool, max_pages_per_list as there;
 *                       on a pool or table that is too small every slot is -1 and the status word is set).
 *   lengths [n_seqs, H] int32 (out);  scores_out [n_tokens, H] fp32 or NULL.
 * A producer that writes each kept row to its slot gets exactly the output of kvzap_prefill_fused
 * (kvzap_prefill_fused_paged), the dropped rows are never stored, and the library moves no K or V byte.
 */
kvzap_status kvzap_prefill_plan(kvzap_ctx *ctx, int32_t layer, const void *hidden,
                                const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                float tau, int32_t w,
                                int32_t *slot, int32_t *lengths, float *scores_out,
                                int32_t page_tokens, int64_t n_pages_pool, int32_t first_page,
                                int32_t *page_table, int32_t max_pages_per_list, int32_t *n_pages_used,
                                void *stream);

/*
 * Decode-time cache (caption of Algorithm 1: decoding is like prefilling but
 * needs a buffer of scores to enforce the sliding window; contributions:
 * delayed eviction with a sliding window).  One list per (sequence, layer, KV
 * head).  The most recent `window` tokens of a list sit in a ring owned by the
 * cache together with their scores; a token that leaves the window joins the
 * list's permanent, position-ordered prefix iff its score >= tau, otherwise it
 * is dropped.  The prefix lives in pages of the caller's pools
 * ([n_pages_pool, page_tokens, D] bf16 each), taken one at a time from a bump
 * allocator.  The logical content of a list is prefix ++ window, oldest first;
 * for a fixed tau it equals the prefill pruning of the whole sequence.
 * kvzap_cache_create allocates (cudaMalloc) the rings
 * (2 * n_seqs*L*H*window*D*2 bytes), score buffers, lengths and page tables.
 */
typedef struct kvzap_cache kvzap_cache;
kvzap_status kvzap_cache_create(kvzap_ctx *ctx, kvzap_cache **out, int32_t n_seqs, int32_t window,
                                int32_t page_tokens, void *K_pool, void *V_pool, int64_t n_pages_pool,
                                int32_t max_pages_per_list);
kvzap_status kvzap_cache_destroy(kvzap_cache *cache);

/*
 * One decode step for layers [layer_begin, layer_end) and all n_seqs sequences:
 * scores the new token of every sequence with each layer's surrogate, appends
 * its key/value row and score to the window, and decides the token that leaves
 * the window (kept iff its buffered score >= tau).
 *   hidden       [layer_end-layer_begin, n_seqs, d_model] bf16
 *   K_new, V_new [layer_end-layer_begin, n_seqs, H, D] bf16
 *   scores_out   [layer_end-layer_begin, n_seqs, H] fp32 or NULL
 * A full pool or page table drops the row that needed the page and sets the
 * status word to KVZAP_ERR_OOM_PAGES.
 * With the MLP surrogate, window > 0 and at most 128 sequences per 128-token
 * tile of a few-layer-by-few-tile launch (the usual decode shape), the whole
 * step is ONE kernel launch: the cache update runs in the scoring kernel's
 * otherwise idle warps, and consecutive steps overlap on the GPU when their
 * scores_out buffers differ (or are NULL).
 * The call may be captured in a CUDA graph (stream capture) and replayed, alone or with kvzap_decode_attention:
 * the number of the step is kept on the device.  Call it (and the attention) once outside the capture first, so
 * that whatever they build on first use exists; pass the same buffers in every replay and refill them in between.
 */
kvzap_status kvzap_decode_step(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer_begin, int32_t layer_end,
                               const void *hidden, const void *K_new, const void *V_new, float tau,
                               float *scores_out, void *stream);

/*
 * The same step with the new tokens' hidden states as E4M3 bytes (layers set with kvzap_set_weights_fp8):
 *   hidden_e4m3 [layer_end - layer_begin, n_seqs, d_model] bytes, x_scale [layer_end - layer_begin, n_seqs]
 *   fp32 or NULL (= 1), both on the device; everything else as kvzap_decode_step.
 * A decode step is bound by reading the first-layer weights once per step; with 8-bit weights that is half
 * the bytes.  Scores as kvzap_score_fp8 gives them (the two scales multiply the first layer's sum before
 * the bias), the cache update is the same.
 */
kvzap_status kvzap_decode_step_fp8(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer_begin, int32_t layer_end,
                                   const void *hidden_e4m3, const float *x_scale, const void *K_new, const void *V_new,
                                   float tau, float *scores_out, void *stream);

/*
 * Attention of the newest token over the pruned cache (Introduction, Criterion 3;
 * Discussion, "Implementation Challenges": lists of different lengths per head
 * need an attention kernel that takes variable-length paged lists).  For every
 * sequence b, layer l in [layer_begin, layer_end) and query head j, with KV head
 * h = j / G, G = n_q_heads / H (grouped-query attention, consecutive query heads
 * share a KV head):
 *   O[l,b,j] = sum_i softmax_i(scale * Q[l,b,j] . K_i) V_i
 * over all rows i list (b,l,h) holds at the time of the call: its paged prefix
 * and the valid slots of its window (the row appended by the latest
 * kvzap_decode_step included).  The order of a list's rows does not matter.
 *   Q, O  [layer_end - layer_begin, n_seqs, n_q_heads, D] bf16 (device, 16-byte aligned)
 *   scale >= 0, usually 1 / sqrt(D)
 * An empty list gives zeros.  Arithmetic: bf16 products with fp32 accumulation,
 * softmax in fp32, probabilities rounded to bf16 for the second product, one
 * rounding of O to bf16.  Reads the cache only; one kernel launch, ordered on
 * the stream after the decode steps enqueued before it.
 * KVZAP_ERR_UNSUPPORTED unless D is 64 or 128, page_tokens and window are
 * multiples of 16, and 1 <= G <= 8.  A bounded wait that runs out sets the
 * status word to KVZAP_ERR_TIMEOUT and zeros the affected outputs.
 */
kvzap_status kvzap_decode_attention(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer_begin, int32_t layer_end,
                                    const void *Q, int32_t n_q_heads, float scale, void *O, void *stream);

/*
 * The same attention over a cache whose rows are 8-bit (Related work, "Quantization": quantising the
 * cache and pruning it compose; the pruning calls move rows as opaque bytes, so only this call has to know
 * the format).  The context is created with head_dim = (D + 16) / 2, where D = 64 or 128 is the number of
 * elements per head: a row of head_dim * 2 bytes is D E4M3 codes (1 sign, 4 exponent, 3 mantissa bits, bias 7,
 * no infinities, S.1111.111 = NaN) followed by a 16-byte trailer, the row's fp32 scale and 12 unused bytes;
 * the row stands for scale * code.  Whoever writes K_new / V_new (the projection's epilogue) quantises; every
 * kvzap_* call that moves rows keeps codes and scale together.
 *   Q, O [layer_end - layer_begin, n_seqs, n_q_heads, D] bf16 (device)
 * logit_i = scale * k_scale_i * (q . K8_i), out = sum_i softmax(logit)_i * v_scale_i * V8_i, fp32 accumulation,
 * codes widened exactly, the probabilities times v_scale_i rounded to bf16 for the second product.
 * Everything else (grouping of query heads, empty lists, released slots, page and window multiples of 16,
 * bounded waits) as kvzap_decode_attention.  A cache serves one of the two attention calls, not both.
 */
kvzap_status kvzap_decode_attention_fp8(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer_begin, int32_t layer_end,
                                        const void *Q, int32_t n_q_heads, float scale, void *O, void *stream);

/*
 * A sequence has ended: all lists (seq, *, *) become empty and their pages go back to the cache's
 * allocator, which hands released pages out again (to any list) before it touches never-used pages
 * of the pool.  Until the slot is given a new prompt (kvzap_prefill_to_cache) decode steps leave its
 * lists alone (its rows of hidden, K_new, V_new are ignored, its scores still computed) and attention over
 * it gives zeros.  Enqueued on the stream like every other call; the paper does not discuss this, it is
 * bookkeeping a serving loop needs around the method.
 */
kvzap_status kvzap_cache_release_seq(kvzap_cache *cache, int32_t seq, void *stream);

/* lengths [n_seqs, L, H] int32 (device): rows currently held by each list (prefix + window). */
kvzap_status kvzap_cache_lengths(kvzap_cache *cache, int32_t *lengths, void *stream);

/* Copies one list, oldest row first, into K_out / V_out [capacity_rows, D] bf16 (device) and
 * writes its row count to *n_rows (device); rows beyond capacity_rows are not copied. */
kvzap_status kvzap_cache_export(kvzap_cache *cache, int32_t seq, int32_t layer, int32_t head,
                                void *K_out, void *V_out, int64_t capacity_rows, int32_t *n_rows,
                                void *stream);

/*
 * Prefill of one sequence's prompt for one layer straight into the decode
 * cache, so that decoding can continue from it: scores the prompt, sends the
 * tokens before the last `window` ones through the threshold (kept ones form
 * the list's paged prefix, pages taken from the cache's allocator), and puts
 * the last min(n_tokens, window) tokens with their scores into the window
 * ring, where later decode steps will decide them.  After it, the lists
 * (seq, layer, *) hold exactly what kvzap_prefill_fused would keep, and
 * prefill(T) followed by k decode steps equals prefill(T + k).
 *   hidden [n_tokens, d_model] bf16, K, V [H, n_tokens, D] bf16 (one sequence)
 *   scores_out [n_tokens, H] fp32 (device) -- required, it also serves as scratch
 * Chunked prefill: the lists need not be empty.  Called again with the next
 * chunk of the same prompt (or after decode steps), the call first decides the
 * tokens of the present window that the chunk pushes out, by their buffered
 * scores, then appends the chunk as described above; prefill in chunks of any
 * lengths equals one prefill of the whole prompt (the score buffer carries the
 * window across chunk boundaries).
 */
kvzap_status kvzap_prefill_to_cache(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer, int32_t seq,
                                    const void *hidden, const void *K, const void *V, int64_t n_tokens,
                                    float tau, float *scores_out, void *stream);

/*
 * The same for several prompts (or chunks of prompts) at once, one layer: sequence i of the call is tokens
 * cu_seqlens[i] .. cu_seqlens[i+1] of the packed buffers and goes to the cache's sequence slot seq_ids[i].
 * One scoring launch over all tokens instead of one small launch per prompt, and three more launches
 * for the whole batch (window side, page assignment, compaction).  Each sequence ends up exactly as
 * kvzap_prefill_to_cache would leave it (which pages a list gets depends on the order of allocation and
 * may differ).
 *   seq_ids    [n_seqs] int32, HOST: distinct slots in 0..n_seqs_of_the_cache-1 (checked; read before return)
 *   cu_seqlens [n_seqs+1] int32 (device); empty sequences are allowed and change nothing
 *   hidden [n_tokens, d_model] bf16, K, V [H, n_tokens, D] bf16 (packed over the sequences),
 *   scores_out [n_tokens, H] fp32 (device) -- required
 * n_seqs <= max_seqs and n_tokens <= max_tokens of the context.
 */
kvzap_status kvzap_prefill_to_cache_batch(kvzap_ctx *ctx, kvzap_cache *cache, int32_t layer, const int32_t *seq_ids,
                                          const int32_t *cu_seqlens, int32_t n_seqs, const void *hidden, const void *K,
                                          const void *V, int64_t n_tokens, float tau, float *scores_out, void *stream);

/*
 * Installs prefix bookkeeping produced elsewhere (used to set up synthetic
 * cache states): prefix_len [n_seqs*L*H] and page_table
 * [n_seqs*L*H, max_pages_per_list], device int32 in list order (seq, layer,
 * head); next_free_page is the first pool page the allocator may hand out.
 * Every list's window becomes empty.  Synchronises `stream`.
 */
kvzap_status kvzap_cache_import(kvzap_cache *cache, const int32_t *prefix_len, const int32_t *page_table,
                                int32_t next_free_page, void *stream);

/*
 * The inverse of kvzap_cache_import, a snapshot of the prefix bookkeeping: copies prefix_len
 * [n_seqs*L*H] and page_table [n_seqs*L*H, max_pages_per_list] (device int32, list order (seq, layer,
 * head)) out of the cache and writes the allocator's cursor -- the first pool page never handed out --
 * to *next_free_page (device).  Entries of a list's table row beyond ceil(prefix_len / page_tokens)
 * are meaningless.  Enqueued on `stream`; used by the tests to check that no page is owned twice.
 */
kvzap_status kvzap_cache_snapshot(kvzap_cache *cache, int32_t *prefix_len, int32_t *page_table,
                                  int32_t *next_free_page, void *stream);

/* Kernel identifiers for kvzap_get_profile. */
enum { KVZAP_KERNEL_SCORE = 0, KVZAP_KERNEL_MASK = 1, KVZAP_KERNEL_SCAN = 2, KVZAP_KERNEL_COMPACT = 3,
       KVZAP_KERNEL_DECODE_UPDATE = 4, KVZAP_KERNEL_ATTENTION = 5 };

/*
 * Per-kernel timing with CUDA events on the launching stream (a measurement
 * aid; the paper has no counterpart).  While enabled, every kernel launch is
 * bracketed by two events.  kvzap_set_profiling(ctx, 0/1) switches it and
 * discards earlier records; kvzap_get_profile synchronises the device and
 * returns the summed duration and the number of launches of one kernel.
 */
kvzap_status kvzap_set_profiling(kvzap_ctx *ctx, int32_t enable);
kvzap_status kvzap_get_profile(kvzap_ctx *ctx, int32_t kernel, double *total_ms, int64_t *n_launches);

/*
 * kvzap_prune_prefill for callers that cannot allocate device memory.  (The
 * paper has no counterpart; this is a deployment variant of the same
 * operation.)
 *
 * Who needs it: a serving process that handed all of the GPU's memory to its
 * own KV-cache pool at start-up, so that a later cudaMalloc (which
 * kvzap_create performs) fails or steals from that pool; and latency-critical
 * loops that may not call cudaMalloc/cudaFree because those calls stall every
 * stream of the device while they run.  This entry point needs no context and
 * never calls cudaMalloc, cudaFree or any other allocating routine.
 *
 * Instead of a context's scratch it uses one fixed array compiled into the
 * library's device image (about 170 KB, held by every GPU that loads the
 * library until the process exits).  Consequences:
 *   - sizes are capped: n_tokens <= KVZAP_NOALLOC_MAX_TOKENS and
 *     n_seqs <= KVZAP_NOALLOC_MAX_SEQS, else KVZAP_ERR_UNSUPPORTED is returned
 *     and nothing is launched;
 *   - it works on the CURRENT device (cudaSetDevice), where all pointers must
 *     live; the first call on each device also looks up the array's device
 *     address, so make that first call before starting any stream capture;
 *   - all calls on a device share the array, which still holds the previous
 *     call's contents (the call rewrites everything it reads, and clears its
 *     status word): two calls that overlap on the GPU -- different streams, or
 *     different host threads -- race on it and produce garbage.  Serialise
 *     them on one stream.
 * Arguments and results are exactly those of kvzap_prune_prefill, with the
 * two shape parameters a context would have carried (n_kv_heads 1..8, head_dim
 * a multiple of 8 in 8..1024) passed explicitly.  Error text is available
 * from kvzap_last_error(NULL).
 */
#define KVZAP_NOALLOC_MAX_TOKENS 131072
#define KVZAP_NOALLOC_MAX_SEQS 256
kvzap_status kvzap_prune_prefill_noalloc(const void *K, const void *V, const float *scores,
                                         const int32_t *cu_seqlens, int32_t n_seqs, int64_t n_tokens,
                                         int32_t n_kv_heads, int32_t head_dim, float tau, int32_t w,
                                         void *K_out, void *V_out, int32_t *lengths, void *stream);

/*
 * Reads the context's device status word (synchronises `stream` first) and
 * clears it.  Returns KVZAP_OK, or the first device-side condition recorded
 * since the last poll (KVZAP_ERR_TIMEOUT, KVZAP_ERR_OOM_PAGES).
 */
kvzap_status kvzap_poll_status(kvzap_ctx *ctx, void *stream);

/*
 * Failure detection (the paper has no counterpart).  Waits on flags in global memory that another
 * CTA or an earlier launch sets -- the step counters that order consecutive fused decode steps, the
 * per-tile counts of the one-launch prefill of short prompts -- give up after `cycles` SM clock cycles
 * (default about one second), set the status word to KVZAP_ERR_TIMEOUT and return without touching
 * the cache, the lengths or the compacted rows (a scores buffer may hold unfinished values).
 * kvzap_set_wait_limit changes that bound for later calls on the context (cycles >= 1000).  Waits on hardware barriers inside a CTA keep their compile-time bound.
 * After a polled KVZAP_ERR_TIMEOUT the step counters of every cache of the context are cleared, so
 * the next decode step starts from a consistent state; steps that were in flight when the wait ran
 * out did nothing.
 */
kvzap_status kvzap_set_wait_limit(kvzap_ctx *ctx, int64_t cycles);

/*
 * Test aid: adds `delta` to the cache's device-side counts of decode steps STARTED (the tickets from which a
 * one-launch step learns its number) without touching the counts of steps COMPLETED.  The next such step then
 * waits for a step that never ran, its bounded wait runs out, and the status word reads KVZAP_ERR_TIMEOUT: the
 * one way to see that path without a fault.  Synchronises the device.  Never call it in production code.
 */
kvzap_status kvzap_cache_debug_skew_steps(kvzap_cache *cache, int32_t delta);

/* Number of kernels the library has launched through this context since it was
 * created (for launch accounting in benchmarks). */
int64_t kvzap_launch_count(const kvzap_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* KVZAP_H_ */
