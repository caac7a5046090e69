/*
 * meda.h - C ABI of the B200-native MEDA prefill KV-cache compression pass
 * (MEDA: "Dynamic KV Cache Allocation for Efficient Multimodal Long-Context Inference",
 *  arXiv 2502.17599, Sections 3.2-3.3 and 4.4, Appendix A.3).
 *
 * The pass runs once after prompt encoding and before decoding:
 *   phase A, per layer : attention of an observation window of text queries against the whole
 *                        key cache -> per-key accumulated scores (Eq. 8) and the cross-modal
 *                        attention entropy E_CM of the layer (Eq. 4-6);
 *   barrier            : softmax over all layers' entropies -> integer per-layer budgets that sum
 *                        to the global budget (Eq. 7), each split recent : important;
 *   phase B, per layer : per KV head, keep the recent tokens plus the top-scoring ones with text
 *                        first (Eq. 9-10); merge every other KV pair into its most cosine-similar
 *                        kept key by averaging (Eq. 11-12).
 *
 * Conventions that hold for every entry point unless it says otherwise
 *  - Every tensor pointer is a DEVICE pointer owned by the caller; the library neither frees it
 *    nor keeps it after the call's work has run.  `spans_host` and `meda_config` are HOST memory.
 *  - Layouts are dense and row-major: caches [n_kv_heads][n_tokens][head_dim], query windows
 *    [n_q_heads][window][head_dim], element type `dtype` (bf16 or fp32).  Query head h belongs
 *    to KV head h / (n_q_heads / n_kv_heads).  Window row i is the token at absolute position
 *    n_tokens - window + i and, as in decoder prefill, sees keys j <= that position.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only enqueue
 *    work and return; nothing is copied back to the host between steps.
 *  - Step calls allocate nothing: all scratch memory is taken from the context at meda_create.
 *    A context may be used by one host thread and one stream at a time.
 *  - Errors the host can see (NULL pointers, bad shapes, bad layer index) return a negative
 *    status before anything is launched.  Errors only the device can see (a budget row that does
 *    not fit `out_capacity`, a bounded wait that ran out) are recorded in a status word that
 *    meda_poll_status returns; the kernel that saw the error skips its work and returns.
 *  - `budgets` is int32 [n_layers][3] = (S_l, M_l, N_l): conserved rows, recent rows, top-scored
 *    rows (S_l = M_l + N_l).  It stays on the device; kernels read their layer's row.
 */
#ifndef MEDA_H_
#define MEDA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct meda_ctx meda_ctx; /* opaque: configuration, modality map and scratch memory */

typedef enum {
  MEDA_OK = 0,
  MEDA_ERR_INVALID_ARG = -1,       /* NULL pointer, bad enum, layer out of range */
  MEDA_ERR_SHAPE = -2,             /* sizes the kernels do not support or that contradict each other */
  MEDA_ERR_BUDGET_INFEASIBLE = -3, /* global budget outside [L*min_budget, L*n_tokens] */
  MEDA_ERR_WORKSPACE = -4,         /* an output capacity is too small for the layer's budget */
  MEDA_ERR_CUDA = -5,              /* a CUDA runtime call failed */
  MEDA_ERR_UNSUPPORTED = -6,       /* valid request that the library does not implement */
  MEDA_ERR_TIMEOUT = -7            /* a bounded device-side wait ran out */
} meda_status;

typedef enum { MEDA_BF16 = 0, MEDA_F32 = 1 } meda_dtype;
enum { MEDA_TEXT = 0, MEDA_VISUAL = 1 };

/* One run of tokens of a single modality, [begin, end).  The table passed to meda_create must be
 * sorted, disjoint and cover [0, n_tokens) exactly (Sec. 3.1: the prompt is an interleaving of
 * text and image / video token runs; Sec. 3.2 splits Q and K "based on the modality index"). */
typedef struct {
  int32_t begin, end, modality;
} meda_span;

typedef struct {
  int32_t n_layers, n_q_heads, n_kv_heads, head_dim, n_tokens, window;
  int32_t dtype;          /* meda_dtype of caches, query windows and outputs */
  int64_t global_budget;  /* B = sum_l S_l in token*layers; Eq. 7 with B = round(rho * L * n_tokens) */
  int32_t beta_recent;    /* recent : important split of each layer budget, 3 : 1 in Sec. 4.4 */
  int32_t beta_important;
  int32_t min_budget;     /* per-layer floor of S_l (>= 1); n_tokens is the ceiling */
  int32_t entropy_mode;   /* 0: entropy of the head-averaged attention (Sec. 3.2); 1: mean of per-head entropies */
  int32_t alloc_mode;     /* 0: Eq. 7; 1: uniform shares (Table 5, the row without dynamic allocation) */
  int32_t merge_mode;     /* 0: Eq. 12 average merging; 1: drop the less important pairs (Table 5, the row without merging) */
} meda_config;

/* Creates a context: validates the configuration, uploads the modality map built from
 * `spans_host` (host memory, n_spans entries) and allocates all scratch memory on the current
 * device (the only allocating call).  Supported shapes: head_dim in {64, 128, 256} for fp32 and
 * bf16, n_q_heads a multiple of n_kv_heads, 1 <= window <= min(n_tokens, 128), n_layers <= 1024; one head's
 * cache below 4 GiB (n_tokens * head_dim * element size < 2^32) and n_tokens * n_kv_heads < 2^31 (MEDA_ERR_SHAPE
 * otherwise).  On failure *out is NULL and the status says why. */
meda_status meda_create(const meda_config* config, const meda_span* spans_host, int32_t n_spans, meda_ctx** out);

/* Frees the context's scratch memory.  The caller must have synchronised the streams that used it. */
void meda_destroy(meda_ctx* ctx);

/* Static, NUL-terminated description of a status code. */
const char* meda_status_string(meda_status status);

/* Bytes of device scratch memory the context holds. */
int64_t meda_workspace_bytes(const meda_ctx* ctx);

/* Synchronises `stream`, returns the first device-side error recorded since the last poll (or
 * MEDA_OK) and clears it. */
meda_status meda_poll_status(meda_ctx* ctx, void* stream);

/* Phase A, one layer (Eq. 4 and Eq. 8 with the query rows restricted to the observation window).
 * Two sweeps over the key cache.  The first computes every window row's softmax normalisers:
 *   row_stats fp32 [n_q_heads][window][4] = (max, sum exp(s - max)) over all visible keys and
 *   (max, sum exp) over the visible VISUAL keys, s = q.k / sqrt(head_dim); a row that sees no
 *   visual key has (-inf, 0) there.
 * The second computes the per-key accumulated attention
 *   scores fp32 [n_kv_heads][n_tokens]: A_s[g][j] = sum over window rows i and query heads h of
 *   KV head g of softmax_j(s)[h][i][j]   (each KV head's scores sum to group_size * window)
 * and, when `entropy` is not NULL, in the same sweep the layer's cross-modal entropy
 *   entropy[layer] (fp32, device array of n_layers): E_CM = -E_TV of Eq. 5-6, the mean over
 *   window rows of the entropy (natural log) of text-to-vision attention, whose softmax is taken
 *   over the visual keys only; averaged over heads before or after the entropy per entropy_mode.
 * q_win, k: device, `dtype`.  row_stats, scores: device outputs, fully overwritten. */
meda_status meda_window_scores(meda_ctx* ctx, int32_t layer, const void* q_win, const void* k,
                               float* row_stats, float* scores, float* entropy, void* stream);

/* The second sweep of meda_window_scores alone, for a caller that already holds the window rows' softmax
 * normalisers (for instance from the prefill attention kernel that produced the cache, if it also tracks the
 * normaliser over the visual keys): one pass over the key cache instead of two.  row_stats is an INPUT here,
 * fp32 [n_q_heads][window][4] with the layout and meaning meda_window_scores writes; scores and
 * entropy[layer] (entropy may be NULL) are written exactly as by meda_window_scores. */
meda_status meda_window_scores_from_stats(meda_ctx* ctx, int32_t layer, const void* q_win, const void* k,
                                          const float* row_stats, float* scores, float* entropy, void* stream);

/* Eq. 8 as printed, with EVERY prompt row as a query instead of an observation window: the accumulated
 * score of key j is the column sum of the whole causal attention matrix of prompt encoding,
 *   scores[g][j] = sum over the query heads h of KV head g and over the rows i >= j of
 *                  softmax_j(q_i . k / sqrt(head_dim))[h][i][j]      (each KV head's scores sum to group_size * n_tokens).
 * q_all: device, `dtype`, [n_q_heads][n_tokens][head_dim], the query rows of all prompt tokens (row i sits at
 * position i and sees keys j <= i); k: device, `dtype`, [n_kv_heads][n_tokens][head_dim].
 * scores: device fp32 [n_kv_heads][n_tokens], fully overwritten; it can be passed to meda_select_topk /
 * meda_compress_layer in place of the window's scores.  The cost is that of the prompt's attention itself
 * (n_tokens^2 / 2 logits per query head, twice: normalisers, then column sums), independent of `window`.
 * scratch: device memory of at least meda_prompt_scores_scratch_bytes(ctx) bytes, 16-byte aligned, owned by
 * the caller and free again when the call's work on `stream` has finished (the per-row normalisers and the
 * partial scores live there: 20 bytes per query head and token or a little more).  When that size is 0 (fp32 or head_dim != 128: the
 * rows then go block by block through the context's own scratch) it may be NULL.  A scratch that is too small
 * returns MEDA_ERR_WORKSPACE and launches nothing. */
int64_t meda_prompt_scores_scratch_bytes(const meda_ctx* ctx);
meda_status meda_prompt_scores(meda_ctx* ctx, const void* q_all, const void* k, float* scores, void* scratch,
                               int64_t scratch_bytes, void* stream);

/* Cross-modal attention entropy of one layer (Eq. 4-6): E_CM = -(E_TV + E_VT), written to entropy[layer].
 *  - The E_TV term uses the text window q_win and its row_stats (from meda_window_scores): one sweep over
 *    the key cache, the same arithmetic as meda_window_scores' own entropy.  For callers that already hold
 *    the normalisers.
 *  - The E_VT term of Eq. 5 needs VISUAL query rows, which a text window does not contain: q_vis (device,
 *    `dtype`, [n_q_heads][n_vis_rows][head_dim]) and q_vis_pos (device int32 [n_vis_rows], the rows'
 *    absolute token positions, each seeing the keys at or before it).  Its softmax is taken over the TEXT keys
 *    a row sees; rows that see no text key are left out of the mean, as are they from its divisor.  With these
 *    two sweeps over the text keys -E_VT is added to entropy[layer].  n_vis_rows <= 128.  Pass NULL, NULL, 0
 *    for the text-window-only definition E_CM = -E_TV.
 *  - q_win (and row_stats) may be NULL when q_vis is given: then only -E_VT is added to what entropy[layer]
 *    already holds (for example the value meda_window_scores wrote). */
meda_status meda_layer_entropy(meda_ctx* ctx, int32_t layer, const void* q_win, const void* k,
                               const float* row_stats, const void* q_vis, const int32_t* q_vis_pos,
                               int32_t n_vis_rows, float* entropy, void* stream);

/* Barrier step (Eq. 7, Appendix A.3, and Sec. 4.4 for the split): one thread block.
 * weights W_l = softmax_l(entropy); real quotas q_l = clip(lambda W_l, min_budget, n_tokens) with
 * lambda such that sum q_l = global_budget; S_l = floor(q_l) and the missing units go one each to
 * the unclamped layers by largest fractional part, ties to the lowest layer;
 * M_l = floor(S_l * beta_recent / (beta_recent + beta_important)), N_l = S_l - M_l.
 * entropy: device fp32 [n_layers].  budgets: device int32 [n_layers][3], overwritten. */
meda_status meda_allocate_budgets(meda_ctx* ctx, const float* entropy, int32_t* budgets, void* stream);

/* Phase B, selection for one layer and all its KV heads (Eq. 9-10).  Candidates are tokens
 * [0, n_tokens - M_l); they are ranked text before visual (Eq. 9's boost), then by score
 * descending, then by index ascending; the first N_l are kept together with the last M_l tokens.
 *   idx_conserved int32 [n_kv_heads][out_capacity]: the S_l kept token indices, ascending
 *   idx_less      int32 [n_kv_heads][n_tokens]    : the n_tokens - S_l others, ascending
 * Entries past those counts are left untouched.  S_l > out_capacity records MEDA_ERR_WORKSPACE. */
meda_status meda_select_topk(meda_ctx* ctx, int32_t layer, const float* scores, const int32_t* budgets,
                             int32_t* idx_conserved, int32_t* idx_less, int32_t out_capacity, void* stream);

/* Phase B, merging for one layer and all its KV heads (Eq. 11-12).  For every less important
 * token i the kept slot with the largest cosine similarity of keys, u = k_i.k_j / (|k_i||k_j|)
 * with each norm clamped below at 1e-8, first maximum in slot order; then for keys and values
 *   x_out[g][s] = (x[c_s] + sum of x[i] over tokens i assigned to s) / counts[g][s],
 * sums over the ORIGINAL rows, accumulated in fp32 in ascending token order, rounded once to
 * `dtype`.  With merge_mode 1 the kept rows are copied and counts are 1.
 *   k_out, v_out `dtype` [n_kv_heads][out_capacity][head_dim]; counts int32 [n_kv_heads][out_capacity]
 *   target int32 [n_kv_heads][n_tokens], optional (may be NULL): slot chosen for idx_less[g][p]
 * Rows past S_l are left untouched. */
meda_status meda_merge_kv(meda_ctx* ctx, int32_t layer, const void* k, const void* v, const int32_t* budgets,
                          const int32_t* idx_conserved, const int32_t* idx_less,
                          void* k_out, void* v_out, int32_t* counts, int32_t* target,
                          int32_t out_capacity, void* stream);

/* Phase B for one layer: meda_select_topk followed by meda_merge_kv, with the less-important
 * list kept in the context's scratch memory (Sec. 3.3 as a whole). */
meda_status meda_compress_layer(meda_ctx* ctx, int32_t layer, const void* k, const void* v, const float* scores,
                                const int32_t* budgets, void* k_out, void* v_out, int32_t* counts,
                                int32_t* idx_conserved, int32_t out_capacity, void* stream);

/* After the pass: attention of one new token's queries over one layer's cache (Eq. 3), the step the compressed
 * caches exist for.  out[h] = softmax(q_h . K_g^T / sqrt(head_dim)) V_g over the cache's rows, g the KV head of
 * query head h; the new token comes after every cached one, so nothing is masked, and merged rows are used as
 * they are (Eq. 3 carries no weights).
 *   q        device, `dtype`, [n_q_heads][head_dim]
 *   k_cache, v_cache  device, `dtype`, [n_kv_heads][capacity][head_dim]: the k_out / v_out of this layer, or a
 *            full cache
 *   budgets  device int32 [n_layers][3] or NULL.  Not NULL: the row count is S_layer, read on the device.
 *            NULL: the row count is n_rows (1 <= n_rows <= capacity), for a cache that was not compressed.
 *   out      device fp32 [n_q_heads][head_dim]
 * Supported: head_dim 64 or 128, n_q_heads / n_kv_heads in {1, 2, 3, 4, 7, 8}; otherwise MEDA_ERR_UNSUPPORTED. */
meda_status meda_decode_attention(meda_ctx* ctx, int32_t layer, const void* q, const void* k_cache, const void* v_cache,
                                  const int32_t* budgets, int32_t n_rows, int32_t capacity, float* out, void* stream);

/* ---- entry point that allocates nothing (the paper has no counterpart) ---------------------- */

/* Largest n_q_heads * window the entry point below accepts, and the size of the scratch array
 * it uses: MEDA_STATIC_STATS_CHUNKS partial results of 4 floats for each of those rows (2 MiB). */
enum { MEDA_STATIC_STATS_MAX_ROWS = 4096, MEDA_STATIC_STATS_CHUNKS = 32 };

/* Softmax normalisers of the window rows (the row_stats array of meda_window_scores, same
 * layout and meaning) for callers that cannot allocate device memory.  Every other entry point
 * needs a context, and meda_create calls cudaMalloc.  A serving process that handed the whole of
 * device memory to its own pool at start-up has none left for cudaMalloc to hand out; a caller in
 * the middle of a latency-critical section cannot afford the device-wide synchronisation that
 * cudaMalloc and cudaFree imply; both can still call this function.  It takes no context, calls
 * no allocating routine, and keeps its only scratch memory, the per-key-chunk partial
 * normalisers, in a fixed 2 MiB array inside the library's device image: every GPU that loads
 * the library holds those 2 MiB until the process exits, whether this function is called or not.
 *
 *   q_win    device, `dtype`, [n_q_heads][window][head_dim]
 *   k        device, `dtype`, [n_kv_heads][n_tokens][head_dim]
 *   modality device, uint8 [n_tokens]: MEDA_TEXT or MEDA_VISUAL per token (the caller's own map;
 *            there is no context to build it from a span table)
 *   row_stats device output, fp32 [n_q_heads][window][4], fully overwritten
 *
 * Limits: n_q_heads * window <= MEDA_STATIC_STATS_MAX_ROWS, window <= 128, head_dim in {64, 128,
 * 256}, n_q_heads a multiple of n_kv_heads; anything else returns MEDA_ERR_SHAPE (or
 * MEDA_ERR_INVALID_ARG for NULL pointers or an unknown dtype) before any CUDA call.
 * It always runs the CUDA-core kernels, so for bf16 / head_dim 128 / window 32 or 64 its numbers
 * agree with meda_window_scores' to rounding (2e-5 on the log-normaliser), not bit for bit.
 *
 * The first call on each device looks up the scratch array's device address and raises the
 * kernel's shared-memory limit, with that device current; make that first call before any stream
 * capture begins.  Later calls on the device only launch.  The array is shared by every call in
 * the process: each call overwrites all the entries it later reads, so nothing needs clearing
 * and the last call's contents are harmless, but two calls whose kernels overlap on the same GPU
 * (different streams, or different host threads) race on it and give wrong results; serialise
 * them. */
meda_status meda_row_stats_static(const void* q_win, const void* k, const uint8_t* modality,
                                  int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t n_tokens,
                                  int32_t window, int32_t dtype, float* row_stats, void* stream);

/* ---- measurement helpers (no counterpart in the paper) ------------------------------------ */

/* Kernel classes the library reports times for. */
enum {
  MEDA_K_STATS = 0,      /* phase A sweep 1: softmax normalisers */
  MEDA_K_STATS_COMBINE,  /* merge of the partial normalisers */
  MEDA_K_SWEEP,          /* phase A sweep 2: scores and/or entropy */
  MEDA_K_ENTROPY_FINAL,  /* reduction of the entropy partials */
  MEDA_K_ALLOCATE,       /* budgets */
  MEDA_K_SELECT,         /* radix select + compaction */
  MEDA_K_PREP,           /* conserved-key gather and inverse norms */
  MEDA_K_NEAREST,        /* similarity contraction + arg-max */
  MEDA_K_NEAREST_SMALL,  /* the same step by the streaming kernel that layers with few kept slots take */
  MEDA_K_GROUP,          /* grouping of the less-important rows by target slot */
  MEDA_K_REDUCE,         /* segmented average */
  MEDA_K_DECODE,         /* decoding-step attention over a cache */
  MEDA_K_CLASSES
};

/* Name of a kernel class ("stats", "sweep", ...), or NULL if out of range. */
const char* meda_kernel_class_name(int32_t kernel_class);

/* Turns per-launch timing on (enable != 0) or off.  Turning it on creates a pool of CUDA events
 * (an allocating call: do it outside timed regions); while on, every kernel launch of a step call
 * is bracketed by two events on the call's stream, up to the pool size, after which launches are
 * still counted but no longer timed. */
meda_status meda_profile_enable(meda_ctx* ctx, int32_t enable);

/* Launches since the last meda_profile_read (or meda_profile_enable) that were NOT timed because
 * the event pool was full.  Per-class times of such a record cover only part of the launches:
 * a caller that divides them by a step count must check that this is 0. */
int64_t meda_profile_dropped(const meda_ctx* ctx);

/* Synchronises the recorded events and writes, per kernel class, the summed device time in
 * milliseconds (ms_out, HOST float[MEDA_K_CLASSES]) and the number of timed launches
 * (launches_out, HOST int32[MEDA_K_CLASSES]); then clears the record.  Either pointer may be NULL. */
meda_status meda_profile_read(meda_ctx* ctx, float* ms_out, int32_t* launches_out);

/* Number of kernels this context has launched since it was created (timing on or off). */
int64_t meda_launch_count(const meda_ctx* ctx);

/* Self-test of the failure path every tensor-core pipeline of the library shares (no counterpart in
 * the paper).  Each device-side wait of those pipelines is bounded: when it runs out, the kernel
 * records MEDA_ERR_TIMEOUT in the context's status word, releases what it holds and returns.  This
 * call launches one small block that waits, with that same routine, on a barrier nothing arrives
 * on, for at most `wait_cycles` cycles of the SM clock (1 .. 2e9; a few thousand is enough), so the
 * path can be exercised without breaking a real kernel: afterwards meda_poll_status returns
 * MEDA_ERR_TIMEOUT once, and the context works as before.  Nothing else is touched. */
meda_status meda_selftest_wait_timeout(meda_ctx* ctx, int64_t wait_cycles, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MEDA_H_ */
