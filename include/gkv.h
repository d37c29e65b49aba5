/*
 * gkv.h -- C ABI of the B200 (sm_100a) G-KV library: decode-time KV-cache eviction with a global
 * attention score, and GQA decode attention over the compressed cache.
 *
 * Method (G-KV paper): Section 3 defines the eviction framework (compress every s generated
 * tokens; the last w tokens are the observation window; keep the top-(b-w) scored tokens per KV
 * head plus the window, so the cache returns to length b), Eq. 1 (window attention), the
 * max-reduce over the query heads of a KV head, and Eq. 2 (local score S = window mean).
 * Section 5 defines the global score F: S is divided by its per-head maximum and merged with the
 * decayed history alpha*F_prev by Eq. 3 (max), Eq. 4 (average) or Eq. 5 (summation); rows
 * without history and the first compression use the normalised S alone; the F of the retained
 * rows is recorded for the next step.
 *
 * Conventions
 *   - Every pointer named in gkv_buffers and every q/k/v/out/q_window/kept_idx argument of the
 *     non-"_host" calls is a DEVICE pointer; the "_host" calls take HOST pointers (pinned memory
 *     recommended). `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - The library owns no device memory: the caller allocates the buffers of gkv_query_sizes,
 *     256-byte aligned, and keeps them alive until gkv_destroy. The context is host memory.
 *   - All work is enqueued on the caller's stream; no call synchronises except
 *     gkv_poll_device_status. Calls on one context must not overlap on the GPU (one stream, or
 *     caller-side ordering).
 *   - Every call returns a gkv_status; nothing is thrown across the boundary. Arguments are
 *     validated before anything is launched; a failed call launches nothing.
 *   - All sequences of the batch advance in lock step (one token per gkv_decode_attn call and
 *     layer), so a layer has one cache length; the host keeps counters that mirror the device
 *     copy.
 *
 * Layouts (d = head_dim = 128, C = budget + buffer rows per head, g = n_q_heads / n_kv_heads <= 8;
 * query head i reads KV head i / g)
 *   k, v     [n_layers][batch][n_kv_heads][C][d]  bf16      rows 0..len-1 valid
 *   f        [n_layers][batch][n_kv_heads][C]     fp32      global score F of rows 0..n_hist-1
 *   sacc     [n_layers][batch][n_kv_heads][C]     fp32      window sums: sum over the window's decode
 *                                                            steps of max over the group of that
 *                                                            step's attention weight (= w * S of Eq. 2)
 *   pos      [n_layers][batch][n_kv_heads][C]     int32     original token position of each row
 *                                                            (only with track_positions)
 *   len      [2][n_layers][batch]                 int32     plane 0: cache length, plane 1: n_hist
 *   q        [batch][n_q_heads][d]                bf16      (with layer = -1: [n_layers] in front)
 *   k_new, v_new [batch][n_kv_heads][d]           bf16      (same)
 *   out      [batch][n_q_heads][d]                bf16      (same)
 *   q_window [batch][n_q_heads][w][d]             bf16      oldest window token first (same)
 *   kept_idx [batch][n_kv_heads][b]               int32     (same)
 */
#ifndef GKV_H_
#define GKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gkv_ctx gkv_ctx; /* opaque, host side, owns no device memory */

typedef enum {
    GKV_OK = 0,
    GKV_ERR_INVALID_ARG = 1, /* NULL pointer, bad layer, inconsistent configuration            */
    GKV_ERR_STATE = 2,       /* call not allowed in the current schedule state                 */
    GKV_ERR_CAPACITY = 3,    /* the cache is full (len == C): evict before decoding further    */
    GKV_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed                            */
    GKV_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired (latched status word)       */
    GKV_ERR_UNSUPPORTED = 6, /* valid but not built (head_dim != 128, g > 8, ...)              */
    GKV_ERR_SCRATCH_LIMIT = 7, /* problem larger than the library's built-in scratch array     */
    GKV_ERR_INTERNAL = 8     /* checked build only (-DGKV_CHECK_BOUNDS): a kernel computed a row index out of
                                range; the access was skipped and the status word latched          */
} gkv_status;

/* Form of the global score (Section 5). LOCAL disables the history: F = normalised S. */
typedef enum { GKV_MODE_MAX = 0, GKV_MODE_MEAN = 1, GKV_MODE_SUM = 2, GKV_MODE_LOCAL = 3 } gkv_mode;
typedef enum { GKV_POLICY_SCORE = 0, GKV_POLICY_STREAMING = 1 } gkv_policy;

typedef struct {
    int32_t n_layers, batch, n_q_heads, n_kv_heads, head_dim; /* head_dim must be 128           */
    int32_t budget;   /* b: cache length after a compression (Section 3)                        */
    int32_t buffer;   /* physical slack: C = budget + buffer rows per head                       */
    int32_t window;   /* w: observation window, 1 <= w < b                                      */
    int32_t interval; /* s: compress every s generated tokens, 1 <= s <= buffer, s >= w         */
    float alpha;      /* memory decay rate of Eq. 3-5, in [0,1]; the paper uses 0.8             */
    int32_t mode;     /* gkv_mode                                                               */
    int32_t fuse_window_scores; /* 1: gkv_decode_attn adds each window token's group-max attention
                                   row to sacc, and gkv_evict needs no q_window                 */
    int32_t track_positions;    /* 1: pos carries original token positions through compaction   */
    /* Redundancy term of the appendix on combining the global score with other methods (off when
     * use_redundancy == 0; the remaining fields are then ignored): the selection runs on
     * lambda * F - (1 - lambda) * R', R' the max-normalised softmax of each key's summed cosine
     * similarity to the cached keys; F itself is what is recorded for the next step. The paper
     * reports lambda = 0.7 / 0.9 as best for its two models and gives no value for the similarity
     * threshold, the number of protected recent tokens or epsilon: they are the caller's. */
    int32_t use_redundancy;
    float redundancy_lambda;    /* in [0,1]                                                       */
    float redundancy_threshold; /* tau > 0: cosine similarities below it count as 0              */
    int32_t redundancy_recent;  /* this many most recent tokens are never rated redundant, >= 0  */
    float redundancy_eps;       /* epsilon of the key normalisation K / (|K| + eps), >= 0        */
    /* SnapKV combination of the same appendix: sequence-wise max-pooling (this kernel size, odd; 0 or 1 =
     * off; window clipped at the ends of the candidate range) of the global score before the selection
     * (and before the redundancy term, if both are on). The unpooled F is what is recorded. The paper
     * gives no kernel size and reports that pooling does not help at decode time. */
    int32_t pool_kernel;
    /* Longest prompt gkv_compress_prompt will be given (rows per head of its K / V buffers); 0 = that call is
     * not used. At most 1048576; above 8192 the window must be a multiple of 16 (UNSUPPORTED
     * otherwise) and q_window 16-byte aligned. Sizes part of the workspace (4 bytes per prompt token and KV head, twice or three times
     * that above 8192). */
    int32_t max_prompt;
    /* Selection policy. GKV_POLICY_SCORE (0): the paper's method, top-(b-w) by the global score. GKV_POLICY_STREAMING:
     * the sink-plus-recent policy of StreamingLLM, one of the baselines of the paper's experimental setup, as a
     * score-free selection on the same compaction path: every compression keeps the first n_sink rows of the cache
     * (the attention sinks; 0 <= n_sink <= b - w) and the most recent b - n_sink rows. No window scores or q_window
     * are needed (they are ignored), the recorded scores are 0, the redundancy term and pooling must be off. */
    int32_t policy;
    int32_t n_sink;
} gkv_config;

typedef struct { uint64_t k, v, f, sacc, pos, len, workspace, staging; } gkv_sizes; /* bytes      */
typedef struct { void *k, *v, *f, *sacc, *pos, *len, *workspace, *staging; } gkv_buffers;

/* Bytes of each caller-allocated device buffer for a configuration. `pos` is 0 without
 * track_positions. `staging` is only needed by the "_host" calls (may be left NULL otherwise).
 * Errors: INVALID_ARG (NULL, non-positive sizes, w >= b, s > buffer, s < w, alpha outside [0,1],
 * n_q_heads not a multiple of n_kv_heads), UNSUPPORTED (head_dim != 128, g > 8, C > 4096). */
gkv_status gkv_query_sizes(const gkv_config* cfg, gkv_sizes* out);

/* Create a context over caller-owned device buffers and enqueue on `stream` the zeroing of k, v,
 * f, sacc, pos, len and workspace (an empty cache: len = 0, no history). Encodes the TMA
 * descriptors of k and v. The device current at this call is the context's device.
 * Errors: as gkv_query_sizes; INVALID_ARG for a NULL or misaligned required buffer; CUDA. */
gkv_status gkv_init(gkv_ctx** out, const gkv_config* cfg, const gkv_buffers* buffers, void* stream);

/* Declare that the caller has filled the cache directly: rows 0..len-1 of k, v (and pos), the
 * global scores of rows 0..n_hist-1 of f, and -- when window_scores_valid != 0 -- sacc holding the
 * window sums of the last w tokens. Sets the host counters and enqueues the device copies.
 * layer = -1 applies to all layers. since_evict is the number of tokens decoded since the last
 * compression. Errors: INVALID_ARG (len > C, n_hist > len, bad layer). */
gkv_status gkv_set_state(gkv_ctx* ctx, int32_t layer, int32_t len, int32_t n_hist, int32_t since_evict,
                         int32_t window_scores_valid, void* stream);

/* One decode step of attention (standard GQA attention over the compressed cache; the every-step
 * part of the path whose cost Section 6.4 measures): append k_new, v_new at row len, then
 * out[i] = sum_t softmax_t(q_i . K[i/g, t] / sqrt(d)) V[i/g, t] over t <= len (the new token
 * included); len += 1. With fuse_window_scores, the last w steps before a scheduled compression
 * also add max over the group of the final attention weights to sacc (this token's row of the
 * group max that Eq. 2 averages). layer = -1 runs all layers in one launch with every tensor
 * argument carrying a leading [n_layers] dimension. q, k_new, v_new and out are 16-byte aligned.
 * Errors: CAPACITY (len == C, nothing launched); STATE (fuse_window_scores and a compression is
 * due: since_evict == interval); INVALID_ARG (NULL or misaligned pointer, bad layer); CUDA. */
gkv_status gkv_decode_attn(gkv_ctx* ctx, int32_t layer, const void* q, const void* k_new,
                           const void* v_new, void* out, void* stream);

/* One compression step (Section 3 framework; Eq. 1-2 local score; Section 5 normalisation and
 * Eq. 3-5 merge; top-(b-w) per KV head, equal scores resolved toward the lower position; kept
 * rows in ascending position followed by the w window rows; K, V, F (and pos) compacted in
 * place; len = b, n_hist = b-w, sacc = 0, since_evict = 0).
 *   q_window == NULL : the local score is read from sacc (requires fuse_window_scores and
 *                      since_evict == interval, or gkv_set_state(window_scores_valid = 1));
 *   q_window != NULL : the local score is recomputed from the window queries and K (Eq. 1-2),
 *                      each window token seeing the keys up to and including its own.
 *   kept_idx_out     : optional; receives the pre-compaction row index of every kept row.
 * With use_redundancy the step first computes every key's redundancy level (two more launches: key
 * norms, then the thresholded cosine-similarity sums on the tensor cores) and selects on the
 * combined score of the appendix.
 * If len <= b nothing is evicted: the call only resets since_evict and sacc.
 * layer = -1 compresses all layers in one launch (leading [n_layers] dimension on the arguments).
 * Errors: STATE (no valid window scores and no q_window; len < w), INVALID_ARG, CUDA. */
gkv_status gkv_evict(gkv_ctx* ctx, int32_t layer, const void* q_window, int32_t* kept_idx_out,
                     void* stream);

/* The stages of gkv_evict as separate launches, for timing them one by one. They communicate
 * through the workspace and must be called in order SCORE (only with q_window) -> REDUNDANCY (only
 * with use_redundancy, then required) -> MERGE -> SELECT -> COMPACT on ONE layer (layer = -1 is
 * UNSUPPORTED: the staged scratch holds one layer); after COMPACT the state equals that after
 * gkv_evict. Results are identical to gkv_evict. kept_idx_out is taken by SELECT.
 * Errors: as gkv_evict; STATE for an out-of-order stage; INVALID_ARG for an unknown stage, SCORE
 * without q_window, or REDUNDANCY with the term off. */
typedef enum { GKV_STAGE_SCORE = 0, GKV_STAGE_MERGE = 1, GKV_STAGE_SELECT = 2, GKV_STAGE_COMPACT = 3,
               GKV_STAGE_REDUNDANCY = 4 /* only with use_redundancy: after SCORE (if any), before MERGE */ } gkv_stage;
gkv_status gkv_evict_stage(gkv_ctx* ctx, int32_t layer, int32_t stage, const void* q_window,
                           int32_t* kept_idx_out, void* stream);

/* Same operations with HOST buffers: inputs are copied to the staging buffer on `stream`, the
 * kernels run, and the result is copied back, all asynchronously on `stream` (synchronise the
 * stream before reading out / kept_idx_out). Require buffers.staging.
 * gkv_decode_attn_host takes a faster route when all four of its buffers are page-locked and mapped
 * (cudaHostAlloc, cudaHostRegister, a pinned torch tensor): the kernel reads and writes them in place
 * across the bus (zero copy, no staging buffer needed), which overlaps the transfers with the
 * attention. The result is again complete once `stream` has been synchronised.
 * Errors: as the device calls; INVALID_ARG when staging is needed and no staging buffer was given. */
gkv_status gkv_decode_attn_host(gkv_ctx* ctx, int32_t layer, const void* q_host, const void* k_new_host,
                                const void* v_new_host, void* out_host, void* stream);
gkv_status gkv_evict_host(gkv_ctx* ctx, int32_t layer, const void* q_window_host,
                          int32_t* kept_idx_out_host, void* stream);

/* (No counterpart in the paper: an engineering variant of gkv_decode_attn.)
 * One decode-attention step for ONE layer that needs no workspace, no context and no device
 * allocation: for callers that cannot obtain device memory when they call -- a plug-in running
 * inside a server whose memory pool it does not own, or a latency-critical loop where cudaMalloc is
 * off limits because it synchronises the device and may fail late. The caller passes only inputs and
 * outputs (device pointers): q [batch][n_q_heads][128], k_new / v_new [batch][n_kv_heads][128],
 * k_cache / v_cache [batch][n_kv_heads][capacity][128], out [batch][n_q_heads][128], all bf16 and
 * 16-byte aligned. Semantics are those of gkv_decode_attn without window-score accumulation: k_new, v_new are
 * written to row `len` of every head's cache and out is the attention over rows 0..len; the caller
 * keeps track of `len` itself (it is passed by value, nothing is read back).
 * The length words, completion and work counters and the status word live in an array of 8.25 KiB
 * that is part of the library's device image: every GPU that loads the library holds it until the
 * process exits. Limit: batch <= 1024 (one length word and one counter per sequence); beyond it the
 * call returns GKV_ERR_SCRATCH_LIMIT and launches nothing.
 * All calls on a device share that array and it keeps the previous call's contents; each call clears
 * the words that must start at zero. Calls that overlap on the GPU (two streams, or unordered host
 * threads) race on the array and produce wrong results: keep them ordered.
 * The first call on each device resolves the array's device address (with that device current);
 * make that first call outside any stream capture. The call itself performs no cudaMalloc / cudaFree.
 * A bounded wait that expires inside the kernel cannot be polled through this entry point; `out` is
 * then undefined.
 * Errors: INVALID_ARG (NULL, non-positive sizes, a pointer not 16-byte aligned), UNSUPPORTED (g > 8, capacity > 4096),
 * CAPACITY (len >= capacity), SCRATCH_LIMIT, CUDA. */
gkv_status gkv_decode_attn_static(const void* q, const void* k_new, const void* v_new, void* k_cache,
                                  void* v_cache, void* out, int32_t batch, int32_t n_q_heads,
                                  int32_t n_kv_heads, int32_t capacity, int32_t len, void* stream);

/* First compression of a freshly prefilled prompt that may be longer than the cache (Section 3 starts from a
 * prefilled cache; Section 5: the first compression uses the normalised local score alone, no history).
 * k_prompt, v_prompt: device, [batch][n_kv_heads][max_prompt][128] bf16 (16-byte aligned), sequence i holding
 * prompt_len_host[i] rows (HOST array of batch int32, 1..max_prompt; lengths may differ per sequence).
 * q_window: device, [batch][n_q_heads][w][128], the queries of each prompt's last w tokens, oldest first
 * (may be NULL when no prompt is longer than b). Per sequence and KV head: a prompt of at most b tokens is
 * copied whole into cache rows 0..len-1 (n_hist = 0); a longer one keeps the top-(b-w) of its first
 * len - w tokens by the max-normalised window score (Eq. 1-2, after the optional pooling and, with
 * use_redundancy, the redundancy term over the prompt's keys) plus the last w tokens, in ascending position, in rows 0..b-1, with F of
 * the kept rows recorded and pos = position in the prompt (with track_positions). sacc of the layer is
 * cleared, since_evict = 0. kept_idx_out (optional, device [batch][n_kv_heads][b]) receives the kept
 * prompt positions, -1 padded. One layer per call (prefill proceeds layer by layer).
 * Afterwards the sequences of the layer may have different cache lengths: the device keeps one length per
 * sequence, every later call handles each sequence at its own length (a scheduled compression evicts
 * nothing from a sequence that holds at most b tokens), and the host counters of gkv_get_state follow the
 * longest sequence.
 * Errors: STATE (max_prompt == 0), INVALID_ARG (NULL / misaligned pointer, layer = -1, a length outside
 * 1..max_prompt, q_window == NULL with a prompt longer than b), CUDA. */
gkv_status gkv_compress_prompt(gkv_ctx* ctx, int32_t layer, const void* k_prompt, const void* v_prompt,
                               const void* q_window, const int32_t* prompt_len_host, int32_t* kept_idx_out,
                               void* stream);

/* Eviction log (what the paper's sparse-training recipes need to rebuild the attention mask of a compressed
 * rollout: which tokens left the cache at which compression step). After this call every gkv_evict /
 * SELECT stage also writes, for each (layer, sequence, KV head) it processes, the tokens it evicted into
 * log_device [n_layers][batch][n_kv_heads][buffer] int32 (device pointer, caller-owned, kept alive while
 * set): original token positions when track_positions is on, else pre-compaction row indices; ascending;
 * unused entries (a step evicts len - b <= buffer tokens) are -1; a step that evicts nothing writes all -1.
 * Only the layers of the call are written. NULL switches the log off.
 * Errors: INVALID_ARG (NULL context, misaligned pointer). */
gkv_status gkv_set_eviction_log(gkv_ctx* ctx, int32_t* log_device);

/* With use_redundancy: copies the redundancy levels cbar (summed thresholded cosine similarity of every
 * cached key, 0 for the protected recent tokens) that the last gkv_evict / REDUNDANCY stage computed for
 * `layer` into out_device [batch][n_kv_heads][C] fp32 (device pointer), asynchronously on `stream`.
 * The values refer to the rows as they were BEFORE that step's compaction.
 * Errors: INVALID_ARG (NULL, bad layer, layer = -1), STATE (redundancy term off), CUDA. */
gkv_status gkv_get_redundancy(gkv_ctx* ctx, int32_t layer, float* out_device, void* stream);

/* Host counters of one layer (no synchronisation): cache length, rows with history, tokens
 * decoded since the last compression. Any output pointer may be NULL. */
gkv_status gkv_get_state(const gkv_ctx* ctx, int32_t layer, int32_t* len, int32_t* n_hist,
                         int32_t* since_evict);

/* Number of kernels this context has launched so far (host counter). */
int64_t gkv_launch_count(const gkv_ctx* ctx);

/* Synchronises `stream` and returns GKV_ERR_TIMEOUT if any kernel latched an expired bounded
 * wait since the last poll (GKV_ERR_INTERNAL if a library built with -DGKV_CHECK_BOUNDS caught a row index out of
 * range), GKV_ERR_CUDA on a CUDA error, else OK. On TIMEOUT the latch and the
 * kernels' completion and work counters in the workspace are cleared, so the context can be used
 * again; what the kernel that gave up had written (outputs, cache rows, lengths) is undefined:
 * declare the state anew with gkv_set_state before going on. */
gkv_status gkv_poll_device_status(gkv_ctx* ctx, void* stream);

/* Self-test of the failure path (no paper counterpart): launches one warp that waits, through the same bounded-wait
 * helper every kernel of the library uses, on a barrier nobody arrives on, with a limit of `spins` polls
 * (1..65536; microseconds). The wait runs out, the kernel latches the status word and returns: nothing traps,
 * faults or hangs. The next gkv_poll_device_status reports GKV_ERR_TIMEOUT once, and the context stays usable
 * (the cache state is untouched by this call). Errors: INVALID_ARG, CUDA. */
gkv_status gkv_selftest_bounded_wait(gkv_ctx* ctx, int32_t spins, void* stream);

/* How gkv_decode_attn would launch its kernel (no paper counterpart: a view of the host-side planning, for
 * capacity planning and for tests that need no GPU). n_layers_in_launch = 1 (one layer per call) or
 * cfg->n_layers (layer = -1); window_step != 0 for a step that accumulates window scores; sm_count = SMs of the
 * device (<= 0: 148). grid = CTAs launched (persistent: never more than are resident at once), splits = pieces a
 * unit's keys are split into (> 1: the pieces of a unit form one thread-block cluster of that size), stages = depth
 * of the K/V tile ring, ctas_per_sm = resident CTAs per SM, smem_bytes = dynamic shared memory per CTA,
 * tmem_cols = tensor-memory columns per CTA on window steps. Pure host arithmetic.
 * Errors: as gkv_query_sizes; INVALID_ARG for a layer count other than 1 or cfg->n_layers. */
typedef struct { int32_t grid, splits, stages, ctas_per_sm, smem_bytes, tmem_cols; } gkv_decode_plan_t;
gkv_status gkv_decode_launch_plan(const gkv_config* cfg, int32_t n_layers_in_launch, int32_t window_step,
                                  int32_t sm_count, gkv_decode_plan_t* out);

/* How gkv_evict would launch its fused kernel (no paper counterpart; host arithmetic, for capacity planning and tests
 * without a GPU; the eviction log, which adds C - b words of shared memory, is taken as off): grid = CTAs launched
 * (persistent: at most the resident ones; with three rounds of units or fewer the rounds are filled equally), stages =
 * depth of the copy ring (32 rows of K and V per stage), ctas_per_sm, smem_bytes = dynamic shared memory per CTA.
 * Errors: as gkv_query_sizes; INVALID_ARG for a layer count other than 1 or cfg->n_layers. */
typedef struct { int32_t grid, stages, ctas_per_sm, smem_bytes; } gkv_evict_plan_t;
gkv_status gkv_evict_launch_plan(const gkv_config* cfg, int32_t n_layers_in_launch, int32_t sm_count, gkv_evict_plan_t* out);

/* How the recompute path would launch its tensor-core scoring kernel on the cache (no paper counterpart; host
 * arithmetic, for capacity planning and tests without a GPU). tensor_core = 0 when the window is not a multiple of 16
 * (the other scoring kernel runs; the remaining fields are 0). items = work items (a unit and up to 64 window rows of
 * all its heads), rows_per_item = query rows of an item, grid = CTAs launched (persistent, one per SM at most, rounds
 * filled equally), stages = depth of the ring of 128-key tiles, query_buffers = 1 or 2, smem_bytes = dynamic shared
 * memory per CTA. With at most 128 query rows per item the ring depth is even (the kernel's two issuing threads then
 * take alternate tiles, and a ring slot must stay with one of them).
 * Errors: as gkv_query_sizes; INVALID_ARG for a layer count other than 1 or cfg->n_layers. */
typedef struct { int32_t tensor_core, grid, items, rows_per_item, stages, query_buffers, smem_bytes; } gkv_score_plan_t;
gkv_status gkv_score_launch_plan(const gkv_config* cfg, int32_t n_layers_in_launch, int32_t sm_count, gkv_score_plan_t* out);

/* Memory model of the paper's appendix "Memory Analysis": bytes of the full KV cache at
 * seq_len tokens, of the compressed cache ((b + s) rows instead of seq_len), and of the score
 * cache F (b - w entries per head), for `elem_bytes`-wide elements, over all layers and the
 * whole batch. Pure host arithmetic. */
typedef struct { uint64_t full_kv, compressed_kv, score_cache; } gkv_memory_model_t;
gkv_status gkv_memory_model(const gkv_config* cfg, int64_t seq_len, int32_t elem_bytes,
                            gkv_memory_model_t* out);

const char* gkv_strerror(gkv_status status);

/* Frees the host context only; device buffers stay with the caller. NULL is allowed. */
void gkv_destroy(gkv_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* GKV_H_ */
