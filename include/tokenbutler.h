/*
 * tokenbutler.h -- C ABI of the B200 (sm_100a) decode hot path of TokenButler.
 *
 * The path, per layer, per KV head and per decode step (paper Sec. 3.1, 3.3, 3.4, Sec. 4
 * "Token Selection Policy"):
 *   append_kv / project_keys   keep the full, never-evicted KV cache and, beside it, the cache of
 *                              keys projected to the low "interaction" dimension d'
 *   score_tokens               dot product of the importance query with every projected key
 *   select_topk                top-B of the candidates (everything but S sink and W recent tokens),
 *                              optional neighbour fetching, reuse of a selection for P steps
 *   sparse_decode_attention    softmax attention over sinks + selected rows + recent window only
 *
 * Conventions
 *   - Every pointer named *_dev is DEVICE memory, every other pointer is HOST memory that is read
 *     before the call returns.  The library never allocates or frees device memory: the caller
 *     allocates the four regions sized by tb_query_sizes() (256-byte aligned) and binds them with
 *     tb_create().  `stream` is a cudaStream_t passed as void*; all work is enqueued on it and the
 *     call returns without synchronising (tb_get_status is the one exception).
 *   - Errors are return codes only.  Every error but TB_ERR_CUDA is found on the host before the call's
 *     first launch (for all of the call's layers): such a call has changed no state and launched nothing.
 *     TB_ERR_CUDA means that the CUDA runtime refused a launch or a copy in mid-call: earlier launches of
 *     that call may have run, and the sequences it named must be reset (tb_reset_sequence) before they
 *     are used again.  Problems only the device can see (an out-of-range entry in a caller-supplied
 *     index list, an internal wait that ran out) set a device status word, skip the offending access
 *     and let the kernel finish; tb_get_status() reads and clears that word.
 *   - Shapes: B sequences, Hq query heads, Hkv KV heads, g = Hq/Hkv, D = head_dim (128),
 *     d' = imp_dim (16 or 32).  kv_dtype is the storage type of K, V, K_imp, W_K and q; importance
 *     queries, scores, outputs and log-sum-exps are fp32.  All arithmetic accumulates in fp32.
 *
 * Device layouts (row-major, element = kv_dtype)
 *   kv    [n_layers][max_batch][Hkv][max_seq_len][2][D]   K row then V row of a token, adjacent
 *   kimp  [n_layers][max_batch][Hkv][max_seq_len][d']     ([1] in place of [Hkv] under TB_SCOPE_LAYER)
 *   W_K   [Hkv][D][d'] per layer (one D x d' matrix per layer AND per KV head)
 *   index lists: int32 rows of tb_index_capacity() entries, ascending token positions
 */
#ifndef TOKENBUTLER_H_
#define TOKENBUTLER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TB_OK = 0,
    TB_ERR_INVALID_ARG = -1,  /* null pointer, index out of range, empty problem               */
    TB_ERR_UNSUPPORTED = -2,  /* shape / mode outside the compiled set                         */
    TB_ERR_CAPACITY = -3,     /* append beyond max_seq_len, budget beyond max_budget, ...      */
    TB_ERR_UNPROJECTED = -4,  /* selection asked over keys that have not been projected yet    */
    TB_ERR_STATE = -5,        /* attention from the stored list before any selection           */
    TB_ERR_CUDA = -6,         /* a CUDA runtime call failed                                    */
    TB_ERR_TIMEOUT = -7,      /* device status: an internal bounded wait ran out               */
    TB_ERR_BAD_INDEX = -8     /* device status: caller-supplied index outside [0, L)           */
} tb_status;

typedef enum { TB_F32 = 0, TB_BF16 = 1 } tb_dtype;
/* How the g importance queries of a GQA group become one ranking per KV head: a token's score is the
 * sum (default) or the largest of the group's g head scores.  TB_PER_QHEAD asks for no reduction: it is
 * accepted by a context whose lists are per query head (TB_SCOPE_Q_HEAD below), where it is the only
 * meaning there is, and refused with TB_ERR_UNSUPPORTED by a context whose lists are per KV head.  On a
 * context with one importance query per list (TB_SCOPE_Q_HEAD, TB_SCOPE_LAYER) all three mean the same. */
typedef enum { TB_GROUP_SUM = 0, TB_GROUP_MAX = 1, TB_PER_QHEAD = 2 } tb_group_reduce;
/* Which heads share one index list (paper Sec. 3.1: importance is predicted per head; App. "additional
 * evaluation": a head-less predictor with one importance per token and layer).  Fixed per context,
 * since it sizes the projected-key cache and the lists:
 *   TB_SCOPE_KV_HEAD  one list per KV head; the g query heads of a group share the gathered rows.
 *                     q_imp [..][Hq][d'], kimp [..][Hkv][max_seq_len][d'], lists [..][Hkv].
 *   TB_SCOPE_Q_HEAD   one list per query head, ranked by that head's importance query against its KV
 *                     head's projected keys; no row sharing in attention.  q_imp [..][Hq][d'], kimp as
 *                     above, lists [..][Hq].
 *   TB_SCOPE_LAYER    one list per layer, shared by every head.  One importance query per layer,
 *                     q_imp [..][1][d'], and one projected key per token, kimp [..][1][max_seq_len][d'] =
 *                     sum over KV heads h of K[h] . W_K[h] (the [Hkv*D] x d' projection of the token's
 *                     concatenated key); lists [..][1].
 * In the calls below, "[Hl]" stands for the number of lists per (layer, sequence): Hkv, Hq or 1. */
typedef enum { TB_SCOPE_KV_HEAD = 0, TB_SCOPE_Q_HEAD = 1, TB_SCOPE_LAYER = 2 } tb_list_scope;
/* Neighbour fetching (Sec. 3.4): DILATE = every position within +-radius of a selected one;
 * CLUSTER = runs of consecutive selected positions get radius*len extra positions just outside the
 * run (ceil half after it, floor half before it). */
typedef enum { TB_NEIGHBOR_DILATE = 0, TB_NEIGHBOR_CLUSTER = 1 } tb_neighbor_mode;

typedef struct {
    int32_t n_layers, n_q_heads, n_kv_heads, head_dim, imp_dim;
    int32_t kv_dtype;      /* tb_dtype                                                       */
    int32_t max_batch;     /* sequences the caches hold                                      */
    int32_t max_seq_len;   /* token capacity per sequence                                    */
    int32_t max_budget;    /* largest `budget` any select call will use                      */
    int32_t max_radius;    /* largest neighbour radius; lists hold (2*max_radius+1)*max_budget */
    int32_t device;        /* CUDA device ordinal the regions live on                        */
    int32_t list_scope;    /* tb_list_scope; 0 = one list per KV head                        */
} tb_config;

typedef struct {
    int32_t budget;        /* dynamic tokens kept per KV head; < 0 in attention = dense       */
    int32_t sinks;         /* S: first S tokens always attended, never candidates             */
    int32_t recent;        /* W: last W tokens always attended, never candidates              */
    int32_t radius;        /* neighbour radius r (0 = off)                                    */
    int32_t nmode;         /* tb_neighbor_mode                                                */
    int32_t interval;      /* P: selection refreshed iff step % interval == 0                 */
    int32_t step;          /* decode step counted from the first sparse step                  */
    int32_t reduce;        /* tb_group_reduce                                                 */
    float score_scale;     /* positive factor applied to materialised scores only             */
} tb_select_params;

typedef struct tb_ctx tb_ctx;

/* Sizes (bytes) of the four caller-allocated device regions for this configuration.
 * Errors: TB_ERR_INVALID_ARG (null, non-positive sizes, Hq % Hkv != 0),
 * TB_ERR_UNSUPPORTED (head_dim != 128, imp_dim not in {16,32}, group size > 8). */
tb_status tb_query_sizes(const tb_config* cfg, size_t* kv_bytes, size_t* kimp_bytes,
                         size_t* state_bytes, size_t* workspace_bytes);

/* Bind the four regions (256-byte aligned device pointers; contents of kv/kimp may be anything,
 * state and workspace are cleared here with a synchronous memset).  The context owns nothing on the
 * device; tb_destroy frees only host memory.  All sequences start empty.
 * Offloaded KV (paper Sec. 4.4 "CPU-offloaded KV"): kv_dev alone may instead be page-locked host
 * memory that the device addresses through the same pointer (cudaHostAlloc under unified addressing).
 * Every call then works unchanged: appends and projections cross the host link, and attention fetches
 * only the rows it attends to; the projected keys, lists and workspace stay in device memory.  Any
 * pointer that is neither is refused here with TB_ERR_INVALID_ARG (it would fault in a kernel later). */
tb_status tb_create(const tb_config* cfg, void* kv_dev, void* kimp_dev, void* state_dev,
                    void* workspace_dev, tb_ctx** out);
tb_status tb_destroy(tb_ctx* ctx);

/* Entries per index-list row: (2*max_radius+1)*max_budget rounded up to a multiple of 4. */
int32_t tb_index_capacity(const tb_ctx* ctx);

/* Copy one layer's key projection W_K [Hkv][D][d'] (kv_dtype, device) into the context's state
 * (Sec. 3.1: learned matrix of the key-cache projection). */
tb_status tb_set_projection(tb_ctx* ctx, int32_t layer, const void* W_dev, void* stream);

/* Forget a sequence in every layer: length and projected length 0 (host mirrors and, when the kernels read
 * them, the device counters, with a blocking clear: call it when no work on that sequence is in flight), stored
 * selections dropped. */
tb_status tb_reset_sequence(tb_ctx* ctx, int32_t seq);

/* Host-side view of a sequence: tokens cached and tokens whose keys are projected. */
tb_status tb_get_length(const tb_ctx* ctx, int32_t layer, int32_t seq, int32_t* len, int32_t* len_projected);

/* Sec. 3.3: write new tokens' K and V rows at the end of each listed sequence, for layers
 * [layer_begin, layer_begin+layer_count).  k_dev, v_dev: [layer_count][sum(n_new)][Hkv][D], the
 * tokens of the listed sequences concatenated in list order.  seq_ids == NULL means 0..n_seq-1.
 * TB_ERR_CAPACITY if any sequence would exceed max_seq_len (nothing is written). */
tb_status tb_append_kv(tb_ctx* ctx, int32_t layer_begin, int32_t layer_count, const int32_t* seq_ids,
                       const int32_t* n_new, int32_t n_seq, const void* k_dev, const void* v_dev, void* stream);

/* Sec. 3.1 "Key-cache projection" K_imp = K W_K for token positions [pos_begin[i], pos_end[i]) of
 * each listed sequence (fp32 accumulation -- tensor-core tiles for bf16 storage, an FMA chain in
 * channel order for fp32 storage -- and one round-to-nearest-even to kv_dtype; a row's result does
 * not depend on which call or batch projected it).  Eager (one token) or deferred batches
 * (Sec. 3.3) are both just ranges.  Ranges must
 * lie inside the cached tokens and start at or before the sequence's projected length (no holes).
 * pos_begin == pos_end == NULL means "everything cached and not yet projected", [projected length, length) of
 * every listed (layer, sequence), read on the device -- the form a captured graph can replay. */
tb_status tb_project_keys(tb_ctx* ctx, int32_t layer_begin, int32_t layer_count, const int32_t* seq_ids,
                          const int32_t* pos_begin, const int32_t* pos_end, int32_t n_seq, void* stream);

/* Sec. 3.4 / App. E importance scores of ALL projected tokens, materialised:
 * scores_dev[i][h][t] = score_scale * sum_j qr[i][h][j] * K_imp[seq_i][h][t][j], t < projected length,
 * h < Hl, row stride max_seq_len, entries past the projected length untouched.  q_imp_dev [n_seq][Hq][d']
 * fp32 ([n_seq][1][d'] under TB_SCOPE_LAYER); qr = sum of the importance queries that share list h
 * (TB_GROUP_SUM), or the score is the largest of their dot products (TB_GROUP_MAX).  The fast path
 * (tb_select_topk) never materialises scores. */
tb_status tb_score_tokens(tb_ctx* ctx, int32_t layer, const int32_t* seq_ids, int32_t n_seq,
                          const float* q_imp_dev, int32_t reduce, float score_scale, float* scores_dev, void* stream);

/* Sec. 4 "Token Selection Policy" + Sec. 3.4 interval / neighbour fetching, fused with scoring, for
 * layers [layer_begin, layer_begin+layer_count) (Sec. 3.3: predictor work is batched over the
 * consumer layers of a producer).  If params->step % params->interval != 0 nothing is launched and
 * the stored lists stay (stale reuse).  Otherwise, per (layer, sequence, list): candidates are
 * positions [min(S,L), max(min(S,L), L-W)); the `budget` highest scores are kept (all candidates if
 * fewer), equal scores resolved toward the LOWER position, -0.0 == +0.0; the list is expanded by the
 * neighbour rule, clipped to the candidates, and stored ascending in the context.
 * q_imp_dev: [layer_count][n_seq][Hq][d'] fp32 ([..][1][d'] under TB_SCOPE_LAYER).  idx_out_dev /
 * cnt_out_dev (optional, may be NULL): copies of the stored lists, [layer_count][n_seq][Hl][tb_index_capacity()]
 * and [..][Hl].
 * TB_ERR_UNPROJECTED if a candidate range is not fully projected; TB_ERR_CAPACITY if budget or radius
 * exceed the configured maxima. */
tb_status tb_select_topk(tb_ctx* ctx, int32_t layer_begin, int32_t layer_count, const int32_t* seq_ids,
                         int32_t n_seq, const float* q_imp_dev, const tb_select_params* params,
                         int32_t* idx_out_dev, int32_t* cnt_out_dev, void* stream);

/* Sec. 3.3 attention of one decode token per listed sequence over
 * sinks [0,min(S,L)) + index list + window [max(min(S,L),L-W), L) of the full cache, each gathered
 * K/V row shared by the g query heads of its KV head (by no one under TB_SCOPE_Q_HEAD, where every
 * query head gathers its own list's rows; under TB_SCOPE_LAYER every KV head reads the layer's one
 * list); split over the rows with a fixed partition and
 * merged in a fixed order (bit-reproducible).  q_dev [layer_count][n_seq][Hq][D] kv_dtype;
 * out_dev [layer_count][n_seq][Hq][D] fp32; lse_dev (optional) [layer_count][n_seq][Hq] natural-log
 * sum-exp of the scaled logits.  idx_dev/cnt_dev: caller lists laid out like tb_select_topk's
 * outputs, or both NULL to use the lists stored by the last selection (TB_ERR_STATE if none).
 * params->budget < 0 selects the dense rule (every cached token; sinks/recent/lists ignored).
 * sm_scale <= 0 means 1/sqrt(D). */
tb_status tb_sparse_decode_attention(tb_ctx* ctx, int32_t layer_begin, int32_t layer_count,
                                     const int32_t* seq_ids, int32_t n_seq, const void* q_dev,
                                     const tb_select_params* params, const int32_t* idx_dev,
                                     const int32_t* cnt_dev, float sm_scale, float* out_dev, float* lse_dev,
                                     void* stream);

/* Allocation-free variant of the attention entry point.  (The paper has no counterpart: this exists
 * for callers that cannot allocate device memory when they need attention -- a plugin inside a
 * serving process whose memory pool was fixed at start-up, a latency-critical thread on which
 * cudaMalloc, which may synchronise the device, is forbidden, or a host that has given all free HBM
 * to its KV cache.)  It needs no tb_ctx and no workspace: the split partials and arrival counters
 * live in a fixed array inside the library image, about 1.1 MB that every GPU loading the library
 * holds until the process exits.  The call itself allocates and frees nothing.
 *
 *   kv_dev     one layer's cache [slot][Hkv][max_seq_len][2][D] in kv_dtype (same row layout as above)
 *   seq_slots  (host, NULL = 0..n_seq-1) cache slot of each listed sequence; seq_lens (host) tokens cached
 *   q_dev      [n_seq][Hq][D] kv_dtype;  out_dev [n_seq][Hq][D] fp32;  lse_dev optional [n_seq][Hq]
 *   idx_dev / cnt_dev  caller lists [n_seq][Hkv][idx_stride] / [n_seq][Hkv] (ascending positions inside the
 *              candidate range), or both NULL for dense attention; entries outside [0, len) are skipped and
 *              recorded as TB_ERR_BAD_INDEX in a status word inside the same array, which tb_static_get_status
 *              returns and clears
 *   sinks, recent, sm_scale  as in tb_sparse_decode_attention
 *
 * Limits: n_seq * Hq <= TB_STATIC_MAX_QHEADS and n_seq <= 64, otherwise TB_ERR_CAPACITY and nothing is
 * launched.  kv_dev must be memory of the current device (or page-locked host memory the device can
 * address), else TB_ERR_INVALID_ARG.  The first call on each device looks up the array's device address (that device must be
 * current) and configures the kernel; make that first call outside any stream capture.  All calls in
 * the process share the one array: the counters are cleared on `stream` at the start of every call, and
 * two calls whose kernels overlap on the GPU (different streams, no ordering) race on the partials. */
#define TB_STATIC_MAX_QHEADS 64
tb_status tb_sparse_decode_attention_static(const void* kv_dev, int32_t kv_dtype, int32_t n_q_heads, int32_t n_kv_heads,
                                            int32_t head_dim, int32_t max_seq_len, const int32_t* seq_slots,
                                            const int32_t* seq_lens, int32_t n_seq, const void* q_dev,
                                            const int32_t* idx_dev, const int32_t* cnt_dev, int32_t idx_stride,
                                            int32_t sinks, int32_t recent, float sm_scale, float* out_dev,
                                            float* lse_dev, void* stream);
/* Synchronise `stream` and return, then clear, the status word of the allocation-free entry point on
 * the current device (TB_OK or TB_ERR_BAD_INDEX).  Allocates nothing. */
tb_status tb_static_get_status(void* stream, int32_t* device_status);

/* Importance-query predictor forward (paper Sec. 3.1 "Query prediction"; App. A: a two-layer MLP with
 * hidden size 512 at every producer layer; Table 6's parameter counts fix bias-free linears and a layer
 * norm with weight and bias).  For each of n_tokens hidden states h [model_dim] (one per decoding
 * sequence):   q = W2 . act(W1 . LN(h)),   LN over the model_dim channels with biased variance and
 * ln_eps inside the root.  The paper does not name the activation; TB_ACT_GELU (exact erf form) is this
 * library's reading, SiLU and ReLU are offered.  It is the step right before tb_select_topk: the output
 *   q_imp_dev [n_slots][n_tokens][n_q_heads][imp_dim] fp32
 * is laid out so that the n_slots consumer layers of a producer can be selected with one
 * tb_select_topk(layer_begin = first consumer, layer_count = n_slots, q_imp_dev).
 *   hidden_dev   [n_tokens][model_dim] in `dtype`
 *   ln_weight, ln_bias [model_dim]; w1 [hidden_dim][model_dim]; w2 [n_slots][n_q_heads][imp_dim][hidden_dim],
 *                row-major (one row per output), all in `dtype`, device memory owned by the caller
 *   scratch_dev  n_tokens * hidden_dim floats of device memory (contents undefined afterwards)
 * All device pointers 16-byte aligned; model_dim and hidden_dim multiples of 8 (bf16) or 4 (fp32) and
 * hidden_dim <= 1536, else TB_ERR_UNSUPPORTED; n_tokens <= 64, else TB_ERR_CAPACITY.  Needs no tb_ctx, keeps no pointer, enqueues two
 * kernels on `stream` and returns. */
typedef enum { TB_ACT_GELU = 0, TB_ACT_SILU = 1, TB_ACT_RELU = 2 } tb_activation;
typedef struct {
    int32_t dtype;                        /* tb_dtype of the hidden states and of every weight */
    int32_t model_dim, hidden_dim;
    int32_t n_q_heads, n_slots, imp_dim;  /* outputs per token = n_slots * n_q_heads * imp_dim */
    int32_t activation;                   /* tb_activation */
    float ln_eps;
    const void* ln_weight;
    const void* ln_bias;
    const void* w1;
    const void* w2;
} tb_predictor;
tb_status tb_predict_importance_queries(const tb_predictor* p, const void* hidden_dev, int32_t n_tokens,
                                        float* scratch_dev, float* q_imp_dev, void* stream);

/* Synchronise `stream`, return the device status word (TB_OK, TB_ERR_TIMEOUT or TB_ERR_BAD_INDEX)
 * in *device_status and clear it. */
tb_status tb_get_status(tb_ctx* ctx, void* stream, int32_t* device_status);

/* Resident sink and window rows for an offloaded cache (paper Sec. 4.4 "CPU-offloaded KV": the full K/V in
 * host memory, only selected rows cross the link).  With the K|V cache in page-locked host memory, every
 * attended row crosses the host link each step -- the sinks and the recent window too, although they are the
 * same rows step after step.  This binds a device region in which the library keeps, per (layer, sequence, KV
 * head), copies of the first `sinks` tokens and of the `window` most recent ones (a ring indexed by position);
 * tb_append_kv writes them beside the cache rows, attention reads sink and window rows from there whenever
 * they are covered (S <= sinks, W <= window) and from the cache otherwise.  Results are the same bits.
 * Bind while every sequence is empty (TB_ERR_STATE otherwise); rows_dev == NULL unbinds.  bytes must be at
 * least tb_resident_rows_bytes(); 256-byte aligned device memory owned by the caller. */
size_t tb_resident_rows_bytes(const tb_config* cfg, int32_t sinks, int32_t window);
tb_status tb_bind_resident_rows(tb_ctx* ctx, void* rows_dev, size_t bytes, int32_t sinks, int32_t window);

/* The paper's contiguous Important buffer (Sec. 3.3: "Sink / Local-Window / Important buffers"; Sec. 3.3 and
 * 3.4: on a prediction step the selected K/V pairs are migrated into it, and the steps in between attend from
 * it).  Once bound, every refreshing tb_select_topk ends with a migration kernel that copies the K|V rows of the
 * stored lists into the buffer, in list order, and tb_sparse_decode_attention reads the list's rows from there
 * (contiguous, no index lookup) when it attends from the stored lists; sinks and window still come from the cache
 * (or the resident rows).  Same bits as gathering from the cache.  With the cache on the device it buys nothing
 * measurable (a 512-byte row is already four full memory sectors) and costs a copy of every selected row per
 * refresh; with an offloaded cache and a prediction interval P it cuts the link traffic P-fold.  Contexts with one
 * list per KV head only (TB_ERR_UNSUPPORTED otherwise).  bytes >= tb_important_buffer_bytes(); buf_dev == NULL
 * unbinds.  Binding drops the stored selections (TB_ERR_STATE from attention until the next selection). */
size_t tb_important_buffer_bytes(const tb_config* cfg);
tb_status tb_bind_important_buffer(tb_ctx* ctx, void* buf_dev, size_t bytes);

/* Where the kernels take the sequence lengths from (Sec. 3.3 / 3.4: the cache grows by a token every decode
 * step and the window moves with it).  The context keeps the lengths twice: host mirrors, advanced when a
 * call is made, which validate arguments; and device counters, advanced by the append and projection kernels
 * themselves while they are in use (switching them on copies the mirrors over, blocking).  By default (on = 0) every launch carries the mirrors' values as kernel parameters: no dependent
 * load at kernel start, but a captured CUDA graph then replays the lengths it was captured with.  With on = 1
 * the kernels read the device counters, so a graph captured once replays a growing sequence: capture a
 * decode step (append, projection with NULL ranges, selection, attention) and replay it every step.
 * growth_reserve = how many tokens a sequence may grow beyond its mirror while graphs are replayed: grids and
 * shared memory are sized for mirror + reserve.  While graphs replay the mirrors stand still; the checks
 * that need true lengths then happen on the device (an append past max_seq_len is skipped and reported as
 * TB_ERR_CAPACITY in the status word).  Call tb_sync_lengths before the next call that is not a replay. */
tb_status tb_use_device_lengths(tb_ctx* ctx, int32_t on, int32_t growth_reserve);
/* Synchronise `stream` and copy the device counters into the host mirrors (lengths and projected lengths). */
tb_status tb_sync_lengths(tb_ctx* ctx, void* stream);

/* Diagnostics of the bounded device waits (every wait of a kernel on a copy it requested polls at most
 * a fixed number of times -- seconds -- then the kernel records TB_ERR_TIMEOUT in the status word, stops
 * requesting copies, finishes normally and leaves nothing in flight; the lists of that call are void).
 * poll_limit > 0 sets the number of polls for this context's selection launches (0 restores the
 * default).  drop_tile >= 0 makes the NEXT selection launch arm the barrier of its drop_tile-th tile of
 * 256 rows without requesting the copy, so that this wait runs out: the way to exercise the path without
 * a fault, a trap or an unbounded wait.  It is honoured only by a launch of one block (one sequence, one
 * list, at most 1023 candidates: nothing else is in flight and no other block waits); any other selection
 * call then returns TB_ERR_UNSUPPORTED and launches nothing.  One-shot; -1 = none. */
tb_status tb_set_wait_diagnostics(tb_ctx* ctx, int32_t poll_limit, int32_t drop_tile);

/* Algorithmic bytes (projected keys scanned + K/V rows gathered, upper bound from host-known sizes)
 * of the most recent select or attention call. */
uint64_t tb_last_step_bytes(const tb_ctx* ctx);

/* Kernels launched by this context since it was created. */
uint64_t tb_launch_count(const tb_ctx* ctx);

const char* tb_status_string(int32_t status);

#ifdef __cplusplus
}
#endif
#endif /* TOKENBUTLER_H_ */
