/*
 * liblaq -- the eviction step of Lookahead Q-Cache (LAQ) on one NVIDIA B200 (sm_100a).
 *
 * Given the full prompt key/value cache of every layer and a small window of post-RoPE
 * "lookahead" queries (the Q-Cache of Section 4.2), the library ranks every cached prompt
 * position and keeps a fixed budget of them per KV head (Section 4.3, Eq. 4):
 *
 *     M_ahead = ArgSort( sum_{q_i in Q} q_i K^T )[:B]
 *
 * Notation (used in every comment of this library):
 *   NL, Bt      layers, batch
 *   Hq, Hkv     query heads, KV heads;  G = Hq / Hkv  query heads share one KV head
 *   D           head dimension (128)
 *   L           prompt length = cached positions before eviction
 *   W           queries per query head in the observation window: lookahead queries, preceded by
 *               W_local causal queries of the last prompt positions for LAQ++ (Eq. 5)
 *   R           retained tail: the last R prompt positions are always kept
 *   k           1-D pooling kernel (odd)
 *   B           budget: positions kept per (layer, batch, KV head), tail included
 *   unit        one (layer, batch, KV head) triple; U = NL*Bt*Hkv units, all independent
 *   M = G*W     softmax rows of a unit;  Ls = L-R scored positions;  Kb = B-R selected slots
 *
 * What one unit computes (Eq. 4 read as attention weights; the paper's Eq. 4 omits the scale,
 * the softmax, the GQA reduction and the pooling, which follow the SnapKV-style "standard KV
 * cache eviction" the paper builds on, Sections 1 and 5.1):
 *   1. logits   s[r][j] = scale * <q_r, k_j>,  r = g*W+i over the G heads x W queries, j in [0,L)
 *               (a local query i < W_local only sees j <= L - W_local + i; the softmax and the
 *               column sums below run over the keys a row sees)
 *   2. softmax  P[r][j] = exp(s[r][j]-m_r) / l_r,  m_r = max_j s[r][j],  l_r = sum_j exp(s[r][j]-m_r)
 *   3. column sums  c[j] = sum_r P[r][j]
 *   4. pooling  p[j] = (1/k) * sum_{|t|<=k/2, 0<=j+t<Ls} c[j+t],  j in [0,Ls)   (zero padded;
 *               or the maximum over the same window, see laq_pool_mode)
 *   5. top-k    the Kb positions of largest p (ties: lower position wins), written ascending,
 *               followed by the tail Ls..L-1
 *   6. gather   K_out[t] = K[idx[t]],  V_out[t] = V[idx[t]]
 *
 * Conventions common to every entry point (the exceptions are named where they apply)
 *   - Data pointers are DEVICE pointers owned by the caller, except in laq_evict_host, whose
 *     tensors live in host memory. The library allocates, retains and frees no device memory;
 *     scratch memory is the caller's workspace `ws` of at least laq_workspace_bytes() bytes,
 *     256-byte aligned. A workspace may be reused by later calls on the same stream; two calls
 *     that overlap on the GPU need two workspaces. The one exception is laq_score_static, whose
 *     scratch is a fixed array inside the library image that all of its calls share.
 *   - Q, K, V, K_out, V_out hold bf16; the innermost (head_dim) stride is 1 and every other
 *     stride, given in ELEMENTS in laq_params, is a multiple of 8 (16 bytes). Base pointers are
 *     16-byte aligned.
 *   - Calls validate on the host, enqueue kernels on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and return without synchronising. A non-OK status
 *     means nothing was enqueued, except LAQ_ERR_CUDA from a failed launch or copy.
 *   - Device-side waits are bounded. If one runs out the kernel records it in the workspace and
 *     finishes; laq_last_device_status() reads that record back (it synchronises the stream).
 *   - No exceptions cross the boundary. Mutable state kept inside the library: cached per-device
 *     attributes; two per-host-thread instrumentation values (the stage events of
 *     laq_set_stage_events and the counter behind laq_last_launch_count); the cached address and
 *     the contents of laq_score_static's scratch array.
 */
#ifndef LAQ_H_
#define LAQ_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define LAQ_API __attribute__((visibility("default")))
#else
#define LAQ_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LAQ_OK = 0,
  LAQ_ERR_INVALID_ARG = 1, /* null pointer, bad size relation, misaligned pointer or stride */
  LAQ_ERR_UNSUPPORTED = 2, /* a valid problem the library has no kernel for (e.g. more than 256 rows) */
  LAQ_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or smaller than laq_workspace_bytes() */
  LAQ_ERR_CUDA = 4,        /* a CUDA runtime or driver call failed */
  LAQ_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out (see laq_last_device_status) */
  LAQ_ERR_INTERNAL = 6
} laq_status;

/* Step 4. LAQ_POOL_AVG: average over the k-wide window, zero padded, divisor always k (the pooling
 * Section 5.1 names). LAQ_POOL_MAX: maximum over the window positions that exist (the other common
 * choice of SnapKV-style eviction; not used by the paper's experiments). */
typedef enum { LAQ_POOL_AVG = 0, LAQ_POOL_MAX = 1 } laq_pool_mode;

/* Steps 2-3. LAQ_SCORE_SOFTMAX: column sums of the per-row softmax (attention weights), the
 * reading used throughout. LAQ_SCORE_RAW: Eq. 4 taken literally, c[j] = sum_r s[r][j], the sum of
 * the raw scaled logits over the window rows with no softmax (one pass over K; scores may be
 * negative; local_window has no effect because it only masks positions inside the tail). */
typedef enum { LAQ_SCORE_SOFTMAX = 0, LAQ_SCORE_RAW = 1 } laq_score_mode;

/* How the G query heads that share a KV head are combined (the paper's Eq. 4 does not say; its
 * models are GQA models). LAQ_GROUP_SUM: the column sums of the group's heads are added, one kept
 * set per KV head (the reading used throughout). LAQ_GROUP_MAX: per key the largest head's column
 * sum counts, one kept set per KV head. LAQ_GROUP_PER_HEAD: every query head ranks and keeps for
 * itself; scores, idx, K_out and V_out then have Hq in place of Hkv in their shapes (query head
 * h*G+g gathers from KV head h; the o_stride_head stride steps over query heads). The last two
 * need LAQ_SCORE_SOFTMAX. */
typedef enum { LAQ_GROUP_SUM = 0, LAQ_GROUP_MAX = 1, LAQ_GROUP_PER_HEAD = 2 } laq_group_mode;

/* Problem description. Plain data; copy freely. All strides are in bf16 ELEMENTS. */
typedef struct {
  int32_t n_layers;    /* NL >= 1 */
  int32_t batch;       /* Bt >= 1 */
  int32_t n_q_heads;   /* Hq, a multiple of n_kv_heads */
  int32_t n_kv_heads;  /* Hkv >= 1; query head h reads KV head h / G */
  int32_t head_dim;    /* D, a multiple of 8 up to 256; 128 takes the tensor-core path */
  int32_t prompt_len;  /* L */
  int32_t window_len;  /* W >= 1 lookahead queries per query head; G*W <= 256 */
  int32_t keep_tail;   /* R, 0 <= R < B: last R positions always kept and never scored */
  int32_t pool_kernel; /* k, odd >= 1; 1 disables pooling */
  int32_t pool_mode;   /* laq_pool_mode */
  int32_t budget;      /* B, R < B < L */
  float softmax_scale; /* 0 selects 1/sqrt(head_dim) */
  /* Scheduling knobs of the scoring kernel; 0 lets the library choose. */
  int32_t tiles_per_task;  /* 128-key tiles per scoring task (a task = one sweep over a key chunk);
                            * it also sets the workspace size, so set it before laq_workspace_bytes */
  int32_t sched_lag_tasks; /* how many tasks the column-sum sweep trails the statistics sweep */
  /* LAQ++ (Eq. 5, unified window W u Q): the first local_window of each head's window_len queries
   * are the queries of the last local_window prompt positions (query i at position
   * L - local_window + i) and attend causally, to positions <= their own; the rest are lookahead
   * queries and see every prompt key. 0 = plain LAQ (Eq. 4). Needs local_window <= window_len and
   * local_window <= keep_tail, so that every scored position is visible to every query. */
  int32_t local_window;
  int32_t score_mode;      /* laq_score_mode */
  int32_t group_mode;      /* laq_group_mode */
  int32_t reserved0;       /* must be 0 */
  /* Q [NL][Bt][Hq][W][D] */
  int64_t q_stride_layer, q_stride_batch, q_stride_head, q_stride_pos;
  /* K [NL][Bt][Hkv][L][D] */
  int64_t k_stride_layer, k_stride_batch, k_stride_head, k_stride_pos;
  /* V [NL][Bt][Hkv][L][D] */
  int64_t v_stride_layer, v_stride_batch, v_stride_head, v_stride_pos;
  /* K_out and V_out [NL][Bt][Hkv][B][D] (the same strides serve both) */
  int64_t o_stride_layer, o_stride_batch, o_stride_head, o_stride_pos;
  /* Prompts of different lengths in one batch (the paper evaluates one prompt at a time; a
   * serving batch is ragged). NULL: every prompt holds prompt_len positions. Otherwise a HOST
   * array of `batch` int32, read during the call only: prompt b holds its first seq_lens[b]
   * positions of the L allocated ones, budget < seq_lens[b] <= prompt_len, and batch <=
   * LAQ_MAX_RAGGED_BATCH. Everything is then relative to that length Lb: keys [0, Lb), local
   * queries at the last local_window of them, scored positions [0, Lb-R), tail [Lb-R, Lb). Rows of
   * K and V beyond Lb are never used (they may hold anything); scores beyond Lb-R are written
   * as 0. The tensors keep their [.. L ..] shapes and strides. */
  const int32_t* seq_lens;
} laq_params;

#define LAQ_MAX_RAGGED_BATCH 512
#define LAQ_MAX_LAYER_BUDGETS 256

/* Fills the stride fields of `p` for densely packed tensors in the index order shown above. */
LAQ_API void laq_params_dense_strides(laq_params* p);

/* Bytes of caller-provided device scratch that laq_score / laq_evict need for `p`
 * (0 if `p` is invalid). laq_select, laq_compact and laq_recall need none and take no workspace
 * argument. */
LAQ_API size_t laq_workspace_bytes(const laq_params* p);

/*
 * Steps 1-4 (Eq. 4's sum over the window, Section 4.3): pooled importance of every scored
 * position.
 *   q       device, bf16, lookahead queries, layout/strides from `p`
 *   k       device, bf16, prompt keys
 *   scores  device, fp32, dense [NL][Bt][Hkv][L-R]; written in full
 *   ws      device scratch, ws_bytes >= laq_workspace_bytes(p)
 * Errors: LAQ_ERR_INVALID_ARG, LAQ_ERR_UNSUPPORTED, LAQ_ERR_WORKSPACE, LAQ_ERR_CUDA.
 */
LAQ_API laq_status laq_score(const laq_params* p, const void* q, const void* k, float* scores,
                     void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * laq_score for callers that cannot allocate device memory. The paper has no counterpart to this
 * entry point; it is an integration aid. It computes exactly what laq_score computes, but takes
 * no workspace: its scratch is a fixed array of LAQ_STATIC_SCRATCH_BYTES bytes inside the library
 * image (one copy on every GPU that loads the library, held until the process exits). It is meant
 * for hosts that give all device memory to their own pool at start-up and may not call the
 * driver's allocator afterwards -- an inference server whose allocator owns the GPU, a plugin
 * that receives tensors and a stream but no allocator, a latency-critical loop that cannot take
 * the device-wide synchronisation of an allocation. After one warm-up call per device the call
 * allocates nothing: no cudaMalloc, no cudaFree, no allocating library routine. The warm-up call
 * is different, because CUDA loads a library's kernels and device arrays lazily: the first call on
 * a device is what makes the driver place the scratch array and the kernel code in that device's
 * memory, so make it at start-up, before the host's own pool claims the GPU (on a GPU with no
 * room left it fails with LAQ_ERR_CUDA), and outside any stream capture.
 *   q, k, scores   as for laq_score (device pointers; scores dense [NL][Bt][Hkv][L-R], fp32)
 * Limits and rules
 *   - The problem's scratch (per-unit counters, per-task row statistics and one fp32 column sum
 *     per key: roughly 4 bytes per cached key plus 8*M bytes per scoring task) must fit in
 *     LAQ_STATIC_SCRATCH_BYTES; otherwise LAQ_ERR_WORKSPACE is returned and nothing is enqueued.
 *     Larger problems can be scored in slices of layers with one call per slice.
 *   - The first call on a device also looks up the array's device address (with that device
 *     current) and caches it for later calls.
 *   - Every call uses the same array, which still holds the previous call's contents; the call
 *     clears the parts that must start at zero. Two calls that overlap on the GPU (different
 *     streams, or different host threads without ordering) race on it: order them.
 *   - laq_last_device_status does not apply; a bounded device-side wait that runs out leaves the
 *     scores undefined, as it does for laq_score.
 * Errors: LAQ_ERR_INVALID_ARG, LAQ_ERR_UNSUPPORTED, LAQ_ERR_WORKSPACE (problem too large for the
 * static scratch), LAQ_ERR_CUDA.
 */
#define LAQ_STATIC_SCRATCH_BYTES (8u * 1024u * 1024u)
LAQ_API laq_status laq_score_static(const laq_params* p, const void* q, const void* k,
                                    float* scores, void* cuda_stream);

/*
 * Step 5 (Eq. 4's ArgSort(...)[:B]): per unit, the B-R positions of largest score, ties to the
 * lower position, then the retained tail.
 *   scores  device, fp32, dense [NL][Bt][Hkv][L-R], no NaN (negative values are allowed)
 *   idx     device, int32, dense [NL][Bt][Hkv][B]; first B-R entries strictly ascending in
 *           [0, L-R), last R entries are L-R .. L-1 (with seq_lens: Lb in place of L)
 * Only n_layers, batch, n_kv_heads, prompt_len, keep_tail, budget and seq_lens of `p` are read.
 */
LAQ_API laq_status laq_select(const laq_params* p, const float* scores, int32_t* idx, void* cuda_stream);

/*
 * Step 6 ("cache re-eviction based on the given budget", Section 4.3): gathers the kept rows.
 *   k, v          device, bf16, prompt keys and values
 *   idx           device, int32, dense [NL][Bt][Hkv][B], every entry in [0, L)
 *   k_out, v_out  device, bf16, [NL][Bt][Hkv][B][D] with the o_stride_* strides; either may be
 *                 NULL to skip that tensor. Must not overlap k / v.
 */
LAQ_API laq_status laq_compact(const laq_params* p, const void* k, const void* v, const int32_t* idx,
                       void* k_out, void* v_out, void* cuda_stream);

/*
 * Steps 1-6 in one call (the whole re-eviction of Section 4.3 for all layers and heads).
 *   idx     optional (NULL allowed) device int32 [NL][Bt][Hkv][B]: receives the kept positions
 *   scores  optional (NULL allowed) device fp32 [NL][Bt][Hkv][L-R]: receives the pooled scores
 * Other arguments as in laq_score / laq_compact.
 */
LAQ_API laq_status laq_evict(const laq_params* p, const void* q, const void* k, const void* v,
                     void* k_out, void* v_out, int32_t* idx, float* scores, void* ws,
                     size_t ws_bytes, void* cuda_stream);

/*
 * laq_evict with one budget per layer. The paper evicts to a fixed budget (Section 5.2) and names
 * layer-wise budgets of the PyramidKV kind as a combination it is compatible with (Section 5.1);
 * the units of different layers are independent, so only steps 5 and 6 change.
 *   layer_budgets  HOST, int32 [NL], read during the call only: layer n keeps layer_budgets[n]
 *                  positions per (batch, KV head), R < layer_budgets[n] < L (and below every
 *                  seq_lens entry). p->budget must equal the largest of them (it sizes the
 *                  workspace). NL <= LAQ_MAX_LAYER_BUDGETS.
 *   idx            optional, device int32: ONE ragged pool, layer after layer; layer n holds
 *                  [Bt][Hkv][layer_budgets[n]] entries and starts at entry
 *                  Bt*Hkv*(layer_budgets[0] + ... + layer_budgets[n-1])
 *   k_out, v_out   device bf16, the same ragged pool with D elements per entry (densely packed:
 *                  the o_stride_* fields are not used); either may be NULL
 *   scores         optional, device fp32, dense [NL][Bt][Hkv][L-R] as for laq_evict
 * laq_layers_pool_entries() returns the number of entries of the pool (0 for invalid arguments).
 * Errors: as laq_evict, LAQ_ERR_UNSUPPORTED for more than LAQ_MAX_LAYER_BUDGETS layers.
 */
LAQ_API size_t laq_layers_pool_entries(const laq_params* p, const int32_t* layer_budgets);
LAQ_API laq_status laq_evict_layers(const laq_params* p, const int32_t* layer_budgets, const void* q,
                                    const void* k, const void* v, void* k_out, void* v_out,
                                    int32_t* idx, float* scores, void* ws, size_t ws_bytes,
                                    void* cuda_stream);

/*
 * The keep-set of a StreamingLLM-style cache: the first n_sink positions ("attention sinks") and
 * the most recent budget - n_sink positions of every prompt. Section 4.2 starts the lookahead from
 * a low-budget cache of this kind (or of the SnapKV kind, which is laq_evict with
 * local_window = window_len); feeding these indices to laq_compact builds it.
 *   idx   device, int32, dense [NL][Bt][Hkv][B], ascending: 0 .. n_sink-1, then Lb-(B-n_sink) .. Lb-1
 *         (Lb = seq_lens[b] if given, else L)
 * Only n_layers, batch, n_kv_heads, prompt_len, budget and seq_lens of `p` are read.
 * Errors: LAQ_ERR_INVALID_ARG (n_sink outside [0, B], B >= Lb), LAQ_ERR_CUDA.
 */
LAQ_API laq_status laq_streaming_indices(const laq_params* p, int32_t n_sink, int32_t* idx,
                                         void* cuda_stream);

/*
 * Recall of one selection against another (Section 3, Eq. 1-3):
 *     Recall = |M_pred n M_gold| / |M_gold|
 * per unit, e.g. M_pred from the lookahead window and M_gold from the queries of the real
 * response, both obtained with laq_score + laq_select.
 *   idx_pred  device, int32, dense [n_units][n_pred], each row ascending (as laq_select writes it)
 *   idx_gold  device, int32, dense [n_units][n_gold], each row ascending and without repeats
 *   n_common  device, int32 [n_units], size of the intersection (may be NULL)
 *   recall    device, fp32 [n_units] (may be NULL; at least one output is required)
 * Errors: LAQ_ERR_INVALID_ARG, LAQ_ERR_UNSUPPORTED (more than 2^34 units), LAQ_ERR_CUDA.
 */
LAQ_API laq_status laq_recall(int64_t n_units, const int32_t* idx_pred, int32_t n_pred,
                              const int32_t* idx_gold, int32_t n_gold, int32_t* n_common,
                              float* recall, void* cuda_stream);

/*
 * The whole step for a cache that lives in HOST memory (ideally pinned): copies Q, K and V to the
 * caller's device staging area, runs laq_evict there and copies the compressed cache back, all
 * ordered on `cuda_stream`. Host tensors are densely packed in the index order of laq_params (the
 * stride fields of `p` are ignored and dense strides are used on both sides).
 *   q_host, k_host, v_host          HOST, bf16, inputs
 *   k_out_host, v_out_host          HOST, bf16 [NL][Bt][Hkv][B][D], outputs
 *   idx_host                        HOST, int32 [NL][Bt][Hkv][B], output (may be NULL)
 *   staging, staging_bytes          DEVICE scratch of at least laq_host_staging_bytes(p) bytes,
 *                                   256-byte aligned
 *   ws, ws_bytes                    DEVICE workspace as for laq_evict
 * Returns after enqueueing; the host outputs are valid once the stream has been synchronised.
 * Only the kept rows of V are needed (step 6): when v_host is pinned (page-locked) memory that
 * the GPU can address, the gather reads those rows directly from it and V is not copied to the
 * device at all, which halves the host-to-device traffic; pageable v_host is staged like Q and K.
 * Pinned k_out_host / v_out_host are likewise written by the gather directly instead of being
 * staged and copied back.
 */
LAQ_API size_t laq_host_staging_bytes(const laq_params* p);
LAQ_API laq_status laq_evict_host(const laq_params* p, const void* q_host, const void* k_host,
                                  const void* v_host, void* k_out_host, void* v_out_host,
                                  int32_t* idx_host, void* staging, size_t staging_bytes, void* ws,
                                  size_t ws_bytes, void* cuda_stream);

/*
 * Synchronises `cuda_stream` and reports what the last laq_score / laq_evict call that used
 * `ws` recorded on the device: LAQ_OK, LAQ_ERR_TIMEOUT (a bounded wait ran out; outputs are
 * not valid) or LAQ_ERR_CUDA (the synchronise or the read-back failed).
 */
LAQ_API laq_status laq_last_device_status(const laq_params* p, const void* ws, size_t ws_bytes,
                                  void* cuda_stream);

/*
 * Instrumentation for benchmarks: caller-owned CUDA events (cudaEvent_t passed as void*) that
 * later laq_score / laq_evict calls made by this host thread record on their stream immediately
 * before and after the scoring kernel (steps 1-3). Pass NULL, NULL to stop recording. The events
 * must outlive the calls that record them.
 */
LAQ_API void laq_set_stage_events(void* score_begin, void* score_end);

/*
 * Instrumentation for benchmarks (no counterpart in the paper): synchronises `cuda_stream` and
 * reads what the tensor-core scoring kernel of the last laq_score / laq_evict call on `ws`
 * recorded about itself: the SM clock cycles and the wall-clock nanoseconds its first thread block
 * ran for (the block is resident for the whole launch). cycles / nanoseconds is the SM clock the
 * kernel really ran at; the board lowers it under load, so cycle counts and times are reported
 * separately. Both read 0 if the call took another scoring path (head_dim other than 128, raw mode).
 *   ws, ws_bytes   the workspace of that call (device)
 *   sm_cycles, nanoseconds   HOST, out
 * Errors: LAQ_ERR_INVALID_ARG, LAQ_ERR_CUDA.
 */
LAQ_API laq_status laq_last_kernel_clock(const void* ws, size_t ws_bytes, void* cuda_stream,
                                         int64_t* sm_cycles, int64_t* nanoseconds);

/* Kernel launches the most recent call on this host thread enqueued (for accounting). */
LAQ_API int laq_last_launch_count(void);

LAQ_API const char* laq_status_string(laq_status s);
LAQ_API int laq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LAQ_H_ */
