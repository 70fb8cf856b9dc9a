/*
 * qc.h -- C ABI of the Lazy Attention / Q Cache decode library (sm_100a).
 *
 * The library implements the decode-step attention of an MLLM decoder stack whose layers
 * are either ordinary ("full") or lazy, as defined in the paper's section "Method":
 *   - Eq. 2   decode attention of an ordinary layer over its KV cache plus the new token;
 *   - section "Lazy Attention": a lazy block is one ordinary layer l_c followed by lazy
 *     layers; the Q Cache holds the query of l_c;
 *   - Eq. 6   GLA decode: Q = Q Cache, K = K cache of l_c, V = the lazy layer's own;
 *   - Eq. 8   VLA decode: K = [own text K, visual K of l_c, own new k], V = own;
 *   - section "Efficiency Analysis": what each layer stores (all V; ordinary layers all K;
 *     VLA lazy layers text K only; GLA lazy layers no K) and the closed-form saving.
 *
 * Conventions common to every call
 *   - Every function returns an int32 status (QC_OK == 0).  Nothing throws, aborts or prints.
 *     On an error status the cache is unchanged and no output is written, with two exceptions:
 *     QC_ERR_CUDA (a CUDA call failed part-way: free the cache) and the device error word.  A
 *     kernel that gives up (a bounded wait that ran out, a page id or work range outside its
 *     limits) ends normally, leaves its part of the output unwritten and records a code in the
 *     device error word, mirrored into mapped host memory: qc_get_stats reports it, and every later
 *     qc_decode_step / qc_decode_step_host on that cache returns it instead of running.
 *   - "dev" pointers are CUDA device pointers on the context's device; "host" pointers are
 *     ordinary host memory.  All device memory is owned by the caller: the pool and the
 *     workspace are handed in at qc_alloc_cache and must outlive the cache.  The library
 *     allocates no device memory.  It owns the qc_ctx / qc_cache host objects and a few KiB of
 *     pinned host memory per cache.
 *   - Kernels are launched asynchronously on the stream given to qc_init.  Device pointers
 *     passed to a call must stay valid until that stream has executed the call.  Host arrays
 *     (seq_ids, n_tokens, kind) are consumed before the call returns.
 *   - bf16 tensors are dense, row-major in the index order written in brackets.
 *   - A sequence id is an integer in [0, max_seqs).  The token axis of a sequence is kept as
 *     two ordered streams, text and visual (the paper's "concatenation" simplification after
 *     Eq. 8); generated tokens are text.
 */
#ifndef QC_H_
#define QC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qc_ctx qc_ctx;     /* device, stream, SM count */
typedef struct qc_cache qc_cache; /* page tables, stream lengths, free list, Q Cache, plans */

enum {
  QC_OK = 0,
  QC_ERR_INVALID_ARG = 1, /* null pointer, out-of-range id or size, misaligned pointer */
  QC_ERR_UNSUPPORTED = 2, /* shape the kernels do not cover */
  QC_ERR_OOM_PAGES = 3,   /* the pool has too few free pages for this call */
  QC_ERR_STATE = 4,       /* lazy layer 0, decode on an unknown sequence, duplicate id, ... */
  QC_ERR_CUDA = 5,        /* a CUDA runtime call failed */
  QC_ERR_TIMEOUT = 6,     /* a bounded wait inside a kernel ran out (device error word) */
  QC_ERR_BAD_PAGE = 7,    /* a kernel met a page id outside the pool and did not follow it (device error word) */
  QC_ERR_PLAN = 8         /* a kernel met a work range outside the limits it was planned for (device error word) */
};

enum { QC_LAYER_FULL = 0, QC_LAYER_LAZY = 1 };

/* Which query scores which keys in a lazy layer (one mode per cache; the paper's overview
 * states that a model is optimised for a single mode).
 *   QC_MODE_VLA_QC  : text keys = own text K scored by the own q; visual keys = leader's
 *                     visual K scored by the Q Cache (the leader's q of the same token).
 *   QC_MODE_VLA_EQ8 : Eq. 8 as printed: the own q scores own text K and leader's visual K.
 *   QC_MODE_GLA     : Eq. 6: the Q Cache scores all of the leader's K.
 * V is always the lazy layer's own. */
enum { QC_MODE_VLA_QC = 0, QC_MODE_VLA_EQ8 = 1, QC_MODE_GLA = 2 };

/* Streams of one (layer, sequence), in allocation order. */
enum { QC_STREAM_K_TEXT = 0, QC_STREAM_K_VISUAL = 1, QC_STREAM_V_TEXT = 2, QC_STREAM_V_VISUAL = 3 };

enum { QC_KIND_TEXT = 0, QC_KIND_VISUAL = 1 };

typedef struct qc_config {
  int32_t n_layers;            /* 1..127 */
  int32_t n_q_heads;           /* multiple of n_kv_heads; query head h reads KV head h / group */
  int32_t n_kv_heads;
  int32_t head_dim;            /* 64 or 128 */
  int32_t page_size;           /* 16 = paged; 0 = contiguous: every stream owns a fixed extent of
                                  the pool (no allocator, no OOM), index
                                  ((layer*4 + stream)*max_seqs + seq) */
  int32_t max_seqs;            /* 1..4096 */
  int32_t max_tokens_per_seq;  /* bound on text tokens and on visual tokens of one sequence */
  int64_t n_pages;             /* pool capacity in pages (paged mode); ignored when contiguous */
  float softmax_scale;         /* 0 => 1/sqrt(head_dim) (Eq. 2) */
  int32_t lazy_mode;           /* QC_MODE_* */
  int32_t split_tokens;        /* keys per split-KV work item, a multiple of 16 in 16..512.  Every
                                  stream is cut into ceil(len/split_tokens) chunks whose partial
                                  results are merged by log-sum-exp.  0 => chosen per step among
                                  64, 128, 256 and 512 from the amount of work (workspace sized for 64). */
  const uint8_t* layer_kind;   /* host, [n_layers], QC_LAYER_*; layer 0 must be FULL; copied */
} qc_config;

typedef struct qc_stats {
  int64_t pages_total;            /* pool capacity in pages */
  int64_t pages_in_use;
  int64_t page_bytes;             /* bytes of one page: n_kv_heads * 16 * head_dim * 2 */
  int64_t kv_bytes_stored;        /* token-exact bytes of K and V rows held */
  int64_t kv_bytes_all_full;      /* token-exact bytes if every layer were ordinary */
  int64_t kv_bytes_stored_paged;  /* pages_in_use * page_bytes */
  int64_t kv_bytes_all_full_paged;/* page-rounded bytes if every layer were ordinary */
  int64_t qcache_bytes;           /* bytes of the Q Cache buffer */
  int64_t decode_steps;           /* qc_decode_step calls completed (enqueued) */
  int64_t attend_launches;        /* launches of the attention kernel so far */
  int32_t device_error;           /* 0, or the QC_ERR_* code the device error word holds */
  int32_t n_active_seqs;
  int64_t kernel_launches;        /* kernels of this library launched for the cache so far */
  int64_t kv_bytes_swept;         /* algorithmic K/V bytes of the decode steps so far: every stored row of the
                                     listed sequences once per step */
} qc_stats;

/* Per-step kernel timing (CUDA events on the library's stream), for roofline accounting. */
typedef struct qc_profile {
  int64_t steps;              /* decode steps covered */
  double attend_ms;           /* summed duration of the attention (split-KV partial) kernel; when a
                                 step runs as several launches, from the start of its first
                                 attention launch to the end of its last (merges between them
                                 included) */
  double step_ms;             /* summed duration of whole steps (setup+append+attend+merge) */
  int64_t kv_bytes_read;      /* algorithmic K/V bytes those steps had to read: every stored
                                 row of the listed sequences once, per step */
  int64_t items;              /* split-KV work items executed */
  int64_t prefill_calls;      /* qc_prefill_attend calls covered */
  double prefill_attend_ms;   /* summed duration of the prefill attention kernel */
  double prefill_flops;       /* its executed arithmetic: per (query, visible key) pair and query head,
                                 2 * head_dim flops for every score pass (one per layer, or one per
                                 run of layers that share their scores) and 2 * head_dim for every
                                 layer's value product */
  double attend_kernel_ms;    /* option "profile" = 2: summed durations of the attention launches alone,
                                 each between events of its own (events between launches end the
                                 overlap of a launch's start with its predecessor's end: this mode is
                                 for the kernel's time, not for the step's) */
  int64_t attend_kernel_launches;
} qc_profile;

/* Create a context on `device` that launches on `cuda_stream` (a cudaStream_t; NULL is the
 * legacy default stream).  Host object only. */
int32_t qc_init(int32_t device, void* cuda_stream, qc_ctx** out);

/* Bytes the caller must provide for a cache of this configuration.  pool_bytes covers the
 * K/V pages, workspace_bytes the page tables, Q Cache, split-KV partials, logit cache, plans and
 * staging. */
int32_t qc_cache_bytes_required(const qc_config* cfg, size_t* pool_bytes, size_t* workspace_bytes);

/* Build a cache over caller-owned device memory (both 256-byte aligned).  Page layout: one
 * page holds 16 tokens of ONE tensor (K or V) for all KV heads, [n_kv_heads][16][head_dim] bf16.
 * A lazy layer gets no visual-K pages (and in GLA no K pages at all): its reads go to the
 * leader's pages.  The pool contents are not initialised. */
int32_t qc_alloc_cache(qc_ctx* ctx, const qc_config* cfg, void* pool_dev, size_t pool_bytes,
                       void* workspace_dev, size_t workspace_bytes, qc_cache** out);

/* Append prompt tokens (Eq. 1: K and V of the prompt go to the KV cache).  Sequence seq_ids[i]
 * receives n_tokens[i] tokens; `kind` (host, QC_KIND_*, concatenated per sequence in call
 * order) routes each token to the text or the visual stream.  k_dev, v_dev:
 * bf16 [n_layers][sum n_tokens][n_kv_heads][head_dim].  K rows that the mode does not store
 * are ignored.  New sequences become active.  No attention is computed.  The call returns
 * after the copies have been enqueued and the host arrays consumed. */
int32_t qc_prefill_append(qc_cache* cache, int32_t n_seqs, const int32_t* seq_ids,
                          const int32_t* n_tokens, const uint8_t* kind, const void* k_dev,
                          const void* v_dev);

/* Prefill attention of one sequence's whole prompt, all layers, followed by what
 * qc_prefill_append does with the same k/v (section "Q Cache", prefilling forms):
 *   ordinary layer  Eq. 1: causal softmax((Q K^T + M)/sqrt(D)) V over the prompt;
 *   GLA lazy layer  Eq. 5: Q = Q Cache (the queries of the block's first layer for every prompt
 *                   token), K = that layer's K, V own;
 *   VLA lazy layer  Eq. 7 (both VLA modes): query rows and key rows of VISUAL tokens come from
 *                   the block's first layer, those of text tokens are the layer's own; V own.
 * Token t of the prompt sees tokens 0..t in the order given (kind[t] tags it text or visual).
 *   q_dev   bf16 [n_layers][n_tokens][n_q_heads][head_dim]   (the Q Cache of a block is its first
 *           layer's slice of this tensor; nothing prompt-sized is kept afterwards)
 *   k_dev, v_dev bf16 [n_layers][n_tokens][n_kv_heads][head_dim]
 *   out_dev bf16 [n_layers][n_tokens][n_q_heads][head_dim]
 * If the sequence already holds tokens (an earlier prompt chunk, generated tokens: a later turn of
 * a conversation), they precede the new ones: every new token also sees all of them, read from
 * the cache with the cache's own sharing (a lazy layer's visual keys -- in GLA all its keys -- are
 * its leader's), which is what Eq. 5 / Eq. 7 select for those tokens.
 * Errors of qc_prefill_append apply; on an error nothing is stored or written. */
int32_t qc_prefill_attend(qc_cache* cache, int32_t seq_id, int32_t n_tokens, const uint8_t* kind,
                          const void* q_dev, const void* k_dev, const void* v_dev, void* out_dev);

/* Calibration by-product (section "Lazy Attention", Eq. 3).  For a cache whose layers are ALL
 * ordinary (the analysis runs on the unmodified stack; otherwise QC_ERR_STATE) and one query
 * token per listed sequence -- normally the prompt's last token, whose K/V are already cached --
 * computes per layer the attention distribution of that query over every cached token, averaged
 * over the query heads, and the Jensen-Shannon divergence (natural log, 0..ln 2) between the
 * distributions of adjacent layers, averaged over the listed sequences:
 *   similarity_host[l] = mean_i JS(a_i^l, a_i^{l+1}),  l = 0 .. n_layers - 2   (host, written on return)
 *   q_dev     bf16 [n_layers][n_seqs][n_q_heads][head_dim]
 *   rows_dev  fp32 [n_layers][n_seqs][max_len], caller-owned scratch and by-product: the
 *             distributions, text tokens first then visual tokens, zero past a sequence's length
 * max_len >= every listed sequence's token count and <= 12288 (else QC_ERR_UNSUPPORTED).  The
 * cache is not changed.  Synchronises the stream. */
int32_t qc_layer_similarity(qc_cache* cache, int32_t n_seqs, const int32_t* seq_ids, const void* q_dev,
                            float* rows_dev, int32_t max_len, float* similarity_host);

/* Eq. 4 (host only): layer l+1 joins the lazy block of layer l when similarity[l] < eps
 * (0 < eps <= 1) and, if max_block > 0, the block has fewer than max_block layers.  Writes
 * layer_kind[n_layers] for qc_config: the first layer of every block stays ordinary. */
int32_t qc_lazy_blocks(const float* similarity, int32_t n_layers, float eps, int32_t max_block,
                       uint8_t* layer_kind);

/* One generated (text) token for each listed sequence through all layers (Eq. 2, 6, 8):
 * appends k/v, refreshes the Q Cache from every ordinary layer's q, computes split-KV partial
 * attention and merges the partials by log-sum-exp.
 *   q_dev   bf16 [n_layers][n_seqs][n_q_heads][head_dim]
 *   k_dev   bf16 [n_layers][n_seqs][n_kv_heads][head_dim]  (rows of GLA lazy layers ignored)
 *   v_dev   bf16 [n_layers][n_seqs][n_kv_heads][head_dim]
 *   out_dev bf16 [n_layers][n_seqs][n_q_heads][head_dim]
 *   lse_out_dev  optional fp32 [n_layers][n_seqs][n_q_heads], natural-log sum of exp; may be NULL
 * seq_ids (host) must be distinct active sequences.  The call is asynchronous. */
int32_t qc_decode_step(qc_cache* cache, int32_t n_seqs, const int32_t* seq_ids, const void* q_dev,
                       const void* k_dev, const void* v_dev, void* out_dev, float* lse_out_dev);

/* The same step issued layer by layer, for a caller whose layer l+1 inputs only exist after layer l's
 * output (a model that computes layer after layer).  qc_decode_begin does the step's page planning
 * for the listed sequences (distinct, active) and plans every layer's launch; then exactly n_layers
 * calls of qc_decode_layer follow, for layer 0, 1, ... in order, each with that layer's slices
 *   q_dev bf16 [n_seqs][n_q_heads][head_dim], k_dev / v_dev bf16 [n_seqs][n_kv_heads][head_dim],
 *   out_dev bf16 [n_seqs][n_q_heads][head_dim], lse_out_dev optional fp32 [n_seqs][n_q_heads].
 * A call appends the layer's k/v (and refreshes the Q Cache from an ordinary layer's q) and runs the
 * layer's attention launch and its merge, asynchronously (the append is part of the attention
 * launch: no launch of its own); out_dev is complete when the stream
 * has executed the call.  The launches are those of the in-order schedule ("in_order_launches"):
 * a leader's call also weights its followers' cached V rows, so a follower's call is short (VLA_QC:
 * its text sweep; GLA: the merge with the new token as one more key; k_dev of a GLA follower is
 * ignored).  Results equal qc_decode_step's.  While a step is open (begun, layers left), every call
 * that would change the cache returns QC_ERR_STATE; a step cannot be abandoned: the sequences'
 * lengths and pages were committed by qc_decode_begin.  Errors: as qc_decode_step; a layer out of
 * order or without an open step is QC_ERR_STATE. */
int32_t qc_decode_begin(qc_cache* cache, int32_t n_seqs, const int32_t* seq_ids);
int32_t qc_decode_layer(qc_cache* cache, int32_t layer, const void* q_dev, const void* k_dev, const void* v_dev,
                        void* out_dev, float* lse_out_dev);

/* Same step with HOST buffers of the same layouts.  The step runs as up to four launch groups of
 * consecutive lazy blocks; on two internal copy streams the inputs of a group are copied to
 * staging in the workspace while the previous group computes, and its outputs are copied back
 * while the next one computes.  Returns when everything has been copied back.  Pinned host
 * buffers make the copies asynchronous; pageable ones also work (without the overlap). */
int32_t qc_decode_step_host(qc_cache* cache, int32_t n_seqs, const int32_t* seq_ids,
                            const void* q_host, const void* k_host, const void* v_host,
                            void* out_host, float* lse_out_host);

/* Release a sequence: its pages return to the free list in reverse order of allocation. */
int32_t qc_free_seq(qc_cache* cache, int32_t seq_id);

/* Destroy a cache and/or a context (either may be NULL).  Waits for the stream first.
 * Caller-owned device memory is not touched. */
int32_t qc_free(qc_ctx* ctx, qc_cache* cache);

/* Accounting for the "KV bytes saved" metric (section "Efficiency Analysis").  Also reads the
 * device error word (this synchronises the stream). */
int32_t qc_get_stats(qc_cache* cache, qc_stats* out);

/* Page table of one stream, from the host mirror.  Writes up to `cap` page ids, the page
 * count, the stream length in tokens and the layer that owns the pages: `layer` itself, the
 * leader if the stream is an alias, -1 (and zero pages) if the sequence is not active. */
int32_t qc_debug_page_table(const qc_cache* cache, int32_t layer, int32_t stream, int32_t seq_id,
                            int32_t* page_ids, int32_t cap, int32_t* n_pages, int32_t* n_tokens,
                            int32_t* owner_layer);

/* Copy the Q Cache entry a lazy layer reads (its leader's latest queries) to the host:
 * bf16 [max_seqs][n_q_heads][head_dim].  Synchronises the stream. */
int32_t qc_debug_read_qcache(qc_cache* cache, int32_t layer, void* host_bf16);

/* Copy one stored row (bf16 [head_dim]) of a stream to the host; aliases resolve to the
 * leader's pages.  Synchronises the stream.  For tests of the append path. */
int32_t qc_debug_read_row(qc_cache* cache, int32_t layer, int32_t stream, int32_t seq_id,
                          int32_t token, int32_t kv_head, void* host_bf16);

/* Tuning knobs (all optional).  key: "split_tokens" (as in qc_config, never below the value
 * the cache was created with; 0 = per-step choice), "layers_per_launch"
 * (0 = one attention launch for the whole step; k>0 = one launch per k consecutive lazy
 * blocks, in layer order), "per_layer_logit_cache" (1 = one attention + merge launch per layer,
 * in layer order: the schedule of a model in which a layer's q/k/v only exist after the previous
 * layer has run.  A leader with followers then also stores its scaled scores -- of the visual keys
 * in VLA_QC, of all keys in GLA -- in a logit cache inside the workspace, 4 bytes per key and
 * query head, and a follower weights its own V rows with them instead of reading the leader's K
 * again; by Eq. 6 / the Q Cache rule the follower's scores are the leader's, so the result is the
 * one of the fused schedule.  VLA_EQ8 followers score with their own query and re-read the
 * leader's visual K.  0 = back to one launch per step.  qc_decode_step only),
 * "prefill_tcgen05" (0 = use the mma.sync prefill kernel), "prefill_shared_scores" (GLA only: by
 * Eq. 5 the layers of a lazy block attend with the same Q and K, so qc_prefill_attend computes and
 * normalises their scores once per run of up to three layers and applies them to each layer's V,
 * bit-identically to one pass per layer; 0 = never, 1 = for prompts of 1536 tokens or more (the
 * default: below that the pass's lower occupancy costs more than it saves), 2 = always),
 * "prefill_pair_min_tokens" (n > 0: prompts of n tokens or more that start a sequence run on the
 * prefill kernel with two query tiles per CTA and 128-key tiles; 0, the default: never),
 * "profile" (1 = record CUDA events per step; 2 = also around every attention launch), "in_order_launches"
 * (1 = one launch per layer in layer order, each using nothing of later layers; what a follower
 * shares with its leader are scores over rows cached before the step, so a leader's launch also
 * weights its followers' cached V rows and leaves their partial rows behind; a VLA_QC follower's
 * launch is its text sweep, a GLA follower's is the merge with the step's new token as one more
 * key, Eq. 6; VLA_EQ8 followers sweep the leader's visual K with their own query), "static_partition"
 * (-1 = a step of several launches cuts each launch's work into equal ranges of K/V tiles, one or a
 * few per worker, instead of handing out chunk items; 0 = never; 1 = always), "static_min_tiles",
 * "static_row_cost" (tuning of those ranges: shortest range, and what one more output row counts
 * for, in 4 KiB tiles), "plan_ahead" (0 = workers locate their ranges themselves instead of reading
 * starting points that one kernel per step works out for every launch), "fused_merge" (1 = the
 * worker that delivers an output row's last partial merges it, instead of a merge launch),
 * "fold_append" (in-order schedule and qc_decode_layer; 1, the default = a layer's new k/v rows and an
 * ordinary layer's q are taken from the inputs and stored by that layer's own launch; 0 = by an
 * append when the step begins, resp. an append launch per layer call),
 * "debug_drop_tile" (test hook for the error path: 1 = every worker of an attention launch leaves
 * out the copy of its first tile and waits for it with a short limit; nothing is in flight for that
 * wait, so it runs out, the worker records QC_ERR_TIMEOUT and returns, and the kernel ends normally
 * with its rows unwritten). */
int32_t qc_set_option(qc_cache* cache, const char* key, int64_t value);

/* Sum the recorded kernel times since the last call (synchronises), then reset them. */
int32_t qc_get_profile(qc_cache* cache, qc_profile* out);

/* ---- A call for callers that cannot allocate ------------------------------------------------
 *
 * The paper has no counterpart to this call; it exists for deployment reasons.  Everything
 * above works on memory the caller allocates and hands over.  Some callers cannot do even
 * that at the moment they need attention computed: a serving process whose device memory
 * was partitioned at start-up and whose allocator is frozen afterwards, or code running
 * inside another framework's callback where device allocation is forbidden.  For them
 * qc_attend_static computes plain decode attention (Eq. 2) using only the tensors passed in
 * plus a fixed scratch array that is part of the library image.
 *
 *   q_dev   bf16 [n_seqs][n_q_heads][head_dim]              one query token per sequence
 *   k_dev   bf16 [n_seqs][n_tokens][n_kv_heads][head_dim]   keys, the new token's included
 *   v_dev   bf16 [n_seqs][n_tokens][n_kv_heads][head_dim]
 *   out_dev bf16 [n_seqs][n_q_heads][head_dim]
 *   softmax_scale 0 => 1/sqrt(head_dim)
 *
 * The key axis is cut into QC_STATIC_SPLITS ranges whose partial softmax results are kept in
 * the scratch array and merged by log-sum-exp.  The array holds QC_STATIC_MAX_ROWS *
 * QC_STATIC_SPLITS * 130 floats (about 2 MiB) on every GPU that loads the library, for the
 * life of the process.  Limits: n_seqs * n_q_heads <= QC_STATIC_MAX_ROWS, n_tokens <=
 * QC_STATIC_MAX_TOKENS, head_dim 64 or 128; anything larger returns QC_ERR_INVALID_ARG and
 * launches nothing.
 *
 * The call performs no device or pinned-host allocation and frees nothing.  Its first call
 * on a device looks up the scratch array's device address (once per device).  That look-up, or
 * the first launch, may be the moment the CUDA runtime loads the library's device code onto the
 * GPU, scratch array included -- the one thing here that does take device memory -- so make one
 * call per device at start-up, while memory may still be taken, and outside any stream capture.
 * The calling thread's current device is the same after the call as before.  All calls share the one array, and it keeps whatever
 * the previous call left there: each call overwrites every entry it later reads, so nothing
 * needs clearing, but two calls whose kernels overlap on the GPU (different streams, or
 * different host threads) race on it.  Serialise them on one stream.  Asynchronous on
 * `cuda_stream`; pointers must be 16-byte aligned. */
#define QC_STATIC_MAX_ROWS 512
#define QC_STATIC_SPLITS 8
#define QC_STATIC_MAX_TOKENS 65536
int32_t qc_attend_static(int32_t device, void* cuda_stream, const void* q_dev, const void* k_dev,
                         const void* v_dev, void* out_dev, int32_t n_seqs, int32_t n_tokens,
                         int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, float softmax_scale);

const char* qc_status_string(int32_t status);

#ifdef __cplusplus
}
#endif
#endif /* QC_H_ */
