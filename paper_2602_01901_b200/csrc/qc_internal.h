// Structures shared by the host runtime (qc_runtime.cu) and the kernels (qc_kernels.cu).
// Not part of the public ABI.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace qc {

constexpr int kPage = 16;      // tokens per page
constexpr int kMaxCons = 4;    // V streams (output layers) one K sweep can feed
constexpr int kMaxChunkPages = 32;
constexpr int kAttendWarps = 12;   // independent workers (warps) per attention CTA; one CTA per SM

// flags of Job / Item
constexpr uint8_t kFlagShared = 1;      // one query scores for every consumer (same weights)
constexpr uint8_t kFlagWriteLogits = 2; // the sweep also stores its scaled scores in the logit cache
constexpr uint8_t kFlagReadLogits = 4;  // the sweep takes its scores from the logit cache: no K tile is read
constexpr uint8_t kFlagStreamEnd = 8;   // (items only) the item's last page is the last page of its stream
constexpr int kFlagCachedShift = 4;     // bit (4 + x): consumer x's query is read from the Q Cache

// layer flags
constexpr uint8_t kLayerOwnsTextK = 1;
constexpr uint8_t kLayerWritesQCache = 2;

// One K sweep: the keys of (k_layer, stream) scored by up to kMaxCons queries, each set of
// weights applied to the V stream of one output layer.
struct Job {
  uint8_t k_layer, stream, n_cons, flags;
  uint8_t v_layer[kMaxCons];
  uint8_t q_layer[kMaxCons];
  uint8_t skip_new;   // bit x: consumer x leaves out the stream's last key (the step's new token, whose
                      // value row of that layer does not exist yet when the sweep runs)
  uint8_t finish;     // bit x: consumer x's output rows are complete once this launch's sweeps of them are
                      // done, so the worker that delivers a row's last partial merges it (no merge launch);
                      // kFinishOwnStream: only this job's stream contributes to those rows in this launch
  uint8_t pad[2];
};
constexpr uint8_t kFinishOwnStream = 0x10;
static_assert(sizeof(Job) == 16, "Job layout");

// One position of the launch plan: a job plus how many visual-stream and text-stream jobs
// precede it in the item list (all launches of a step share one list), and the tiles per page
// (one K tile unless the scores come from the logit cache, one V tile per consumer) of the
// visual-stream and text-stream jobs that precede it in its own launch.  Static per cache.
struct __align__(16) PlanJob {
  Job job;
  int32_t vis_before, text_before, wv_before, wt_before;
};
static_assert(sizeof(PlanJob) == 32, "PlanJob layout");

// One split-KV work item: a chunk of pages of one (job, sequence, head).
struct __align__(16) Item {
  uint8_t k_layer, stream, n_cons, flags;
  uint8_t v_layer[kMaxCons];
  uint8_t q_layer[kMaxCons];
  uint16_t seq_id, seq_idx;
  uint16_t head, slot;
  uint16_t first_page, n_pages;
  uint16_t n_valid_last;
  uint8_t skip_new, finish;     // as in Job
  uint8_t n_heads, pad1;        // query heads head .. head + n_heads - 1 share a KV head (head / group); 1 without GQA
  uint16_t n_pieces;            // static partition, the piece with a row's first page: pieces of the row; else 0
};
static_assert(sizeof(Item) == 32, "Item layout");

// One listed sequence of a step.  Lengths count the new token; ncv chunks of the visual stream
// come first among the n_slots partial slots of an output row; pre_v / pre_t are the numbers
// of items that the sequences listed before this one contribute to one visual / text job
// (under the static partition of a launch: the pages of their visual / text streams).
struct __align__(16) StepSeq {
  int32_t seq_id, len_text, len_vis, n_slots;
  int32_t pre_v, pre_t, ncv, pad;
};
static_assert(sizeof(StepSeq) == 32, "StepSeq layout");

// Step descriptors small enough to travel as a kernel argument instead of a copy.
constexpr int kInlineSeqs = 64;
struct StepInline {
  StepSeq seqs[kInlineSeqs];
};

struct Patch {
  int32_t index, page;
};

// Static partition of one attention launch, as the kernel that plans a step ahead needs it.
struct LaunchDesc {
  int32_t pos_begin, pos_end;
  int32_t part_q, part_k, part_vw, part_workers, part_row_cost;
  int32_t merge_wide;   // a row of the launch may leave more than four partial rows of its visual stream
};
static_assert(sizeof(LaunchDesc) == 32, "LaunchDesc layout");
constexpr int kMaxPlanLaunches = 128;   // launches of a step that can be planned ahead (a launch per layer fits)
constexpr int kPlanWorkers = 2048;      // worker descriptors kept per launch
struct LaunchList {
  LaunchDesc launch[kMaxPlanLaunches];
};

// Where a worker of a statically partitioned launch starts: its first item, the page ids of that
// item's first two pages (K stream, then the V stream of each consumer) so that the first tiles
// can be requested at once, and the cursor from which its later items follow.  Written for every
// launch of a step by one kernel when the step begins; a worker then starts from one 160-byte read.
struct __align__(16) WorkerDesc {
  Item item;                        // n_pages == 0: the worker has no work
  int32_t pids[1 + kMaxCons][2];
  int32_t pad[2];
  int32_t cursor[20];               // a RangeCursor
};
static_assert(sizeof(WorkerDesc) == 160, "WorkerDesc layout");

// Kernel parameter block.
struct Params {
  // cache-lifetime
  CUtensorMap tmap;        // the pool as a 2-D bf16 tensor [pages * hkv * 16 rows][d], box 16 x min(d, 64),
                           // 128-byte swizzle (used by the tensor-core kernel only)
  uint16_t* pool;          // bf16 pages
  int32_t* table;          // [n_layers][4][max_seqs][max_pages]
  uint16_t* qcache;        // bf16 [n_layers][max_seqs][hq][d]
  float* part_acc;         // [n_layers][max_seqs][max_slots][hq][d]
  float2* part_ml;         // [n_layers][max_seqs][max_slots][hq]  (max, sum) in the log2 domain
  float* logits;           // [2 streams][max_seqs][hq][max_pages * 16] scaled scores (log2 domain) of a block's leader
  Item* items;
  const PlanJob* plan;
  const Job* jobs;
  StepSeq* seqs;
  const Patch* patches;
  const uint8_t* layer_flags;
  int32_t* err;
  int32_t* err_host;       // the same word in mapped host memory: the host sees an error without a copy
  int32_t* work_counter;   // [n_layers] next unclaimed item of each attention launch of a step
  uint16_t* row_slots;     // [n_layers][max_seqs][hq][2]: partial rows the visual / the text sweep left for an
                           // output row (static partition only)
  const WorkerDesc* wdesc; // [launches of the step][kPlanWorkers] planned ahead, or null: workers find their own start
  int32_t* row_done;       // [n_layers][max_seqs][hq]: pages of an output row swept so far in the current launch
                           // (the worker that completes the count merges the row and resets it)
  int64_t n_pool_pages;    // bound for page ids (reads never leave the pool)
  int32_t n_layers, hq, hkv, d, group, max_seqs, max_pages, max_slots, chunk_pages;
  int32_t heads_per_item_dim;   // work items per (chunk, sequence): hq, or with GQA hkv * ceil(group / 8)
  int32_t heads_per_item;       // query heads one item covers: 1, or with GQA up to 8 heads of one KV head
  float scale_log2;             // softmax scale * log2(e)
  // per step
  const uint16_t* q;
  const uint16_t* k;
  const uint16_t* v;
  uint16_t* out;
  float* lse;
  int32_t n_seqs, n_pos, n_items, n_patches;   // n_pos: plan positions (jobs) of the step
  int32_t tot_v, tot_t;                        // items of one visual / text job over all listed sequences
  int32_t inline_seqs;                         // 1: the StepSeq array arrives as a kernel argument
  int32_t fused_append;                        // 1: the set-up launch also does the append
  int32_t item_begin, item_end;      // range handled by one attention launch
  int32_t launch_index;              // which work counter that launch uses
  int32_t layer_begin, layer_end;    // range handled by one merge launch
  // static partition of an attention launch: the launch's work, counted in tiles in the order
  // plan position -> listed sequence -> row (head or query group) -> page, is cut into part_vw
  // ranges of part_q tiles; worker w takes ranges w * part_k .. w * part_k + part_k - 1.  A page
  // belongs to the range its first tile falls into.
  int32_t part_static;               // 0: items are claimed from the list
  int32_t part_vw, part_k, part_workers;
  int32_t part_q, part_tiles;        // tiles per range; tiles of the launch
  int32_t part_row_cost;             // what a row counts for besides its pages, in tiles
  int32_t tp_v, tp_t;                // pages of the visual / text streams, summed over the listed sequences
  int32_t pos_begin, pos_end;        // plan positions of the launch
  int32_t slots_per_stream;          // partial-row slots of one stream of an output row (text slots start here)
  int32_t fold_append;               // in-order schedule: the new token's k/v rows (and an ordinary layer's q for the
                                     // Q Cache) are taken from the step's inputs by the attention worker (or the
                                     // merge warp) that meets the end of the layer's text stream, which also stores
                                     // them: no append launch, nothing of a layer is touched before its own launch
  int32_t merge_wide;                // merge: rows may have more than four partial rows of the visual stream
  int32_t debug_drop_tile;           // test hook: every worker of an attention launch leaves out the copy of its first
                                     // tile and waits for it with a short limit (nothing in flight, nothing faults)
  int32_t extra_key_leader;          // merge only, >= 0: the rows also take the step's new token as one more key,
                                     // scored by that layer's Q Cache entry and new k (Eq. 6), valued by the own new v
};

// launchers (qc_kernels.cu); all asynchronous on `stream`
cudaError_t launch_setup(const Params& p, const StepInline* inl, cudaStream_t stream);
cudaError_t launch_append(const Params& p, cudaStream_t stream);
cudaError_t launch_plan(const Params& p, const LaunchList& list, int n_launches, cudaStream_t stream);   // writes p.wdesc
cudaError_t launch_attend(const Params& p, int n_sms, cudaStream_t stream);      // one query head per item
cudaError_t launch_attend_tc(const Params& p, int n_sms, cudaStream_t stream);   // query-group items (GQA)
cudaError_t launch_merge(const Params& p, cudaStream_t stream);
cudaError_t launch_prefill_scatter(const Params& p, const int32_t* tok_seq, const int32_t* tok_stream,
                                   const int32_t* tok_ord, int32_t n_tokens, int32_t tok_stride,
                                   int32_t tok_offset, cudaStream_t stream);
// Tensor maps of one prompt for the tcgen05 prefill kernel: q, k, v as 3-D tensors
// {128, heads, n_layers * T} read in boxes of 64 tokens x one head x 64 elements, and the output
// as a 4-D tensor {128, hq, T, n_layers} written in boxes of 128 tokens x one head x 64 elements
// (the token dimension of its own so that a store is clipped at the end of the prompt).
// One launch unit of the tcgen05 kernel along blockIdx.z: n layers of one lazy block whose scores
// are identical (GLA, Eq. 5: Q and K are the block's first layer's), so that they are computed and
// normalised once and applied to each layer's own V; n = 1 is an ordinary single layer.
struct PrefillPass {
  int32_t n, v[3];
};

constexpr int kPrefillSharedLayers = 3;   // layers one shared-score pass feeds

struct PrefillMaps {
  CUtensorMap q, k, v, out;
};
cudaError_t launch_prefill_attend(const Params& p, const uint8_t* kind_dev, const uint8_t* layer_kind_dev,
                                  const uint8_t* leader_dev, const void* q, const void* k, const void* v, void* out,
                                  int32_t n_tokens, int32_t gla, const PrefillMaps* maps,
                                  const uint8_t* tile_code_dev, int32_t seq_id, int32_t n0_text, int32_t n0_vis,
                                  const PrefillPass* passes_dev, int32_t n_single, int32_t n_shared,
                                  int32_t pair_min_tokens, cudaStream_t stream);   // qc_prefill.cu; maps null or head_dim 64 = mma.sync kernel
cudaError_t configure_prefill_kernels();
cudaError_t launch_calibration(const Params& p, const int32_t* seq_ids_dev, const int32_t* len_text_dev,
                               const int32_t* len_vis_dev, float* rows_dev, int32_t max_len, float* js_dev,
                               cudaStream_t stream);   // qc_calib.cu
cudaError_t configure_kernels(int* attend_smem_bytes);
cudaError_t configure_kernels_tc(int* attend_smem_bytes);

}  // namespace qc
