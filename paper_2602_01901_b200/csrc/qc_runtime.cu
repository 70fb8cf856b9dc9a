// Host runtime behind the C ABI of include/qc.h: context, cache object, paged allocator,
// page tables, per-step planning and kernel launches.  No device memory is allocated here:
// everything lives in the pool and the workspace the caller hands to qc_alloc_cache.

#include "../../include/qc.h"
#include "qc_internal.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <string>
#include <vector>

using namespace qc;

namespace {

constexpr int kStageSlots = 8;       // pinned step-descriptor ring
constexpr int kMaxProfileSteps = 16384;
constexpr int kPrefillBatchTokens = 1 << 16;
// Shared-score passes run one CTA per SM (three accumulators fill tensor memory); that pays once
// a CTA has enough key tiles: measured -16 % / -10 % call time at 2048 / 3008 tokens, +4 % / +9 %
// at 1120 / 675.
constexpr int kPrefillShareMinTokens = 1536;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct SeqState {
  bool active = false;
  int32_t len_text = 0, len_vis = 0;
  std::vector<int32_t> alloc_order;
};

// One attention launch: a run of consecutive lazy blocks.
struct LaunchGroup {
  int job_begin, job_end, layer_begin, layer_end;
  int extra_key_leader;   // >= 0: the merge of these layers adds the step's new token (in-order schedule, GLA followers)
  bool needs_merge;       // some output row of these layers is not merged by the attention kernel itself
  int wv, wt;             // tiles per page summed over the launch's visual / text jobs
  int w_min, w_max;       // smallest / largest tiles per page of a job of the launch
  int w_max_v, w_max_t;   // largest tiles per page among its visual / text jobs
};

// A step opened by qc_decode_begin: what its layer-by-layer launches need.
struct OpenStep {
  bool active = false;
  Params p{};
  LaunchList launches{};
  bool use_static = false;
  int64_t tot_v = 0, tot_t = 0, bytes = 0;
  int next_layer = 0;
};

struct Layout {   // byte offsets into the workspace
  size_t table, layer_flags, layer_kind, leader, jobs, plan, qcache, part_acc, part_ml, logits, items, step, err, counters, row_slots, row_done, wdesc, stage_q,
      stage_k, stage_v, stage_out, stage_lse, tok, total;
  size_t step_seqs, step_patches, step_bytes;   // offsets inside the step block
};

}  // namespace

struct qc_ctx {
  int device = 0;
  cudaStream_t stream = nullptr;
  int n_sms = 0;
};

struct qc_cache {
  qc_ctx* ctx = nullptr;
  qc_config cfg{};
  std::vector<uint8_t> kind;
  std::vector<int> leader;
  std::vector<uint8_t> layer_flags;
  int D = 0, hq = 0, hkv = 0, group = 0;
  int heads_per_item = 1;  // query heads one work item covers (8 with GQA: one query group, or a slice of it)
  int items_per_chunk = 0; // work items per (chunk, sequence)
  CUtensorMap tmap{};      // the pool as a swizzled 2-D tensor (query-group kernel)
  bool paged = true;
  int max_pages = 0;       // per stream
  int chunk_pages = 0, min_chunk_pages = 0, max_slots = 0;
  bool auto_split = false;         // choose chunk_pages per step from the amount of work
  int n_visual_jobs = 0, n_text_jobs = 0;
  int64_t visual_row_reads = 0, text_row_reads = 0;   // K/V rows read per visual / text token per step
  // launch plan: jobs in item-list order (launch group by launch group, heaviest first)
  std::vector<PlanJob> plan;                 // plan[p] for p < n_pos, uploaded to the workspace
  std::vector<int> plan_vis_before, plan_text_before;   // n_pos + 1 entries
  std::vector<LaunchGroup> groups;
  std::vector<std::pair<int, int>> group_pos;           // plan positions [begin, end) of each launch
  bool plan_dirty = true;
  int plan_per = 0;               // blocks per launch the plan was built for (0 = all in one)
  // host-buffer entry point: copies of one launch group overlap the kernels of the others
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  std::vector<cudaEvent_t> ev_in, ev_done;
  bool prefill_tcgen05 = true;    // head_dim 128: tcgen05 kernel; otherwise (or when switched off) mma.sync kernel
  bool pool_map_ok = false;       // c->tmap was encoded
  int prefill_pair_min_tokens = 0;   // prompts this long that start a sequence run two query tiles per CTA (0: never)
  int prefill_shared = 1;         // GLA prefill: layers of a block whose scores coincide share one score pass
                                  // (0 never, 1 for prompts of kPrefillShareMinTokens or more, 2 always)
  std::vector<PrefillPass> prefill_passes;   // singles first, then shared passes (GLA only; else empty)
  int prefill_n_single = 0, prefill_n_shared = 0;
  int64_t n_pool_pages = 0;
  int layers_per_launch = 0;
  float scale = 0.f;

  uint8_t* ws = nullptr;
  uint16_t* pool = nullptr;
  Layout lay{};
  size_t max_items = 0, max_segs = 0, max_patches = 0;

  std::vector<int32_t> table;          // host mirror
  std::vector<int32_t> free_stack;
  std::vector<SeqState> seqs;
  std::vector<Job> jobs;
  std::vector<std::pair<int, int>> block_jobs;   // per lazy block: [job_begin, job_end)
  std::vector<std::pair<int, int>> block_layers; // per lazy block: [layer_begin, layer_end)
  std::vector<Job> layer_jobs;                    // per-layer schedule (logit cache)
  std::vector<std::pair<int, int>> layer_job_range;   // per layer: [job_begin, job_end) in layer_jobs
  std::vector<Job> inorder_jobs;                  // in-order schedule (a leader's launch also sweeps its followers' cached V)
  std::vector<std::pair<int, int>> inorder_job_range;
  std::vector<int> inorder_extra_key;             // per layer: the leader whose new token the merge adds, or -1
  int slots_per_stream = 0;
  int static_partition = -1;      // -1: static ranges when a step is several launches; 0 never; 1 always
  bool fused_merge = false;       // the worker that delivers an output row's last partial merges it (no merge launch)
  bool fold_append = true;        // in-order schedule: new rows are taken and stored by the layer's own launch
  bool plan_ahead = true;         // one kernel per step works out where every worker of every launch starts
  int static_row_cost = 4;        // tiles a row counts for besides its pages (a worker's cost of one more item)
  int static_min_tiles = 6;       // a static range is at least this long when the launch has the work for it
                                  // (measured on launches of one layer: 3..8 equal, 12 and 16 slower)
  int text_streams_per_seq = 0;        // pages a sequence needs when its text crosses a page

  // pinned staging ring for step descriptors
  uint8_t* pinned = nullptr;
  int32_t* err_host = nullptr;        // mapped host word the kernels mirror the device error word into
  int32_t* err_host_dev = nullptr;    // its device address
  int debug_drop_tile = 0;
  cudaEvent_t stage_done[kStageSlots]{};
  bool stage_used[kStageSlots]{};
  int stage_next = 0;

  // profiling
  int profile = 0;                     // 1: events per step; 2: also around every attention launch
  std::vector<cudaEvent_t> ev_launch;  // profile 2: begin / end of every attention launch
  int ev_launches = 0;
  std::vector<cudaEvent_t> ev;         // 4 per step: step begin, attend begin, attend end, step end
  int ev_steps = 0;
  int64_t prof_bytes = 0, prof_items = 0;
  std::vector<cudaEvent_t> ev_prefill; // 2 per profiled qc_prefill_attend call
  int ev_prefill_calls = 0;
  double prof_prefill_flops = 0.0;

  int64_t decode_steps = 0, attend_launches = 0, kernel_launches = 0, kv_bytes_swept = 0;
  OpenStep open;
};

namespace {

inline bool owns(const qc_cache* c, int layer, int stream) {
  if (stream >= 2 || c->kind[layer] == QC_LAYER_FULL) return true;
  if (stream == QC_STREAM_K_TEXT) return c->cfg.lazy_mode != QC_MODE_GLA;
  return false;
}

inline size_t trow(const qc_cache* c, int layer, int stream, int seq) {
  return ((static_cast<size_t>(layer) * 4 + stream) * c->cfg.max_seqs + seq) * c->max_pages;
}

int validate_config(const qc_config* cfg) {
  if (!cfg || !cfg->layer_kind) return QC_ERR_INVALID_ARG;
  if (cfg->n_layers < 1 || cfg->n_layers > 127) return QC_ERR_INVALID_ARG;
  if (cfg->n_kv_heads < 1 || cfg->n_q_heads < 1 || cfg->n_q_heads % cfg->n_kv_heads) return QC_ERR_INVALID_ARG;
  if (cfg->n_q_heads > 65535) return QC_ERR_INVALID_ARG;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return QC_ERR_UNSUPPORTED;
  if (cfg->page_size != 16 && cfg->page_size != 0) return QC_ERR_UNSUPPORTED;
  if (cfg->max_seqs < 1 || cfg->max_seqs > 4096) return QC_ERR_INVALID_ARG;
  if (cfg->max_tokens_per_seq < 1 || cfg->max_tokens_per_seq > (1 << 20) - 16) return QC_ERR_INVALID_ARG;
  if (cfg->page_size == 16 && (cfg->n_pages < 1 || cfg->n_pages > 0x7fffffffLL)) return QC_ERR_INVALID_ARG;
  if (cfg->lazy_mode < 0 || cfg->lazy_mode > 2) return QC_ERR_INVALID_ARG;
  if (cfg->split_tokens != 0 &&
      (cfg->split_tokens % 16 || cfg->split_tokens < 16 || cfg->split_tokens > 16 * kMaxChunkPages))
    return QC_ERR_INVALID_ARG;
  if (!(cfg->softmax_scale >= 0.f) || !std::isfinite(cfg->softmax_scale)) return QC_ERR_INVALID_ARG;
  for (int l = 0; l < cfg->n_layers; ++l)
    if (cfg->layer_kind[l] != QC_LAYER_FULL && cfg->layer_kind[l] != QC_LAYER_LAZY) return QC_ERR_INVALID_ARG;
  if (cfg->layer_kind[0] != QC_LAYER_FULL) return QC_ERR_STATE;
  return QC_OK;
}

// Jobs of the whole stack, lazy block by lazy block.
void build_jobs(const qc_config* cfg, std::vector<Job>& jobs, std::vector<std::pair<int, int>>& block_jobs,
                std::vector<std::pair<int, int>>& block_layers) {
  const int N = cfg->n_layers;
  // own-query sweeps keep one set of query fragments per consumer in registers: the
  // query-group (tensor-core) kernel feeds two layers per sweep, the one-head kernel four
  const int max_own = cfg->n_q_heads > cfg->n_kv_heads ? 2 : kMaxCons;
  int l = 0;
  while (l < N) {
    const int c = l;
    int e = l + 1;
    while (e < N && cfg->layer_kind[e] == QC_LAYER_LAZY) ++e;   // followers c+1 .. e-1
    const int job0 = static_cast<int>(jobs.size());
    auto shared_jobs = [&](int stream, bool cached) {
      // the leader's query scores once; weights applied to the V of the leader and followers
      for (int first = c; first < e; first += kMaxCons) {
        Job j{};
        j.k_layer = static_cast<uint8_t>(c);
        j.stream = static_cast<uint8_t>(stream);
        j.n_cons = static_cast<uint8_t>(std::min(kMaxCons, e - first));
        j.flags = kFlagShared;
        j.finish = static_cast<uint8_t>((1u << j.n_cons) - 1);   // a block's launch sweeps both streams of all its layers
        for (int x = 0; x < j.n_cons; ++x) {
          j.v_layer[x] = static_cast<uint8_t>(first + x);
          j.q_layer[x] = static_cast<uint8_t>(c);
        }
        if (cached && e - c > 1) j.flags |= static_cast<uint8_t>(1u << kFlagCachedShift);
        jobs.push_back(j);
      }
    };
    auto own_query_jobs_on_leader_keys = [&](int stream) {   // Eq. 8: own q on the leader's visual K
      for (int first = c; first < e; first += max_own) {
        Job j{};
        j.k_layer = static_cast<uint8_t>(c);
        j.stream = static_cast<uint8_t>(stream);
        j.n_cons = static_cast<uint8_t>(std::min(max_own, e - first));
        j.flags = (j.n_cons == 1) ? kFlagShared : 0;
        j.finish = static_cast<uint8_t>((1u << j.n_cons) - 1);
        for (int x = 0; x < j.n_cons; ++x) {
          j.v_layer[x] = static_cast<uint8_t>(first + x);
          j.q_layer[x] = static_cast<uint8_t>(first + x);
        }
        jobs.push_back(j);
      }
    };
    auto own_jobs = [&](int stream) {   // every layer of the block: own q, own K, own V
      for (int x = c; x < e; ++x) {
        Job j{};
        j.k_layer = static_cast<uint8_t>(x);
        j.stream = static_cast<uint8_t>(stream);
        j.n_cons = 1;
        j.flags = kFlagShared;
        j.finish = 1;
        j.v_layer[0] = static_cast<uint8_t>(x);
        j.q_layer[0] = static_cast<uint8_t>(x);
        jobs.push_back(j);
      }
    };
    switch (cfg->lazy_mode) {
      case QC_MODE_VLA_QC:
        shared_jobs(1, true);
        own_jobs(0);
        break;
      case QC_MODE_VLA_EQ8:
        own_query_jobs_on_leader_keys(1);
        own_jobs(0);
        break;
      default:   // GLA
        shared_jobs(1, true);
        shared_jobs(0, true);
        break;
    }
    block_jobs.emplace_back(job0, static_cast<int>(jobs.size()));
    block_layers.emplace_back(c, e);
    l = e;
  }
}

// Jobs of the per-layer schedule, layer by layer: every sweep feeds one layer.  A leader with
// followers stores the scaled scores that its followers share (VLA_QC: of the visual keys; GLA: of
// all keys) in the logit cache; such a follower sweeps its own V pages with those scores and reads
// no K at all.  VLA_EQ8 followers score the leader's visual keys with their own query.
void build_layer_jobs(const qc_config* cfg, std::vector<Job>& jobs, std::vector<std::pair<int, int>>& layer_jobs) {
  const int N = cfg->n_layers;
  int leader = 0;
  for (int l = 0; l < N; ++l) {
    const bool lazy = cfg->layer_kind[l] == QC_LAYER_LAZY;
    if (!lazy) leader = l;
    const bool has_followers = !lazy && l + 1 < N && cfg->layer_kind[l + 1] == QC_LAYER_LAZY;
    const int job0 = static_cast<int>(jobs.size());
    for (int stream = 1; stream >= 0; --stream) {
      const bool shared_scores =
          cfg->lazy_mode == QC_MODE_GLA || (cfg->lazy_mode == QC_MODE_VLA_QC && stream == 1);
      Job j{};
      j.stream = static_cast<uint8_t>(stream);
      j.n_cons = 1;
      j.flags = kFlagShared;
      j.finish = 1;   // the layer's launch sweeps both of its streams
      j.v_layer[0] = static_cast<uint8_t>(l);
      j.q_layer[0] = static_cast<uint8_t>(l);
      j.k_layer = static_cast<uint8_t>(l);
      if (lazy) {
        if (shared_scores) {
          j.k_layer = static_cast<uint8_t>(leader);   // (lengths and chunking follow the leader's stream)
          j.q_layer[0] = static_cast<uint8_t>(leader);
          j.flags |= kFlagReadLogits;
        } else if (stream == 1) {
          j.k_layer = static_cast<uint8_t>(leader);   // Eq. 8: own query on the leader's visual keys
        }
      } else if (has_followers && shared_scores) {
        j.flags |= kFlagWriteLogits;
      }
      jobs.push_back(j);
    }
    layer_jobs.emplace_back(job0, static_cast<int>(jobs.size()));
  }
}

// Jobs of the in-order schedule, layer by layer: the launch of layer l uses nothing of the layers
// after l, as in a model where a layer's q/k/v only exist once the previous layer has run.  What a
// follower shares with its leader are the scores (GLA: Q and K are the leader's, Eq. 6; VLA_QC: the
// cached query on the leader's visual K), and the V rows they weight were cached before the step:
// the visual stream never holds the new token, the text stream holds it last.  So the leader's
// sweep also weights its followers' cached V rows, one K read and one set of weights for up to
// kMaxCons layers, and leaves their partial rows behind.  A VLA_QC follower's own launch is its
// text sweep (own q, own text K); a GLA follower has no sweep at all: its merge adds the new token
// as one more key.  VLA_EQ8 followers score the leader's visual keys with their own query (Eq. 8
// shares K only), in their own launch.
void build_inorder_jobs(const qc_config* cfg, std::vector<Job>& jobs, std::vector<std::pair<int, int>>& layer_jobs,
                        std::vector<int>& extra_key) {
  const int N = cfg->n_layers;
  extra_key.assign(N, -1);
  int l = 0;
  while (l < N) {
    const int c = l;
    int e = l + 1;
    while (e < N && cfg->layer_kind[e] == QC_LAYER_LAZY) ++e;
    auto own = [&](int layer, int k_layer, int stream, bool only_stream) {
      Job j{};
      j.k_layer = static_cast<uint8_t>(k_layer);
      j.stream = static_cast<uint8_t>(stream);
      j.n_cons = 1;
      j.flags = kFlagShared;
      j.finish = static_cast<uint8_t>(1 | (only_stream ? kFinishOwnStream : 0));
      j.v_layer[0] = static_cast<uint8_t>(layer);
      j.q_layer[0] = static_cast<uint8_t>(layer);
      jobs.push_back(j);
    };
    auto shared = [&](int stream, bool skip_new) {   // the leader's query; consumers c .. e-1, kMaxCons per sweep
      for (int first = c; first < e; first += kMaxCons) {
        Job j{};
        j.k_layer = static_cast<uint8_t>(c);
        j.stream = static_cast<uint8_t>(stream);
        j.n_cons = static_cast<uint8_t>(std::min(kMaxCons, e - first));
        j.flags = kFlagShared;
        for (int x = 0; x < j.n_cons; ++x) {
          j.v_layer[x] = static_cast<uint8_t>(first + x);
          j.q_layer[x] = static_cast<uint8_t>(c);
          if (skip_new && first + x != c) j.skip_new |= static_cast<uint8_t>(1u << x);
          if (first + x == c) j.finish |= static_cast<uint8_t>(1u << x);   // the followers' rows are completed later
        }
        jobs.push_back(j);
      }
    };
    // the leader's launch
    int job0 = static_cast<int>(jobs.size());
    if (cfg->lazy_mode == QC_MODE_VLA_EQ8 || e - c == 1) {
      own(c, c, 1, false);
      own(c, c, 0, false);
    } else if (cfg->lazy_mode == QC_MODE_VLA_QC) {
      shared(1, false);
      own(c, c, 0, false);
    } else {
      shared(1, false);
      shared(0, true);
    }
    layer_jobs.emplace_back(job0, static_cast<int>(jobs.size()));
    // the followers' launches
    for (int f = c + 1; f < e; ++f) {
      job0 = static_cast<int>(jobs.size());
      if (cfg->lazy_mode == QC_MODE_VLA_EQ8) {
        own(f, c, 1, false);
        own(f, f, 0, false);
      } else if (cfg->lazy_mode == QC_MODE_VLA_QC) {
        own(f, f, 0, true);   // the visual partials are there already
      } else {
        extra_key[f] = c;
      }
      layer_jobs.emplace_back(job0, static_cast<int>(jobs.size()));
    }
    l = e;
  }
}

struct Sizes {
  int D, hq, hkv, max_pages, chunk_pages, max_slots, slots_per_stream;
  int64_t n_pool_pages;
  size_t page_bytes, pool_bytes, max_items, max_segs, max_patches;
  Layout lay;
};

int compute_sizes(const qc_config* cfg, Sizes* s) {
  int st = validate_config(cfg);
  if (st != QC_OK) return st;
  s->D = cfg->head_dim;
  s->hq = cfg->n_q_heads;
  s->hkv = cfg->n_kv_heads;
  s->max_pages = (cfg->max_tokens_per_seq + kPage - 1) / kPage;
  const int split = cfg->split_tokens ? cfg->split_tokens : 64;   // auto: the smallest chunk the per-step choice may take
  s->chunk_pages = split / kPage;
  // partial-row slots per stream of an output row: one per chunk when items are claimed.  Under the
  // static partition a row of P pages at w tiles per page is cut into at most P w / q + 2 pieces by
  // ranges of q tiles, and q may not exceed 30 pages of the launch's lightest job (a piece holds at
  // most kMaxChunkPages page ids); tiles per page differ by at most 5x between the jobs of a launch
  // (1 .. 1 + kMaxCons), so max_pages / 3 + 2 slots always leave room for a q within both bounds
  s->slots_per_stream = std::max((s->max_pages + s->chunk_pages - 1) / s->chunk_pages, (s->max_pages + 2) / 3 + 2);
  s->max_slots = 2 * s->slots_per_stream;
  s->page_bytes = static_cast<size_t>(s->hkv) * kPage * s->D * 2;
  if (cfg->page_size == 0)
    s->n_pool_pages = static_cast<int64_t>(cfg->n_layers) * 4 * cfg->max_seqs * s->max_pages;
  else
    s->n_pool_pages = cfg->n_pages;
  if (s->n_pool_pages > 0x7fffffffLL) return QC_ERR_INVALID_ARG;
  s->pool_bytes = static_cast<size_t>(s->n_pool_pages) * s->page_bytes;

  std::vector<Job> jobs;
  std::vector<std::pair<int, int>> bj, bl;
  build_jobs(cfg, jobs, bj, bl);
  std::vector<Job> layer_jobs;
  std::vector<std::pair<int, int>> lj;
  build_layer_jobs(cfg, layer_jobs, lj);
  std::vector<Job> inorder_jobs;
  std::vector<int> extra;
  lj.clear();
  build_inorder_jobs(cfg, inorder_jobs, lj, extra);
  const size_t n_jobs = std::max(std::max(jobs.size(), layer_jobs.size()), inorder_jobs.size());   // any schedule fits
  const size_t chunks_per_stream = (s->max_pages + s->chunk_pages - 1) / s->chunk_pages;
  s->max_segs = n_jobs * cfg->max_seqs;
  s->max_items = s->max_segs * chunks_per_stream * s->hq;
  s->max_patches = static_cast<size_t>(cfg->n_layers) * 2 * cfg->max_seqs;

  Layout& L = s->lay;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  const size_t N = cfg->n_layers, S = cfg->max_seqs;
  L.table = take(N * 4 * S * s->max_pages * sizeof(int32_t));
  L.layer_flags = take(N);
  L.layer_kind = take(N);
  L.leader = take(N);
  L.jobs = take(n_jobs * sizeof(Job));
  L.plan = take(n_jobs * sizeof(PlanJob));
  L.qcache = take(N * S * s->hq * s->D * 2);
  L.part_acc = take(N * S * s->max_slots * s->hq * s->D * sizeof(float));
  L.part_ml = take(N * S * s->max_slots * s->hq * sizeof(float2));
  L.logits = take(2 * S * s->hq * static_cast<size_t>(s->max_pages) * kPage * sizeof(float));
  L.items = take(s->max_items * sizeof(Item));
  // step block: header-free arrays at fixed offsets
  L.step_seqs = 0;
  L.step_patches = align_up(L.step_seqs + S * sizeof(StepSeq), 16);
  L.step_bytes = align_up(L.step_patches + s->max_patches * sizeof(Patch), 256);
  L.step = take(L.step_bytes);
  L.err = take(256);
  L.counters = take(N * sizeof(int32_t));
  L.row_slots = take(N * S * s->hq * 2 * sizeof(uint16_t));
  L.row_done = take(N * S * s->hq * sizeof(int32_t));
  L.wdesc = take(std::min<size_t>(N, kMaxPlanLaunches) * kPlanWorkers * sizeof(WorkerDesc));
  L.stage_q = take(N * S * s->hq * s->D * 2);
  L.stage_k = take(N * S * s->hkv * s->D * 2);
  L.stage_v = take(N * S * s->hkv * s->D * 2);
  L.stage_out = take(N * S * s->hq * s->D * 2);
  L.stage_lse = take(N * S * s->hq * sizeof(float));
  L.tok = take(static_cast<size_t>(kPrefillBatchTokens) * 3 * sizeof(int32_t));
  L.total = off;
  return QC_OK;
}

#define QC_CUDA(expr)                            \
  do {                                           \
    cudaError_t e__ = (expr);                    \
    if (e__ != cudaSuccess) return QC_ERR_CUDA;  \
  } while (0)

Params base_params(const qc_cache* c) {
  Params p{};
  p.pool = c->pool;
  p.table = reinterpret_cast<int32_t*>(c->ws + c->lay.table);
  p.qcache = reinterpret_cast<uint16_t*>(c->ws + c->lay.qcache);
  p.part_acc = reinterpret_cast<float*>(c->ws + c->lay.part_acc);
  p.part_ml = reinterpret_cast<float2*>(c->ws + c->lay.part_ml);
  p.logits = reinterpret_cast<float*>(c->ws + c->lay.logits);
  p.items = reinterpret_cast<Item*>(c->ws + c->lay.items);
  p.plan = reinterpret_cast<const PlanJob*>(c->ws + c->lay.plan);
  p.jobs = reinterpret_cast<const Job*>(c->ws + c->lay.jobs);
  p.seqs = reinterpret_cast<StepSeq*>(c->ws + c->lay.step + c->lay.step_seqs);
  p.patches = reinterpret_cast<const Patch*>(c->ws + c->lay.step + c->lay.step_patches);
  p.layer_flags = c->ws + c->lay.layer_flags;
  p.err = reinterpret_cast<int32_t*>(c->ws + c->lay.err);
  p.err_host = c->err_host_dev;
  p.debug_drop_tile = c->debug_drop_tile;
  p.work_counter = reinterpret_cast<int32_t*>(c->ws + c->lay.counters);
  p.row_slots = reinterpret_cast<uint16_t*>(c->ws + c->lay.row_slots);
  p.row_done = reinterpret_cast<int32_t*>(c->ws + c->lay.row_done);
  p.slots_per_stream = c->slots_per_stream;
  p.extra_key_leader = -1;
  p.n_pool_pages = c->n_pool_pages;
  p.n_layers = c->cfg.n_layers;
  p.hq = c->hq;
  p.hkv = c->hkv;
  p.d = c->D;
  p.group = c->group;
  p.max_seqs = c->cfg.max_seqs;
  p.max_pages = c->max_pages;
  p.max_slots = c->max_slots;
  p.chunk_pages = c->chunk_pages;
  p.heads_per_item_dim = c->items_per_chunk;
  p.heads_per_item = c->heads_per_item;
  p.tmap = c->tmap;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  return p;
}

// Pop pages for `n_new` more pages of (layer, stream, seq); records them in the host mirror.
void grow_stream(qc_cache* c, int layer, int stream, int seq, int have, int n_new, std::vector<Patch>* patches) {
  for (int i = 0; i < n_new; ++i) {
    const int32_t pid = c->free_stack.back();
    c->free_stack.pop_back();
    const size_t idx = trow(c, layer, stream, seq) + have + i;
    c->table[idx] = pid;
    c->seqs[seq].alloc_order.push_back(pid);
    if (patches) patches->push_back(Patch{static_cast<int32_t>(idx), pid});
  }
}

inline int pages_for(int tokens) { return (tokens + kPage - 1) / kPage; }

// The pool seen as a 2-D bf16 tensor [n_pool_pages * hkv * 16 rows][D]: a (page, head) tile is
// 16 consecutive rows.  Box = 16 rows x 64 elements (128 bytes) with the 128-byte swizzle, so
// a D = 128 tile is fetched as two column halves.  The driver entry point is looked up at run
// time; nothing links against the driver library.
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn tensor_map_encoder() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  return reinterpret_cast<EncodeFn>(fn);
}

// A prompt tensor [n_layers][T][heads][128] bf16 as a 3-D tensor {128, heads, n_layers * T}: a
// box is 64 tokens x one head x 64 elements (128 bytes) with the 128-byte swizzle.  Rows past
// the end of the tensor read as zero.
int make_prompt_tensor_map(CUtensorMap* out, const void* base, int n_layers, int T, int heads) {
  EncodeFn enc = tensor_map_encoder();
  if (!enc) return QC_ERR_CUDA;
  const cuuint64_t dims[3] = {128, static_cast<cuuint64_t>(heads), static_cast<cuuint64_t>(n_layers) * T};
  const cuuint64_t strides[2] = {128 * 2, static_cast<cuuint64_t>(heads) * 128 * 2};
  const cuuint32_t box[3] = {64, 1, 64};
  const cuuint32_t elem_strides[3] = {1, 1, 1};
  const CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
                         elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? QC_OK : QC_ERR_CUDA;
}

// The prefill output [n_layers][T][hq][128] bf16 as a 4-D tensor {128, hq, T, n_layers}: a box is
// 128 tokens x one head x 64 elements; rows of a box past token T are not written.
int make_output_tensor_map(CUtensorMap* out, void* base, int n_layers, int T, int heads) {
  EncodeFn enc = tensor_map_encoder();
  if (!enc) return QC_ERR_CUDA;
  const cuuint64_t dims[4] = {128, static_cast<cuuint64_t>(heads), static_cast<cuuint64_t>(T),
                              static_cast<cuuint64_t>(n_layers)};
  const cuuint64_t strides[3] = {128 * 2, static_cast<cuuint64_t>(heads) * 128 * 2,
                                 static_cast<cuuint64_t>(T) * heads * 128 * 2};
  const cuuint32_t box[4] = {64, 1, 128, 1};
  const cuuint32_t elem_strides[4] = {1, 1, 1, 1};
  const CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, elem_strides,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? QC_OK : QC_ERR_CUDA;
}

int make_pool_tensor_map(qc_cache* c) {
  EncodeFn enc = tensor_map_encoder();
  if (!enc) return QC_ERR_CUDA;
  const cuuint64_t rows = static_cast<cuuint64_t>(c->n_pool_pages) * c->hkv * kPage;
  if (rows > 0x7fffffffULL) return QC_ERR_INVALID_ARG;   // tile coordinates are 32-bit
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(c->D), rows};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(c->D) * 2};
  const cuuint32_t box[2] = {64, kPage};
  const cuuint32_t elem_strides[2] = {1, 1};
  const CUresult r = enc(
      &c->tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, c->pool, dims, strides, box, elem_strides,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? QC_OK : QC_ERR_CUDA;
}

// Launch groups and the item-list order of the jobs.  Within a launch the heaviest sweeps (most
// tiles per page, visual before text) come first: items are claimed in list order, so the work
// left for the end of the launch comes in small pieces.
int rebuild_plan(qc_cache* c, int per_launch) {
  c->groups.clear();
  c->group_pos.clear();
  c->plan.clear();
  c->plan_vis_before.assign(1, 0);
  c->plan_text_before.assign(1, 0);
  // per_launch -1: the per-layer schedule with the logit cache; -2: the in-order schedule (one
  // launch per layer, a leader's launch also sweeps its followers' cached V); otherwise launches of
  // `per_launch` lazy blocks (0 = all blocks in one launch)
  const bool per_layer = per_launch < 0;
  const std::vector<Job>& jobs = per_launch == -2 ? c->inorder_jobs : (per_launch == -1 ? c->layer_jobs : c->jobs);
  const std::vector<std::pair<int, int>>& layer_range = per_launch == -2 ? c->inorder_job_range : c->layer_job_range;
  const int nb = static_cast<int>(per_layer ? layer_range.size() : c->block_jobs.size());
  const int per = per_layer ? 1 : (per_launch == 0 ? nb : per_launch);
  c->n_visual_jobs = c->n_text_jobs = 0;
  c->visual_row_reads = c->text_row_reads = 0;
  auto tiles_per_page = [](const Job& j) { return ((j.flags & kFlagReadLogits) ? 0 : 1) + j.n_cons; };
  for (const Job& j : jobs) {
    (j.stream ? c->n_visual_jobs : c->n_text_jobs)++;
    (j.stream ? c->visual_row_reads : c->text_row_reads) += tiles_per_page(j);
  }
  std::vector<int> order;
  for (int b = 0; b < nb; b += per) {
    const int e = std::min(nb, b + per);
    LaunchGroup g = per_layer ? LaunchGroup{layer_range[b].first, layer_range[b].second, b, b + 1}
                              : LaunchGroup{c->block_jobs[b].first, c->block_jobs[e - 1].second,
                                            c->block_layers[b].first, c->block_layers[e - 1].second};
    g.extra_key_leader = per_launch == -2 ? c->inorder_extra_key[b] : -1;
    order.resize(g.job_end - g.job_begin);
    for (int j = g.job_begin; j < g.job_end; ++j) order[j - g.job_begin] = j;
    std::stable_sort(order.begin(), order.end(), [&](int x, int y) {
      const Job &jx = jobs[x], &jy = jobs[y];
      if (jx.n_cons != jy.n_cons) return jx.n_cons > jy.n_cons;
      return jx.stream > jy.stream;
    });
    const int begin = static_cast<int>(c->plan.size());
    g.wv = g.wt = g.w_max = g.w_max_v = g.w_max_t = 0;
    g.w_min = 1 << 20;
    std::vector<bool> finished(c->cfg.n_layers, false);
    for (int j : order) {
      const int vb = c->plan_vis_before.back(), tb = c->plan_text_before.back();
      Job job = jobs[j];
      if (!c->fused_merge) job.finish = 0;
      for (int x = 0; x < job.n_cons; ++x)
        if ((job.finish >> x) & 1) finished[job.v_layer[x]] = true;
      c->plan.push_back(PlanJob{job, vb, tb, g.wv, g.wt});
      c->plan_vis_before.push_back(vb + (jobs[j].stream ? 1 : 0));
      c->plan_text_before.push_back(tb + (jobs[j].stream ? 0 : 1));
      const int w = tiles_per_page(jobs[j]);
      (jobs[j].stream ? g.wv : g.wt) += w;
      int& w_max_s = jobs[j].stream ? g.w_max_v : g.w_max_t;
      w_max_s = std::max(w_max_s, w);
      g.w_min = std::min(g.w_min, w);
      g.w_max = std::max(g.w_max, w);
    }
    g.needs_merge = false;
    for (int l = g.layer_begin; l < g.layer_end; ++l) g.needs_merge = g.needs_merge || !finished[l];
    c->groups.push_back(g);
    c->group_pos.emplace_back(begin, static_cast<int>(c->plan.size()));
  }
  QC_CUDA(cudaMemcpyAsync(c->ws + c->lay.plan, c->plan.data(), c->plan.size() * sizeof(PlanJob),
                          cudaMemcpyHostToDevice, c->ctx->stream));
  QC_CUDA(cudaStreamSynchronize(c->ctx->stream));   // the host vector may be rebuilt later
  c->plan_dirty = false;
  c->plan_per = per_launch;
  return QC_OK;
}

int sync_and_check(qc_cache* c) {
  QC_CUDA(cudaStreamSynchronize(c->ctx->stream));
  return QC_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------

extern "C" {

const char* qc_status_string(int32_t s) {
  switch (s) {
    case QC_OK: return "ok";
    case QC_ERR_INVALID_ARG: return "invalid argument";
    case QC_ERR_UNSUPPORTED: return "unsupported configuration";
    case QC_ERR_OOM_PAGES: return "out of pages";
    case QC_ERR_STATE: return "invalid state";
    case QC_ERR_CUDA: return "CUDA error";
    case QC_ERR_TIMEOUT: return "device wait timed out";
    case QC_ERR_BAD_PAGE: return "page id outside the pool";
    case QC_ERR_PLAN: return "work range outside its planned limits";
    default: return "unknown status";
  }
}

int32_t qc_init(int32_t device, void* cuda_stream, qc_ctx** out) {
  if (!out || device < 0) return QC_ERR_INVALID_ARG;
  *out = nullptr;
  int n_dev = 0;
  QC_CUDA(cudaGetDeviceCount(&n_dev));
  if (device >= n_dev) return QC_ERR_INVALID_ARG;
  QC_CUDA(cudaSetDevice(device));
  cudaDeviceProp prop;
  QC_CUDA(cudaGetDeviceProperties(&prop, device));
  if (prop.major < 10) return QC_ERR_UNSUPPORTED;
  int smem = 0, smem_tc = 0;
  QC_CUDA(configure_kernels(&smem));
  QC_CUDA(configure_kernels_tc(&smem_tc));
  QC_CUDA(configure_prefill_kernels());
  if (static_cast<size_t>(std::max(smem, smem_tc)) > prop.sharedMemPerBlockOptin) return QC_ERR_UNSUPPORTED;
  qc_ctx* ctx = new (std::nothrow) qc_ctx();
  if (!ctx) return QC_ERR_INVALID_ARG;
  ctx->device = device;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  ctx->n_sms = prop.multiProcessorCount;
  *out = ctx;
  return QC_OK;
}

int32_t qc_cache_bytes_required(const qc_config* cfg, size_t* pool_bytes, size_t* workspace_bytes) {
  Sizes s;
  int st = compute_sizes(cfg, &s);
  if (st != QC_OK) return st;
  if (pool_bytes) *pool_bytes = s.pool_bytes;
  if (workspace_bytes) *workspace_bytes = s.lay.total;
  return QC_OK;
}

int32_t qc_alloc_cache(qc_ctx* ctx, const qc_config* cfg, void* pool_dev, size_t pool_bytes, void* workspace_dev,
                       size_t workspace_bytes, qc_cache** out) {
  if (!ctx || !out || !pool_dev || !workspace_dev) return QC_ERR_INVALID_ARG;
  *out = nullptr;
  Sizes s;
  int st = compute_sizes(cfg, &s);
  if (st != QC_OK) return st;
  if (pool_bytes < s.pool_bytes || workspace_bytes < s.lay.total) return QC_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(pool_dev) & 255) || (reinterpret_cast<uintptr_t>(workspace_dev) & 255))
    return QC_ERR_INVALID_ARG;
  QC_CUDA(cudaSetDevice(ctx->device));

  qc_cache* c = new (std::nothrow) qc_cache();
  if (!c) return QC_ERR_INVALID_ARG;
  c->ctx = ctx;
  c->cfg = *cfg;
  c->kind.assign(cfg->layer_kind, cfg->layer_kind + cfg->n_layers);
  c->cfg.layer_kind = c->kind.data();
  c->D = s.D;
  c->hq = s.hq;
  c->hkv = s.hkv;
  c->group = s.hq / s.hkv;
  c->heads_per_item = c->group > 1 ? 8 : 1;
  // what one more item costs a worker, in tiles: a query-group item fetches its query fragments when it
  // starts and leaves up to eight partial rows (measured on launches of one layer: 4 resp. 12 best,
  // with ranges of at least 6 resp. 4 tiles)
  c->static_row_cost = c->group > 1 ? 12 : 4;
  c->static_min_tiles = c->group > 1 ? 4 : 6;
  c->items_per_chunk = c->group > 1 ? s.hkv * ((c->group + 7) / 8) : s.hq;
  c->paged = cfg->page_size == 16;
  c->max_pages = s.max_pages;
  c->chunk_pages = c->min_chunk_pages = s.chunk_pages;
  c->auto_split = cfg->split_tokens == 0;
  c->max_slots = s.max_slots;
  c->slots_per_stream = s.slots_per_stream;
  c->n_pool_pages = s.n_pool_pages;
  c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt(static_cast<float>(s.D));
  c->ws = static_cast<uint8_t*>(workspace_dev);
  c->pool = static_cast<uint16_t*>(pool_dev);
  c->lay = s.lay;
  c->max_items = s.max_items;
  c->max_segs = s.max_segs;
  c->max_patches = s.max_patches;
  c->leader.resize(cfg->n_layers);
  c->layer_flags.resize(cfg->n_layers);
  int last = 0;
  c->text_streams_per_seq = 0;
  for (int l = 0; l < cfg->n_layers; ++l) {
    if (c->kind[l] == QC_LAYER_FULL) last = l;
    c->leader[l] = last;
    uint8_t f = 0;
    if (owns(c, l, QC_STREAM_K_TEXT)) f |= kLayerOwnsTextK;
    if (c->kind[l] == QC_LAYER_FULL) f |= kLayerWritesQCache;
    c->layer_flags[l] = f;
    c->text_streams_per_seq += 1 + (owns(c, l, QC_STREAM_K_TEXT) ? 1 : 0);
  }
  build_jobs(&c->cfg, c->jobs, c->block_jobs, c->block_layers);
  build_layer_jobs(&c->cfg, c->layer_jobs, c->layer_job_range);
  build_inorder_jobs(&c->cfg, c->inorder_jobs, c->inorder_job_range, c->inorder_extra_key);
  if (c->cfg.lazy_mode == QC_MODE_GLA) {
    // Eq. 5: every layer of a lazy block attends with the block's first layer's Q and K, so runs
    // of up to three of its layers share one score pass of the prefill kernel
    std::vector<PrefillPass> shared;
    for (const auto& bl : c->block_layers) {
      for (int first = bl.first; first < bl.second; first += kPrefillSharedLayers) {
        PrefillPass ps{};
        ps.n = std::min(kPrefillSharedLayers, bl.second - first);
        for (int x = 0; x < ps.n; ++x) ps.v[x] = first + x;
        (ps.n > 1 ? shared : c->prefill_passes).push_back(ps);
      }
    }
    c->prefill_n_single = static_cast<int>(c->prefill_passes.size());
    c->prefill_n_shared = static_cast<int>(shared.size());
    c->prefill_passes.insert(c->prefill_passes.end(), shared.begin(), shared.end());
  }
  c->seqs.resize(cfg->max_seqs);
  c->table.assign(static_cast<size_t>(cfg->n_layers) * 4 * cfg->max_seqs * c->max_pages, -1);
  if (c->paged) {
    c->free_stack.resize(s.n_pool_pages);
    for (int64_t i = 0; i < s.n_pool_pages; ++i) c->free_stack[i] = static_cast<int32_t>(s.n_pool_pages - 1 - i);
  } else {
    // contiguous: stream (layer, stream, seq) owns pages [extent*max_pages, (extent+1)*max_pages)
    for (size_t i = 0; i < c->table.size(); ++i) c->table[i] = static_cast<int32_t>(i);
  }

  // the pool's tensor map: needed by the query-group decode kernel; the prefill kernel uses it for
  // cached tiles when it exists
  c->pool_map_ok = make_pool_tensor_map(c) == QC_OK;
  if (c->group > 1 && !c->pool_map_ok) {
    delete c;
    return QC_ERR_CUDA;
  }

  cudaStream_t stream = ctx->stream;
  bool ok = cudaHostAlloc(reinterpret_cast<void**>(&c->pinned), kStageSlots * c->lay.step_bytes,
                          cudaHostAllocDefault) == cudaSuccess;
  for (int i = 0; ok && i < kStageSlots; ++i)
    ok = cudaEventCreateWithFlags(&c->stage_done[i], cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaHostAlloc(reinterpret_cast<void**>(&c->err_host), 64, cudaHostAllocMapped) == cudaSuccess;
  if (ok) {
    *c->err_host = 0;
    ok = cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->err_host_dev), c->err_host, 0) == cudaSuccess;
  }
  ok = ok && cudaMemcpyAsync(c->ws + c->lay.table, c->table.data(), c->table.size() * sizeof(int32_t),
                             cudaMemcpyHostToDevice, stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(c->ws + c->lay.layer_flags, c->layer_flags.data(), c->layer_flags.size(),
                             cudaMemcpyHostToDevice, stream) == cudaSuccess;
  std::vector<uint8_t> leader8(c->leader.begin(), c->leader.end());
  ok = ok && cudaMemcpyAsync(c->ws + c->lay.layer_kind, c->kind.data(), c->kind.size(), cudaMemcpyHostToDevice,
                             stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(c->ws + c->lay.leader, leader8.data(), leader8.size(), cudaMemcpyHostToDevice,
                             stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(c->ws + c->lay.jobs, c->jobs.data(), c->jobs.size() * sizeof(Job),
                             cudaMemcpyHostToDevice, stream) == cudaSuccess;
  ok = ok && cudaMemsetAsync(c->ws + c->lay.err, 0, 256, stream) == cudaSuccess;
  ok = ok && cudaMemsetAsync(c->ws + c->lay.row_done, 0, c->lay.wdesc - c->lay.row_done, stream) == cudaSuccess;
  ok = ok && cudaMemsetAsync(c->ws + c->lay.qcache, 0, c->lay.part_acc - c->lay.qcache, stream) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  if (!ok) {
    qc_free(nullptr, c);
    return QC_ERR_CUDA;
  }
  *out = c;
  return QC_OK;
}

int32_t qc_free(qc_ctx* ctx, qc_cache* cache) {
  if (cache) {
    if (cache->ctx) {
      cudaSetDevice(cache->ctx->device);
      cudaStreamSynchronize(cache->ctx->stream);
    }
    for (int i = 0; i < kStageSlots; ++i)
      if (cache->stage_done[i]) cudaEventDestroy(cache->stage_done[i]);
    for (cudaEvent_t e : cache->ev) cudaEventDestroy(e);
    for (cudaEvent_t e : cache->ev_launch) cudaEventDestroy(e);
    for (cudaEvent_t e : cache->ev_in) cudaEventDestroy(e);
    for (cudaEvent_t e : cache->ev_done) cudaEventDestroy(e);
    if (cache->copy_in) cudaStreamDestroy(cache->copy_in);
    if (cache->copy_out) cudaStreamDestroy(cache->copy_out);
    for (cudaEvent_t e : cache->ev_prefill) cudaEventDestroy(e);
    if (cache->pinned) cudaFreeHost(cache->pinned);
    if (cache->err_host) cudaFreeHost(cache->err_host);
    delete cache;
  }
  if (ctx) delete ctx;
  return QC_OK;
}

int32_t qc_prefill_append(qc_cache* c, int32_t n_seqs, const int32_t* seq_ids, const int32_t* n_tokens,
                          const uint8_t* kind, const void* k_dev, const void* v_dev) {
  if (!c || n_seqs < 0 || (n_seqs > 0 && (!seq_ids || !n_tokens))) return QC_ERR_INVALID_ARG;
  if (c->open.active) return QC_ERR_STATE;   // a decode step is open
  if (n_seqs == 0) return QC_OK;
  if (!k_dev || !v_dev) return QC_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k_dev) & 15) || (reinterpret_cast<uintptr_t>(v_dev) & 15)) return QC_ERR_INVALID_ARG;
  const int N = c->cfg.n_layers;
  // ---- validate and plan without touching the state
  int64_t total = 0, need = 0;
  std::vector<uint8_t> seen(c->cfg.max_seqs, 0);
  std::vector<int32_t> add_t(n_seqs), add_v(n_seqs);
  for (int i = 0; i < n_seqs; ++i) {
    const int s = seq_ids[i];
    if (s < 0 || s >= c->cfg.max_seqs || n_tokens[i] < 0) return QC_ERR_INVALID_ARG;
    if (seen[s]) return QC_ERR_STATE;
    seen[s] = 1;
    if (n_tokens[i] > 0 && !kind) return QC_ERR_INVALID_ARG;
    int nt = 0, nv = 0;
    for (int t = 0; t < n_tokens[i]; ++t) {
      const uint8_t kd = kind[total + t];
      if (kd == QC_KIND_TEXT) ++nt;
      else if (kd == QC_KIND_VISUAL) ++nv;
      else return QC_ERR_INVALID_ARG;
    }
    add_t[i] = nt;
    add_v[i] = nv;
    const SeqState& st = c->seqs[s];
    if (st.len_text + nt > c->cfg.max_tokens_per_seq || st.len_vis + nv > c->cfg.max_tokens_per_seq)
      return QC_ERR_INVALID_ARG;
    if (c->paged) {
      const int dt = pages_for(st.len_text + nt) - pages_for(st.len_text);
      const int dv = pages_for(st.len_vis + nv) - pages_for(st.len_vis);
      for (int l = 0; l < N; ++l)
        for (int stream = 0; stream < 4; ++stream)
          if (owns(c, l, stream)) need += (stream & 1) ? dv : dt;
    }
    total += n_tokens[i];
  }
  if (total > 0x7fffffffLL) return QC_ERR_INVALID_ARG;
  if (c->paged && need > static_cast<int64_t>(c->free_stack.size())) return QC_ERR_OOM_PAGES;
  QC_CUDA(cudaSetDevice(c->ctx->device));
  cudaStream_t stream = c->ctx->stream;

  // ---- commit: pages (sequence -> layer -> stream order), token routing
  std::vector<int32_t> tok_seq(total), tok_stream(total), tok_ord(total);
  int64_t t0 = 0;
  for (int i = 0; i < n_seqs; ++i) {
    const int s = seq_ids[i];
    SeqState& st = c->seqs[s];
    if (c->paged) {
      const int have_t = pages_for(st.len_text), have_v = pages_for(st.len_vis);
      const int dt = pages_for(st.len_text + add_t[i]) - have_t;
      const int dv = pages_for(st.len_vis + add_v[i]) - have_v;
      for (int l = 0; l < N; ++l)
        for (int sm = 0; sm < 4; ++sm)
          if (owns(c, l, sm)) grow_stream(c, l, sm, s, (sm & 1) ? have_v : have_t, (sm & 1) ? dv : dt, nullptr);
    }
    int ot = st.len_text, ov = st.len_vis;
    for (int t = 0; t < n_tokens[i]; ++t) {
      const bool vis = kind[t0 + t] == QC_KIND_VISUAL;
      tok_seq[t0 + t] = s;
      tok_stream[t0 + t] = vis ? 1 : 0;
      tok_ord[t0 + t] = vis ? ov++ : ot++;
    }
    st.len_text = ot;
    st.len_vis = ov;
    st.active = true;
    t0 += n_tokens[i];
  }
  // the whole host mirror goes to the device (prefill is not the hot path)
  if (c->paged)
    QC_CUDA(cudaMemcpyAsync(c->ws + c->lay.table, c->table.data(), c->table.size() * sizeof(int32_t),
                            cudaMemcpyHostToDevice, stream));
  Params p = base_params(c);
  p.k = static_cast<const uint16_t*>(k_dev);
  p.v = static_cast<const uint16_t*>(v_dev);
  int32_t* tok_dev = reinterpret_cast<int32_t*>(c->ws + c->lay.tok);
  for (int64_t off = 0; off < total; off += kPrefillBatchTokens) {
    const int n = static_cast<int>(std::min<int64_t>(kPrefillBatchTokens, total - off));
    QC_CUDA(cudaMemcpyAsync(tok_dev, tok_seq.data() + off, n * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
    QC_CUDA(cudaMemcpyAsync(tok_dev + kPrefillBatchTokens, tok_stream.data() + off, n * sizeof(int32_t),
                            cudaMemcpyHostToDevice, stream));
    QC_CUDA(cudaMemcpyAsync(tok_dev + 2 * kPrefillBatchTokens, tok_ord.data() + off, n * sizeof(int32_t),
                            cudaMemcpyHostToDevice, stream));
    c->kernel_launches++;
    QC_CUDA(launch_prefill_scatter(p, tok_dev, tok_dev + kPrefillBatchTokens, tok_dev + 2 * kPrefillBatchTokens, n,
                                   static_cast<int32_t>(total), static_cast<int32_t>(off), stream));
    // the host vectors and the device token arrays are reused by the next batch
    QC_CUDA(cudaStreamSynchronize(stream));
  }
  return QC_OK;
}

int32_t qc_prefill_attend(qc_cache* c, int32_t seq_id, int32_t n_tokens, const uint8_t* kind, const void* q_dev,
                          const void* k_dev, const void* v_dev, void* out_dev) {
  if (!c || n_tokens < 0 || seq_id < 0 || seq_id >= c->cfg.max_seqs) return QC_ERR_INVALID_ARG;
  if (n_tokens == 0) return QC_OK;
  if (!kind || !q_dev || !k_dev || !v_dev || !out_dev) return QC_ERR_INVALID_ARG;
  const void* ptrs[4] = {q_dev, k_dev, v_dev, out_dev};
  for (const void* ptr : ptrs)
    if (reinterpret_cast<uintptr_t>(ptr) & 15) return QC_ERR_INVALID_ARG;
  // tokens the sequence holds already (an earlier prompt chunk, generated tokens) precede the new ones
  const int n0_text = c->seqs[seq_id].active ? c->seqs[seq_id].len_text : 0;
  const int n0_vis = c->seqs[seq_id].active ? c->seqs[seq_id].len_vis : 0;
  const size_t tok_bytes = static_cast<size_t>(kPrefillBatchTokens) * 3 * sizeof(int32_t);   // kinds, tile codes, passes
  if (align_up(n_tokens, 256) + align_up((n_tokens + 63) / 64, 256) + c->prefill_passes.size() * sizeof(PrefillPass) >
      tok_bytes)
    return QC_ERR_INVALID_ARG;
  // what can fail without touching the cache comes first: the tensor maps over the caller's tensors
  PrefillMaps maps;
  const bool tc5 = c->prefill_tcgen05 && c->D == 128 && (c->pool_map_ok || n0_text + n0_vis == 0);
  if (tc5) {
    if (make_prompt_tensor_map(&maps.q, q_dev, c->cfg.n_layers, n_tokens, c->hq) != QC_OK ||
        make_prompt_tensor_map(&maps.k, k_dev, c->cfg.n_layers, n_tokens, c->hkv) != QC_OK ||
        make_prompt_tensor_map(&maps.v, v_dev, c->cfg.n_layers, n_tokens, c->hkv) != QC_OK ||
        make_output_tensor_map(&maps.out, out_dev, c->cfg.n_layers, n_tokens, c->hq) != QC_OK)
      return QC_ERR_CUDA;
  }
  // store K/V: this validates the rest and leaves the cache unchanged on an error
  int st = qc_prefill_append(c, 1, &seq_id, &n_tokens, kind, k_dev, v_dev);
  if (st != QC_OK) return st;
  cudaStream_t stream = c->ctx->stream;
  uint8_t* kind_dev = c->ws + c->lay.tok;   // free again: qc_prefill_append has waited for its copies
  // per 64-token tile: all text, all visual or mixed (the tcgen05 kernel fetches unmixed tiles whole)
  const int n_tiles = (n_tokens + 63) / 64;
  std::vector<uint8_t> codes(n_tiles);
  for (int i = 0; i < n_tiles; ++i) {
    int nv = 0, n = std::min(64, n_tokens - 64 * i);
    for (int t = 0; t < n; ++t) nv += kind[64 * i + t] == QC_KIND_VISUAL;
    codes[i] = nv == 0 ? 0 : (nv == n ? 1 : 2);
  }
  uint8_t* codes_dev = kind_dev + align_up(n_tokens, 256);
  QC_CUDA(cudaMemcpyAsync(kind_dev, kind, n_tokens, cudaMemcpyHostToDevice, stream));
  QC_CUDA(cudaMemcpyAsync(codes_dev, codes.data(), n_tiles, cudaMemcpyHostToDevice, stream));
  PrefillPass* passes_dev = reinterpret_cast<PrefillPass*>(codes_dev + align_up(n_tiles, 256));
  const bool share = c->prefill_n_shared > 0 && n0_text + n0_vis == 0 &&
                     (c->prefill_shared == 2 || (c->prefill_shared == 1 && n_tokens >= kPrefillShareMinTokens));
  if (share)
    QC_CUDA(cudaMemcpyAsync(passes_dev, c->prefill_passes.data(), c->prefill_passes.size() * sizeof(PrefillPass),
                            cudaMemcpyHostToDevice, stream));
  QC_CUDA(cudaStreamSynchronize(stream));   // `kind` is the caller's host memory
  const Params p = base_params(c);
  cudaEvent_t* ev = nullptr;
  if (c->profile && c->ev_prefill_calls < kMaxProfileSteps) {
    if (static_cast<int>(c->ev_prefill.size()) < 2 * (c->ev_prefill_calls + 1)) {
      for (int i = 0; i < 2; ++i) {
        cudaEvent_t e;
        QC_CUDA(cudaEventCreate(&e));
        c->ev_prefill.push_back(e);
      }
    }
    ev = &c->ev_prefill[2 * c->ev_prefill_calls];
    QC_CUDA(cudaEventRecord(ev[0], stream));
  }
  QC_CUDA(launch_prefill_attend(p, kind_dev, c->ws + c->lay.layer_kind, c->ws + c->lay.leader, q_dev, k_dev, v_dev,
                                out_dev, n_tokens, c->cfg.lazy_mode == QC_MODE_GLA ? 1 : 0, tc5 ? &maps : nullptr,
                                codes_dev, seq_id, n0_text, n0_vis, (tc5 && share) ? passes_dev : nullptr,
                                c->prefill_n_single, c->prefill_n_shared, c->prefill_pair_min_tokens, stream));
  const bool shared_run = tc5 && share;
  if (ev) {
    QC_CUDA(cudaEventRecord(ev[1], stream));
    c->ev_prefill_calls++;
    // executed arithmetic: 2 D flops per pair for the scores of every score pass, 2 D per pair for
    // the value product of every layer
    const double pairs = 0.5 * n_tokens * (n_tokens + 1.0) + static_cast<double>(n_tokens) * (n0_text + n0_vis);
    const int score_passes = shared_run ? c->prefill_n_single + c->prefill_n_shared : c->cfg.n_layers;
    c->prof_prefill_flops += 2.0 * c->D * pairs * c->hq * (score_passes + c->cfg.n_layers);
  }
  c->kernel_launches += (shared_run && c->prefill_n_single > 0) ? 2 : 1;
  return QC_OK;
}

int32_t qc_layer_similarity(qc_cache* c, int32_t n_seqs, const int32_t* seq_ids, const void* q_dev, float* rows_dev,
                            int32_t max_len, float* similarity_host) {
  if (!c || n_seqs < 1 || n_seqs > c->cfg.max_seqs || !seq_ids || !q_dev || !rows_dev || !similarity_host)
    return QC_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q_dev) & 15) || (reinterpret_cast<uintptr_t>(rows_dev) & 15)) return QC_ERR_INVALID_ARG;
  if (max_len < 1 || max_len > 12288) return QC_ERR_UNSUPPORTED;   // one head's logits live in shared memory
  const int N = c->cfg.n_layers;
  for (int l = 0; l < N; ++l)
    if (c->kind[l] != QC_LAYER_FULL) return QC_ERR_STATE;          // the analysis runs on the unmodified stack
  std::vector<int32_t> host(3 * static_cast<size_t>(n_seqs));
  for (int i = 0; i < n_seqs; ++i) {
    const int s = seq_ids[i];
    if (s < 0 || s >= c->cfg.max_seqs) return QC_ERR_INVALID_ARG;
    const SeqState& st = c->seqs[s];
    if (!st.active || st.len_text + st.len_vis == 0) return QC_ERR_STATE;
    if (st.len_text + st.len_vis > max_len) return QC_ERR_INVALID_ARG;
    host[i] = s;
    host[n_seqs + i] = st.len_text;
    host[2 * n_seqs + i] = st.len_vis;
  }
  QC_CUDA(cudaSetDevice(c->ctx->device));
  cudaStream_t stream = c->ctx->stream;
  int32_t* ids_dev = reinterpret_cast<int32_t*>(c->ws + c->lay.tok);
  float* js_dev = reinterpret_cast<float*>(c->ws + c->lay.stage_lse);   // (n_layers - 1) * n_seqs floats fit
  QC_CUDA(cudaMemcpyAsync(ids_dev, host.data(), host.size() * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
  Params p = base_params(c);
  p.q = static_cast<const uint16_t*>(q_dev);
  p.n_seqs = n_seqs;
  QC_CUDA(launch_calibration(p, ids_dev, ids_dev + n_seqs, ids_dev + 2 * n_seqs, rows_dev, max_len, js_dev, stream));
  c->kernel_launches += N > 1 ? 2 : 1;
  std::vector<float> js(static_cast<size_t>(std::max(0, N - 1)) * n_seqs);
  if (!js.empty())
    QC_CUDA(cudaMemcpyAsync(js.data(), js_dev, js.size() * sizeof(float), cudaMemcpyDeviceToHost, stream));
  QC_CUDA(cudaStreamSynchronize(stream));
  for (int l = 0; l + 1 < N; ++l) {
    double acc = 0.0;
    for (int i = 0; i < n_seqs; ++i) acc += js[static_cast<size_t>(l) * n_seqs + i];
    similarity_host[l] = static_cast<float>(acc / n_seqs);
  }
  return QC_OK;
}

int32_t qc_lazy_blocks(const float* similarity, int32_t n_layers, float eps, int32_t max_block, uint8_t* layer_kind) {
  if (n_layers < 1 || !layer_kind || (n_layers > 1 && !similarity) || !(eps > 0.f) || eps > 1.f)
    return QC_ERR_INVALID_ARG;
  layer_kind[0] = QC_LAYER_FULL;
  int size = 1;
  for (int l = 1; l < n_layers; ++l) {
    if (similarity[l - 1] < eps && (max_block <= 0 || size < max_block)) {
      layer_kind[l] = QC_LAYER_LAZY;
      ++size;
    } else {
      layer_kind[l] = QC_LAYER_FULL;
      size = 1;
    }
  }
  return QC_OK;
}

}  // extern "C"

namespace {

// Events of the host-buffer entry point: launch group g waits for in[g] (its inputs have been
// copied) and records done[g] (its outputs may be copied back).
struct HostPipe {
  int per_launch;
  cudaEvent_t* in;
  cudaEvent_t* done;
};

// One attention launch of a step (group gi of the launch plan) with its merge; optionally the
// append of the group's layers first (host-buffer entry point, per-layer entry point).
int run_group(qc_cache* c, Params& p, size_t gi, const LaunchList& launches, bool use_static, int64_t tot_v,
              int64_t tot_t, bool append_first, cudaEvent_t wait_in, cudaEvent_t record_done, cudaEvent_t* ev,
              cudaStream_t stream) {
  const int pb = c->group_pos[gi].first, pe = c->group_pos[gi].second;
  p.item_begin = static_cast<int32_t>(c->plan_vis_before[pb] * tot_v + c->plan_text_before[pb] * tot_t);
  p.item_end = static_cast<int32_t>(c->plan_vis_before[pe] * tot_v + c->plan_text_before[pe] * tot_t);
  p.layer_begin = c->groups[gi].layer_begin;
  p.layer_end = c->groups[gi].layer_end;
  p.launch_index = static_cast<int32_t>(gi);
  p.pos_begin = pb;
  p.pos_end = pe;
  p.extra_key_leader = c->groups[gi].extra_key_leader;
  bool has_work = p.item_end > p.item_begin;
  if (use_static) {   // (a step has at most n_layers <= 127 launches: every one has its entry)
    const LaunchDesc& one = launches.launch[gi];
    has_work = one.part_workers > 0;
    p.part_q = one.part_q;
    p.part_k = one.part_k;
    p.part_vw = one.part_vw;
    p.part_workers = one.part_workers;
    p.part_row_cost = one.part_row_cost;
    p.merge_wide = one.merge_wide;
    p.part_tiles = 0;
  }
  if (wait_in) QC_CUDA(cudaStreamWaitEvent(stream, wait_in, 0));
  if (append_first) {
    QC_CUDA(launch_append(p, stream));   // this group's layers only
    c->kernel_launches++;
  }
  if (ev && gi == 0) QC_CUDA(cudaEventRecord(ev[1], stream));
  cudaEvent_t* evl = nullptr;
  if (ev && c->profile == 2 && has_work && c->ev_launches < 64 * kMaxProfileSteps) {
    if (static_cast<int>(c->ev_launch.size()) < 2 * (c->ev_launches + 1)) {
      for (int i = 0; i < 2; ++i) {
        cudaEvent_t e;
        QC_CUDA(cudaEventCreate(&e));
        c->ev_launch.push_back(e);
      }
    }
    evl = &c->ev_launch[2 * c->ev_launches++];
    QC_CUDA(cudaEventRecord(evl[0], stream));
  }
  if (!has_work) {
    // (a GLA follower of the in-order schedule: its merge does everything)
  } else if (c->group > 1) {
    QC_CUDA(launch_attend_tc(p, c->ctx->n_sms, stream));
  } else {
    QC_CUDA(launch_attend(p, c->ctx->n_sms, stream));
  }
  if (evl) QC_CUDA(cudaEventRecord(evl[1], stream));
  if (ev && gi + 1 == c->groups.size()) QC_CUDA(cudaEventRecord(ev[2], stream));
  if (c->groups[gi].needs_merge) QC_CUDA(launch_merge(p, stream));
  if (record_done) QC_CUDA(cudaEventRecord(record_done, stream));
  c->attend_launches += has_work ? 1 : 0;
  c->kernel_launches += (has_work ? 1 : 0) + (c->groups[gi].needs_merge ? 1 : 0);
  return QC_OK;
}

int decode_step_core(qc_cache* c, int32_t n_seqs, const int32_t* seq_ids, const void* q_dev, const void* k_dev,
                     const void* v_dev, void* out_dev, float* lse_out_dev, const HostPipe* pipe,
                     bool open_only = false) {
  if (!c || n_seqs < 0 || (n_seqs > 0 && !seq_ids)) return QC_ERR_INVALID_ARG;
  if (c->open.active) return QC_ERR_STATE;   // a step opened by qc_decode_begin has layers left
  if (n_seqs == 0) return open_only ? QC_ERR_INVALID_ARG : QC_OK;
  if (!open_only && (!q_dev || !k_dev || !v_dev || !out_dev)) return QC_ERR_INVALID_ARG;
  if (n_seqs > c->cfg.max_seqs) return QC_ERR_INVALID_ARG;
  const void* ptrs[4] = {q_dev, k_dev, v_dev, out_dev};
  for (const void* ptr : ptrs)
    if (reinterpret_cast<uintptr_t>(ptr) & 15) return QC_ERR_INVALID_ARG;
  if (const int32_t dev_err = *static_cast<volatile int32_t*>(c->err_host)) return dev_err;   // an earlier kernel gave up
  const int N = c->cfg.n_layers;
  // ---- validate, count pages
  int64_t need = 0;
  {
    std::vector<uint8_t> seen(c->cfg.max_seqs, 0);
    for (int i = 0; i < n_seqs; ++i) {
      const int s = seq_ids[i];
      if (s < 0 || s >= c->cfg.max_seqs) return QC_ERR_INVALID_ARG;
      if (!c->seqs[s].active || seen[s]) return QC_ERR_STATE;
      seen[s] = 1;
      if (c->seqs[s].len_text + 1 > c->cfg.max_tokens_per_seq) return QC_ERR_INVALID_ARG;
      if (c->paged && c->seqs[s].len_text % kPage == 0) need += c->text_streams_per_seq;
    }
  }
  if (c->paged && need > static_cast<int64_t>(c->free_stack.size())) return QC_ERR_OOM_PAGES;
  QC_CUDA(cudaSetDevice(c->ctx->device));
  cudaStream_t stream = c->ctx->stream;

  const int want_per = open_only ? -2 : (pipe ? pipe->per_launch : c->layers_per_launch);
  if (c->plan_dirty || c->plan_per != want_per) {
    const int st = rebuild_plan(c, want_per);
    if (st != QC_OK) return st;
  }

  // ---- page planning (sequence -> layer -> K_T, V_T) and lengths
  std::vector<Patch> patches;
  for (int i = 0; i < n_seqs; ++i) {
    const int s = seq_ids[i];
    SeqState& st = c->seqs[s];
    if (c->paged && st.len_text % kPage == 0) {
      const int have = st.len_text / kPage;
      for (int l = 0; l < N; ++l) {
        if (owns(c, l, QC_STREAM_K_TEXT)) grow_stream(c, l, QC_STREAM_K_TEXT, s, have, 1, &patches);
        grow_stream(c, l, QC_STREAM_V_TEXT, s, have, 1, &patches);
      }
    }
    st.len_text += 1;
  }
  const int n_patches = static_cast<int>(patches.size());
  if (c->auto_split) {
    // Larger chunks mean fewer partial results to write and merge; smaller chunks mean more
    // work items to balance over the workers.  Take the largest chunk that still leaves
    // every worker several items per launch: five when the step is one launch, one and a half
    // when it is one launch per layer (a short launch's partial rows and their merge weigh more
    // than the balance of its tail; 1, 2 and 3 were measured too).  With several launches per
    // step, a long stream cut small also means many partial rows per output row for every one of
    // those launches' merges: beyond 24 rows the chunk is doubled as long as one and a half items
    // per worker remain.
    const int64_t workers = static_cast<int64_t>(c->ctx->n_sms) * kAttendWarps * static_cast<int64_t>(c->groups.size());
    auto items_at = [&](int cp, int* max_slots) {
      int64_t cv = 0, ct = 0;
      int slots = 0;
      for (int i = 0; i < n_seqs; ++i) {
        const SeqState& st = c->seqs[seq_ids[i]];
        const int v = (pages_for(st.len_vis) + cp - 1) / cp, t = (pages_for(st.len_text) + cp - 1) / cp;
        cv += v;
        ct += t;
        slots = std::max(slots, v + t);
      }
      if (max_slots) *max_slots = slots;
      return (cv * c->n_visual_jobs + ct * c->n_text_jobs) * c->items_per_chunk;
    };
    const int64_t twice_per_worker = c->plan_per < 0 ? 3 : 10;
    // (a query group writes one partial row per head and chunk: its chunks stay at 128 keys or more)
    const int floor_pages = c->group > 1 ? std::max(c->min_chunk_pages, 8) : c->min_chunk_pages;
    int pick = floor_pages;
    for (int cp = kMaxChunkPages; cp > floor_pages; cp /= 2) {
      if (2 * items_at(cp, nullptr) >= twice_per_worker * workers) {
        pick = cp;
        break;
      }
    }
    if (c->groups.size() > 1) {
      int slots = 0;
      items_at(pick, &slots);
      while (slots > 24 && pick * 2 <= kMaxChunkPages && 2 * items_at(pick * 2, nullptr) >= 3 * workers) {
        pick *= 2;
        items_at(pick, &slots);
      }
    }
    c->chunk_pages = pick;
  }

  // ---- step descriptors: as a kernel argument when they are small and no page table entry
  // changes, otherwise through a pinned slot and one copy
  const bool inline_step = n_seqs <= kInlineSeqs && n_patches == 0;
  StepInline inl;
  StepSeq* h_seqs = inl.seqs;
  int slot = -1;
  uint8_t* hb = nullptr;
  if (!inline_step) {
    slot = c->stage_next;
    c->stage_next = (c->stage_next + 1) % kStageSlots;
    if (c->stage_used[slot]) QC_CUDA(cudaEventSynchronize(c->stage_done[slot]));   // its last copy must have run
    hb = c->pinned + static_cast<size_t>(slot) * c->lay.step_bytes;
    h_seqs = reinterpret_cast<StepSeq*>(hb + c->lay.step_seqs);
    if (n_patches) std::memcpy(hb + c->lay.step_patches, patches.data(), n_patches * sizeof(Patch));
  }
  // Static partition: the step's launches cut their work into equal ranges instead of claiming
  // items (by default whenever a step is several launches, whose short tails a few large items
  // per worker would dominate).
  bool use_static = c->static_partition == 1 || (c->static_partition < 0 && c->groups.size() > 1);
  int64_t tp_v = 0, tp_t = 0;                     // pages of the visual / text streams over the listed sequences
  int pmax_v = 0, pmax_t = 0;
  for (int i = 0; i < n_seqs; ++i) {
    const SeqState& st = c->seqs[seq_ids[i]];
    const int pv = pages_for(st.len_vis), pt = pages_for(st.len_text);
    tp_v += pv;
    tp_t += pt;
    pmax_v = std::max(pmax_v, pv);
    pmax_t = std::max(pmax_t, pt);
  }
  // Static ranges pay off for launches that leave a worker one or two ranges' worth of tiles (a
  // launch per layer or per lazy block); on larger launches claimed 512-key items were measured
  // faster (config 2, five blocks per launch: 0.89 against 1.05 ms per step; two blocks: 1.04
  // against 1.12).  Tile offsets are 32-bit.
  if (c->static_partition < 0) {
    const int64_t workers = static_cast<int64_t>(c->ctx->n_sms) * kAttendWarps;
    for (const LaunchGroup& g : c->groups) {
      const int64_t tiles = static_cast<int64_t>(c->items_per_chunk) * (g.wv * tp_v + g.wt * tp_t);
      if (tiles > workers * 60 * std::max(1, g.w_min)) use_static = false;
    }
  }
  for (const LaunchGroup& g : c->groups)
    if (static_cast<int64_t>(c->items_per_chunk) * (g.wv * tp_v + g.wt * tp_t + 64LL * n_seqs * (g.job_end - g.job_begin)) >= (1LL << 31))
      use_static = false;
  int64_t tot_v = 0, tot_t = 0, step_rows = 0;   // step_rows: K/V rows the step has to read (for the profile)
  int64_t pre_pv = 0, pre_pt = 0;
  for (int i = 0; i < n_seqs; ++i) {
    const int s = seq_ids[i];
    const SeqState& st = c->seqs[s];
    const int pv = pages_for(st.len_vis), pt = pages_for(st.len_text);
    const int ncv = (pv + c->chunk_pages - 1) / c->chunk_pages;
    const int nct = (pt + c->chunk_pages - 1) / c->chunk_pages;
    h_seqs[i] = StepSeq{s, st.len_text, st.len_vis, ncv + nct, static_cast<int32_t>(use_static ? pre_pv : tot_v),
                        static_cast<int32_t>(use_static ? pre_pt : tot_t), ncv, 0};
    tot_v += static_cast<int64_t>(ncv) * c->items_per_chunk;
    tot_t += static_cast<int64_t>(nct) * c->items_per_chunk;
    pre_pv += pv;
    pre_pt += pt;
    step_rows += st.len_vis * c->visual_row_reads + st.len_text * c->text_row_reads;
  }
  const int n_pos = static_cast<int>(c->plan.size());
  const int64_t n_items64 = c->plan_vis_before[n_pos] * tot_v + c->plan_text_before[n_pos] * tot_t;
  const int n_items = use_static ? 0 : static_cast<int>(n_items64);   // <= max_items: the item list was sized at allocation

  // ---- enqueue
  if (!inline_step) {
    QC_CUDA(cudaMemcpyAsync(c->ws + c->lay.step, hb, c->lay.step_bytes, cudaMemcpyHostToDevice, stream));
    QC_CUDA(cudaEventRecord(c->stage_done[slot], stream));
    c->stage_used[slot] = true;
  }

  Params p = base_params(c);
  p.q = static_cast<const uint16_t*>(q_dev);
  p.k = static_cast<const uint16_t*>(k_dev);
  p.v = static_cast<const uint16_t*>(v_dev);
  p.out = static_cast<uint16_t*>(out_dev);
  p.lse = lse_out_dev;
  p.n_seqs = n_seqs;
  p.n_pos = use_static ? 0 : n_pos;   // static ranges need no item list
  p.n_items = n_items;
  p.part_static = use_static ? 1 : 0;
  p.tp_v = static_cast<int32_t>(tp_v);
  p.tp_t = static_cast<int32_t>(tp_t);
  p.n_patches = n_patches;
  p.tot_v = static_cast<int32_t>(tot_v);
  p.tot_t = static_cast<int32_t>(tot_t);
  p.inline_seqs = inline_step ? 1 : 0;
  // the append reads the page table (not beside its patches) and every layer's k/v (not before
  // the host pipe has copied them)
  // in-order schedule: nothing of a layer is touched before its own launch (the worker that meets
  // the end of the layer's text stream takes the new rows from the inputs and stores them)
  const bool fold = want_per == -2 && c->fold_append;
  p.fold_append = fold ? 1 : 0;
  p.fused_append = (n_patches == 0 && !pipe && !open_only && !fold) ? 1 : 0;

  // static partition of every launch of the step (part_workers == 0: the launch has nothing to sweep)
  auto partition_of = [&](size_t gi) {
    const LaunchGroup& g = c->groups[gi];
    const int pb = c->group_pos[gi].first, pe = c->group_pos[gi].second;
    LaunchDesc L{};
    L.pos_begin = pb;
    L.pos_end = pe;
    L.part_row_cost = c->static_row_cost;
    const int64_t kv_tiles = static_cast<int64_t>(c->items_per_chunk) * (g.wv * tp_v + g.wt * tp_t);
    if (kv_tiles <= 0) return L;
    const int64_t T = kv_tiles + static_cast<int64_t>(c->items_per_chunk) * c->static_row_cost * n_seqs * (pe - pb);
    // tiles per page of the lightest / heaviest job that has any page, longest row in tiles
    const int w_min = (tp_v > 0 && tp_t > 0) ? g.w_min : g.w_max_v * (tp_v > 0) + g.w_max_t * (tp_t > 0);
    const int w_lo = std::max(1, std::min(w_min, g.w_min));
    const int64_t row_max = std::max<int64_t>(static_cast<int64_t>(pmax_v) * g.w_max_v,
                                              static_cast<int64_t>(pmax_t) * g.w_max_t);
    const int64_t q_max = 30LL * w_lo;
    int64_t q_min = std::max<int64_t>(2LL * g.w_max, (row_max + c->slots_per_stream - 3) / (c->slots_per_stream - 2));
    q_min = std::max<int64_t>(q_min, std::min<int64_t>(c->static_min_tiles, q_max / 2));
    const int64_t W = static_cast<int64_t>(c->ctx->n_sms) * kAttendWarps;
    int64_t k = 1, q;
    if (T > W * q_max) {   // several ranges per worker, each as long as a piece may be
      k = (T + W * q_max - 1) / (W * q_max);
      q = (T + W * k - 1) / (W * k);
    } else {
      q = std::max<int64_t>(q_min, (T + W - 1) / W);
    }
    const int64_t vw = (T + q - 1) / q;
    L.part_vw = static_cast<int32_t>(vw);
    L.part_k = static_cast<int32_t>(k);
    L.part_workers = static_cast<int32_t>((vw + k - 1) / k);
    L.part_q = static_cast<int32_t>(q);
    L.merge_wide = (static_cast<int64_t>(pmax_v) * g.w_max_v + q - 1) / q + 1 > 4 ? 1 : 0;
    return L;
  };
  LaunchList launches;
  const bool planned = use_static && c->plan_ahead && c->groups.size() <= static_cast<size_t>(kMaxPlanLaunches) &&
                       c->groups.size() <= static_cast<size_t>(std::min(c->cfg.n_layers, kMaxPlanLaunches)) &&
                       c->ctx->n_sms * kAttendWarps <= kPlanWorkers;
  if (use_static)
    for (size_t gi = 0; gi < c->groups.size() && gi < static_cast<size_t>(kMaxPlanLaunches); ++gi)
      launches.launch[gi] = partition_of(gi);
  p.wdesc = planned ? reinterpret_cast<const WorkerDesc*>(c->ws + c->lay.wdesc) : nullptr;

  cudaEvent_t* ev = nullptr;
  if (c->profile && !open_only && c->ev_steps < kMaxProfileSteps) {
    if (static_cast<int>(c->ev.size()) < 4 * (c->ev_steps + 1)) {
      for (int i = 0; i < 4; ++i) {
        cudaEvent_t e;
        QC_CUDA(cudaEventCreate(&e));
        c->ev.push_back(e);
      }
    }
    ev = &c->ev[4 * c->ev_steps];
    QC_CUDA(cudaEventRecord(ev[0], stream));
  }
  QC_CUDA(launch_setup(p, inline_step ? &inl : nullptr, stream));
  c->kernel_launches++;
  if (!p.fused_append && !pipe && !open_only && !fold) {
    p.layer_begin = 0;
    p.layer_end = N;
    QC_CUDA(launch_append(p, stream));
    c->kernel_launches++;
  }
  if (planned) {
    QC_CUDA(launch_plan(p, launches, static_cast<int>(c->groups.size()), stream));
    c->kernel_launches++;
  }
  if (open_only) {   // qc_decode_begin: the launches follow layer by layer (qc_decode_layer)
    OpenStep& o = c->open;
    o.p = p;
    o.launches = launches;
    o.use_static = use_static;
    o.tot_v = tot_v;
    o.tot_t = tot_t;
    o.next_layer = 0;
    o.bytes = step_rows * c->hkv * c->D * 2;
    o.active = true;
    return QC_OK;
  }
  for (size_t gi = 0; gi < c->groups.size(); ++gi) {
    const int st = run_group(c, p, gi, launches, use_static, tot_v, tot_t, pipe != nullptr,
                             pipe ? pipe->in[gi] : nullptr, pipe ? pipe->done[gi] : nullptr, ev, stream);
    if (st != QC_OK) return st;
  }
  if (ev) {
    QC_CUDA(cudaEventRecord(ev[3], stream));
    c->ev_steps++;
    c->prof_bytes += step_rows * c->hkv * c->D * 2;
    c->prof_items += n_items;
  }
  c->decode_steps++;
  c->kv_bytes_swept += step_rows * c->hkv * c->D * 2;
  return QC_OK;
}

}  // namespace

extern "C" {

int32_t qc_decode_step(qc_cache* c, int32_t n_seqs, const int32_t* seq_ids, const void* q_dev, const void* k_dev,
                       const void* v_dev, void* out_dev, float* lse_out_dev) {
  return decode_step_core(c, n_seqs, seq_ids, q_dev, k_dev, v_dev, out_dev, lse_out_dev, nullptr);
}

int32_t qc_decode_begin(qc_cache* c, int32_t n_seqs, const int32_t* seq_ids) {
  return decode_step_core(c, n_seqs, seq_ids, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, true);
}

int32_t qc_decode_layer(qc_cache* c, int32_t layer, const void* q_dev, const void* k_dev, const void* v_dev,
                        void* out_dev, float* lse_out_dev) {
  if (!c || !q_dev || !k_dev || !v_dev || !out_dev) return QC_ERR_INVALID_ARG;
  const void* ptrs[4] = {q_dev, k_dev, v_dev, out_dev};
  for (const void* ptr : ptrs)
    if (reinterpret_cast<uintptr_t>(ptr) & 15) return QC_ERR_INVALID_ARG;
  OpenStep& o = c->open;
  if (!o.active || layer != o.next_layer) return QC_ERR_STATE;
  if (const int32_t dev_err = *static_cast<volatile int32_t*>(c->err_host)) return dev_err;
  QC_CUDA(cudaSetDevice(c->ctx->device));
  // the kernels index a step's tensors as [layer][sequence]...: hand them this layer's slices at that place
  Params p = o.p;
  const uintptr_t q_off = static_cast<uintptr_t>(layer) * p.n_seqs * c->hq * c->D * 2;
  const uintptr_t kv_off = static_cast<uintptr_t>(layer) * p.n_seqs * c->hkv * c->D * 2;
  p.q = reinterpret_cast<const uint16_t*>(reinterpret_cast<uintptr_t>(q_dev) - q_off);
  p.k = reinterpret_cast<const uint16_t*>(reinterpret_cast<uintptr_t>(k_dev) - kv_off);
  p.v = reinterpret_cast<const uint16_t*>(reinterpret_cast<uintptr_t>(v_dev) - kv_off);
  p.out = reinterpret_cast<uint16_t*>(reinterpret_cast<uintptr_t>(out_dev) - q_off);
  p.lse = lse_out_dev ? reinterpret_cast<float*>(reinterpret_cast<uintptr_t>(lse_out_dev) -
                                                  static_cast<uintptr_t>(layer) * p.n_seqs * c->hq * sizeof(float))
                      : nullptr;
  const int st = run_group(c, p, static_cast<size_t>(layer), o.launches, o.use_static, o.tot_v, o.tot_t,
                           !p.fold_append, nullptr, nullptr, nullptr, c->ctx->stream);
  if (st != QC_OK) return st;
  if (++o.next_layer == c->cfg.n_layers) {
    o.active = false;
    c->decode_steps++;
    c->kv_bytes_swept += o.bytes;
  }
  return QC_OK;
}

int32_t qc_decode_step_host(qc_cache* c, int32_t n_seqs, const int32_t* seq_ids, const void* q_host,
                            const void* k_host, const void* v_host, void* out_host, float* lse_out_host) {
  if (!c || n_seqs < 0) return QC_ERR_INVALID_ARG;
  if (n_seqs == 0) return QC_OK;
  if (!q_host || !k_host || !v_host || !out_host || n_seqs > c->cfg.max_seqs) return QC_ERR_INVALID_ARG;
  QC_CUDA(cudaSetDevice(c->ctx->device));
  cudaStream_t stream = c->ctx->stream;
  // The step runs as up to four launch groups of consecutive lazy blocks: while one group
  // computes, the inputs of the next are copied in and the outputs of the previous copied out.
  // (a small step is not worth cutting up: one group)
  const int nb = static_cast<int>(c->block_jobs.size());
  const size_t in_bytes = static_cast<size_t>(c->cfg.n_layers) * n_seqs * (c->hq + 2 * c->hkv) * c->D * 2;
  const int per = in_bytes < (1u << 20) ? nb : (nb + 3) / 4;
  if (c->plan_dirty || c->plan_per != per) {
    const int st = rebuild_plan(c, per);
    if (st != QC_OK) return st;
  }
  const size_t G = c->groups.size();
  if (!c->copy_in) {
    QC_CUDA(cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking));
    QC_CUDA(cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking));
  }
  while (c->ev_in.size() < G) {
    cudaEvent_t a, b;
    QC_CUDA(cudaEventCreateWithFlags(&a, cudaEventDisableTiming));
    QC_CUDA(cudaEventCreateWithFlags(&b, cudaEventDisableTiming));
    c->ev_in.push_back(a);
    c->ev_done.push_back(b);
  }
  const size_t q_layer = static_cast<size_t>(n_seqs) * c->hq * c->D * 2;    // bytes of one layer's q (and out)
  const size_t kv_layer = static_cast<size_t>(n_seqs) * c->hkv * c->D * 2;
  const size_t lse_layer = static_cast<size_t>(n_seqs) * c->hq * sizeof(float);
  uint8_t* dq = c->ws + c->lay.stage_q;
  uint8_t* dk = c->ws + c->lay.stage_k;
  uint8_t* dv = c->ws + c->lay.stage_v;
  uint8_t* dout = c->ws + c->lay.stage_out;
  uint8_t* dlse = c->ws + c->lay.stage_lse;
  const uint8_t* hq = static_cast<const uint8_t*>(q_host);
  const uint8_t* hk = static_cast<const uint8_t*>(k_host);
  const uint8_t* hv = static_cast<const uint8_t*>(v_host);
  for (size_t g = 0; g < G; ++g) {
    const size_t lb = c->groups[g].layer_begin, nl = c->groups[g].layer_end - lb;
    QC_CUDA(cudaMemcpyAsync(dq + lb * q_layer, hq + lb * q_layer, nl * q_layer, cudaMemcpyHostToDevice, c->copy_in));
    QC_CUDA(cudaMemcpyAsync(dk + lb * kv_layer, hk + lb * kv_layer, nl * kv_layer, cudaMemcpyHostToDevice, c->copy_in));
    QC_CUDA(cudaMemcpyAsync(dv + lb * kv_layer, hv + lb * kv_layer, nl * kv_layer, cudaMemcpyHostToDevice, c->copy_in));
    QC_CUDA(cudaEventRecord(c->ev_in[g], c->copy_in));
  }
  const HostPipe pipe{per, c->ev_in.data(), c->ev_done.data()};
  const int st = decode_step_core(c, n_seqs, seq_ids, dq, dk, dv, dout,
                                  lse_out_host ? reinterpret_cast<float*>(dlse) : nullptr, &pipe);
  if (st != QC_OK) {
    cudaStreamSynchronize(c->copy_in);
    cudaStreamSynchronize(stream);
    return st;
  }
  for (size_t g = 0; g < G; ++g) {
    const size_t lb = c->groups[g].layer_begin, nl = c->groups[g].layer_end - lb;
    QC_CUDA(cudaStreamWaitEvent(c->copy_out, c->ev_done[g], 0));
    QC_CUDA(cudaMemcpyAsync(static_cast<uint8_t*>(out_host) + lb * q_layer, dout + lb * q_layer, nl * q_layer,
                            cudaMemcpyDeviceToHost, c->copy_out));
    if (lse_out_host)
      QC_CUDA(cudaMemcpyAsync(reinterpret_cast<uint8_t*>(lse_out_host) + lb * lse_layer, dlse + lb * lse_layer,
                              nl * lse_layer, cudaMemcpyDeviceToHost, c->copy_out));
  }
  QC_CUDA(cudaStreamSynchronize(c->copy_out));
  QC_CUDA(cudaStreamSynchronize(stream));
  return QC_OK;
}

int32_t qc_free_seq(qc_cache* c, int32_t seq_id) {
  if (!c || seq_id < 0 || seq_id >= c->cfg.max_seqs) return QC_ERR_INVALID_ARG;
  SeqState& st = c->seqs[seq_id];
  if (!st.active || c->open.active) return QC_ERR_STATE;
  if (c->paged) {
    for (auto it = st.alloc_order.rbegin(); it != st.alloc_order.rend(); ++it) c->free_stack.push_back(*it);
    for (int l = 0; l < c->cfg.n_layers; ++l)
      for (int sm = 0; sm < 4; ++sm) {
        const size_t r = trow(c, l, sm, seq_id);
        std::fill(c->table.begin() + r, c->table.begin() + r + c->max_pages, -1);
      }
  }
  st = SeqState();
  return QC_OK;
}

int32_t qc_get_stats(qc_cache* c, qc_stats* out) {
  if (!c || !out) return QC_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  const int N = c->cfg.n_layers;
  const int64_t row = static_cast<int64_t>(c->hkv) * c->D * 2;
  out->page_bytes = row * kPage;
  out->pages_total = c->n_pool_pages;
  int64_t rows = 0, rows_full = 0, pages = 0, pages_full = 0;
  for (const SeqState& st : c->seqs) {
    if (!st.active) continue;
    out->n_active_seqs++;
    for (int l = 0; l < N; ++l)
      for (int sm = 0; sm < 4; ++sm) {
        const int len = (sm & 1) ? st.len_vis : st.len_text;
        if (owns(c, l, sm)) {
          rows += len;
          pages += pages_for(len);
        }
        rows_full += len;
        pages_full += pages_for(len);
      }
  }
  out->pages_in_use = c->paged ? c->n_pool_pages - static_cast<int64_t>(c->free_stack.size()) : pages;
  out->kv_bytes_stored = rows * row;
  out->kv_bytes_all_full = rows_full * row;
  out->kv_bytes_stored_paged = pages * out->page_bytes;
  out->kv_bytes_all_full_paged = pages_full * out->page_bytes;
  out->qcache_bytes = static_cast<int64_t>(N) * c->cfg.max_seqs * c->hq * c->D * 2;
  out->decode_steps = c->decode_steps;
  out->attend_launches = c->attend_launches;
  out->kernel_launches = c->kernel_launches;
  out->kv_bytes_swept = c->kv_bytes_swept;
  QC_CUDA(cudaSetDevice(c->ctx->device));
  int32_t err = 0;
  QC_CUDA(cudaMemcpyAsync(&err, c->ws + c->lay.err, sizeof(err), cudaMemcpyDeviceToHost, c->ctx->stream));
  QC_CUDA(cudaStreamSynchronize(c->ctx->stream));
  out->device_error = err;
  return QC_OK;
}

int32_t qc_debug_page_table(const qc_cache* c, int32_t layer, int32_t stream, int32_t seq_id, int32_t* page_ids,
                            int32_t cap, int32_t* n_pages, int32_t* n_tokens, int32_t* owner_layer) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || stream < 0 || stream > 3 || seq_id < 0 ||
      seq_id >= c->cfg.max_seqs || cap < 0 || (cap > 0 && !page_ids))
    return QC_ERR_INVALID_ARG;
  const SeqState& st = c->seqs[seq_id];
  int owner = -1, np = 0, nt = 0;
  if (st.active) {
    owner = owns(c, layer, stream) ? layer : c->leader[layer];
    nt = (stream & 1) ? st.len_vis : st.len_text;
    np = pages_for(nt);
    const size_t r = trow(c, owner, stream, seq_id);
    for (int i = 0; i < np && i < cap; ++i) page_ids[i] = c->table[r + i];
  }
  if (n_pages) *n_pages = np;
  if (n_tokens) *n_tokens = nt;
  if (owner_layer) *owner_layer = owner;
  return QC_OK;
}

int32_t qc_debug_read_qcache(qc_cache* c, int32_t layer, void* host_bf16) {
  if (!c || !host_bf16 || layer < 0 || layer >= c->cfg.n_layers) return QC_ERR_INVALID_ARG;
  QC_CUDA(cudaSetDevice(c->ctx->device));
  const size_t bytes = static_cast<size_t>(c->cfg.max_seqs) * c->hq * c->D * 2;
  const uint8_t* src = c->ws + c->lay.qcache + static_cast<size_t>(c->leader[layer]) * bytes;
  QC_CUDA(cudaMemcpyAsync(host_bf16, src, bytes, cudaMemcpyDeviceToHost, c->ctx->stream));
  return sync_and_check(c);
}

int32_t qc_debug_read_row(qc_cache* c, int32_t layer, int32_t stream, int32_t seq_id, int32_t token,
                          int32_t kv_head, void* host_bf16) {
  if (!c || !host_bf16 || layer < 0 || layer >= c->cfg.n_layers || stream < 0 || stream > 3 || seq_id < 0 ||
      seq_id >= c->cfg.max_seqs || kv_head < 0 || kv_head >= c->hkv)
    return QC_ERR_INVALID_ARG;
  const SeqState& st = c->seqs[seq_id];
  if (!st.active) return QC_ERR_STATE;
  const int len = (stream & 1) ? st.len_vis : st.len_text;
  if (token < 0 || token >= len) return QC_ERR_INVALID_ARG;
  const int owner = owns(c, layer, stream) ? layer : c->leader[layer];
  const int32_t pid = c->table[trow(c, owner, stream, seq_id) + token / kPage];
  if (pid < 0 || pid >= c->n_pool_pages) return QC_ERR_STATE;
  const size_t off = ((static_cast<size_t>(pid) * c->hkv + kv_head) * kPage + token % kPage) * c->D;
  QC_CUDA(cudaSetDevice(c->ctx->device));
  QC_CUDA(cudaMemcpyAsync(host_bf16, c->pool + off, c->D * 2, cudaMemcpyDeviceToHost, c->ctx->stream));
  return sync_and_check(c);
}

int32_t qc_set_option(qc_cache* c, const char* key, int64_t value) {
  if (!c || !key) return QC_ERR_INVALID_ARG;
  const std::string k(key);
  if (k == "split_tokens") {
    if (value == 0) {   // back to the per-step choice
      c->auto_split = true;
      return QC_OK;
    }
    if (value % 16 || value < 16 || value > 16 * kMaxChunkPages) return QC_ERR_INVALID_ARG;
    const int cp = static_cast<int>(value / 16);
    if (cp < c->min_chunk_pages) return QC_ERR_INVALID_ARG;   // the workspace was sized for the initial split
    c->chunk_pages = cp;
    c->auto_split = false;
    return QC_OK;
  }
  if (k == "layers_per_launch") {
    if (value < 0 || value > c->cfg.n_layers) return QC_ERR_INVALID_ARG;
    c->layers_per_launch = static_cast<int>(value);
    c->plan_dirty = true;
    return QC_OK;
  }
  if (k == "per_layer_logit_cache") {   // one launch per layer; followers take shared scores from the logit cache
    c->layers_per_launch = value ? -1 : 0;
    c->plan_dirty = true;
    return QC_OK;
  }
  if (k == "in_order_launches") {   // one launch per layer; a leader's launch also sweeps its followers' cached V
    c->layers_per_launch = value ? -2 : 0;
    c->plan_dirty = true;
    return QC_OK;
  }
  if (k == "fused_merge") {   // 0: partial rows are merged by a launch of their own
    c->fused_merge = value != 0;
    c->plan_dirty = true;
    return QC_OK;
  }
  if (k == "static_partition") {
    if (value < -1 || value > 1) return QC_ERR_INVALID_ARG;
    c->static_partition = static_cast<int>(value);
    return QC_OK;
  }
  if (k == "debug_drop_tile") {   // test hook, see qc.h
    c->debug_drop_tile = value != 0;
    return QC_OK;
  }
  if (k == "fold_append") {
    c->fold_append = value != 0;
    return QC_OK;
  }
  if (k == "plan_ahead") {
    c->plan_ahead = value != 0;
    return QC_OK;
  }
  if (k == "static_row_cost") {
    if (value < 0 || value > 64) return QC_ERR_INVALID_ARG;
    c->static_row_cost = static_cast<int>(value);
    return QC_OK;
  }
  if (k == "static_min_tiles") {
    if (value < 1 || value > 4096) return QC_ERR_INVALID_ARG;
    c->static_min_tiles = static_cast<int>(value);
    return QC_OK;
  }
  if (k == "prefill_shared_scores") {
    if (value < 0 || value > 2) return QC_ERR_INVALID_ARG;
    c->prefill_shared = static_cast<int>(value);
    return QC_OK;
  }
  if (k == "prefill_pair_min_tokens") {
    if (value < 0) return QC_ERR_INVALID_ARG;
    c->prefill_pair_min_tokens = static_cast<int>(std::min<int64_t>(value, 1 << 30));
    return QC_OK;
  }
  if (k == "prefill_tcgen05") {
    c->prefill_tcgen05 = value != 0;
    return QC_OK;
  }
  if (k == "profile") {
    if (value < 0 || value > 2) return QC_ERR_INVALID_ARG;
    c->profile = static_cast<int>(value);
    return QC_OK;
  }
  return QC_ERR_INVALID_ARG;
}

int32_t qc_get_profile(qc_cache* c, qc_profile* out) {
  if (!c || !out) return QC_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  QC_CUDA(cudaSetDevice(c->ctx->device));
  QC_CUDA(cudaStreamSynchronize(c->ctx->stream));
  for (int s = 0; s < c->ev_steps; ++s) {
    float a = 0.f, t = 0.f;
    QC_CUDA(cudaEventElapsedTime(&a, c->ev[4 * s + 1], c->ev[4 * s + 2]));
    QC_CUDA(cudaEventElapsedTime(&t, c->ev[4 * s + 0], c->ev[4 * s + 3]));
    out->attend_ms += a;
    out->step_ms += t;
  }
  for (int i = 0; i < c->ev_prefill_calls; ++i) {
    float a = 0.f;
    QC_CUDA(cudaEventElapsedTime(&a, c->ev_prefill[2 * i], c->ev_prefill[2 * i + 1]));
    out->prefill_attend_ms += a;
  }
  out->prefill_calls = c->ev_prefill_calls;
  out->prefill_flops = c->prof_prefill_flops;
  c->ev_prefill_calls = 0;
  c->prof_prefill_flops = 0.0;
  for (int i = 0; i < c->ev_launches; ++i) {
    float a = 0.f;
    QC_CUDA(cudaEventElapsedTime(&a, c->ev_launch[2 * i], c->ev_launch[2 * i + 1]));
    out->attend_kernel_ms += a;
  }
  out->attend_kernel_launches = c->ev_launches;
  c->ev_launches = 0;
  out->steps = c->ev_steps;
  out->kv_bytes_read = c->prof_bytes;
  out->items = c->prof_items;
  c->ev_steps = 0;
  c->prof_bytes = 0;
  c->prof_items = 0;
  return QC_OK;
}

}  // extern "C"
