// CUDA kernels of the Lazy Attention decode path (sm_100a).
//
//   setup_kernel    expands the step's (plan position, sequence) pairs into split-KV work items,
//                   applies page-table patches, resets the work counters and -- on steps without
//                   patches -- also does the append
//   append_kernel   writes the new token's k / v rows into the text streams and every
//                   ordinary layer's q into the Q Cache (a launch of its own on steps with patches
//                   and per launch group of the host-buffer entry point)
//   plan_kernel     for a step whose launches are cut into static tile ranges: where every worker of
//                   every launch starts (first item, its first page ids, the cursor for the rest)
//   attend_kernel   persistent split-KV partial attention, one query head per work item (MHA):
//                   each warp is an independent worker that takes items -- claimed from a counter,
//                   or the pieces of its static range of the launch's tiles -- streams K/V page
//                   tiles through its own shared-memory ring with bulk asynchronous copies and
//                   keeps an online softmax in registers; a leader's sweep can weight several
//                   layers' V rows with one set of scores, store its scaled scores in the logit
//                   cache, or leave out the step's new token for its followers
//                   (the grouped-query variant on tensor cores is in qc_attend_tc.cu)
//   merge_kernel    log-sum-exp merge of the partials, bf16 output
//   prefill_scatter_kernel  stores prompt K/V rows into their pages
//
// Attention arithmetic: scores are kept in the log2 domain (q is pre-multiplied by
// scale * log2 e), accumulation is fp32, inputs and outputs are bf16.

#include "qc_device.cuh"

namespace qc {
namespace {

// ------------------------------------------------------------------------------------------
// setup: page-table patches + item expansion
// ------------------------------------------------------------------------------------------

// new token's k, v rows of one (sequence, layer) and the Q Cache refresh
__device__ __forceinline__ void append_rows(const Params& P, const StepSeq& sq, int si, int layer) {
  const int pos = sq.len_text - 1;          // ordinal of the new token in the text stream
  const int pg = pos / kPage, slot = pos % kPage;
  const uint8_t lf = P.layer_flags[layer];
  const int vec_per_row = P.d / 8;          // uint4 per head row
  const int n_kv_vec = P.hkv * vec_per_row;
  const size_t in_kv = (static_cast<size_t>(layer) * P.n_seqs + si) * P.hkv * P.d;

  const int pid_v = P.table[table_row(P, layer, 2, sq.seq_id) + pg];
  const int pid_k = (lf & kLayerOwnsTextK) ? P.table[table_row(P, layer, 0, sq.seq_id) + pg] : -1;
  for (int e = threadIdx.x; e < n_kv_vec; e += blockDim.x) {
    const int head = e / vec_per_row, j = e - head * vec_per_row;
    const size_t src = in_kv + static_cast<size_t>(head) * P.d + j * 8;
    const size_t dst_v = ((static_cast<size_t>(pid_v) * P.hkv + head) * kPage + slot) * P.d + j * 8;
    *reinterpret_cast<uint4*>(P.pool + dst_v) = *reinterpret_cast<const uint4*>(P.v + src);
    if (pid_k >= 0) {
      const size_t dst_k = ((static_cast<size_t>(pid_k) * P.hkv + head) * kPage + slot) * P.d + j * 8;
      *reinterpret_cast<uint4*>(P.pool + dst_k) = *reinterpret_cast<const uint4*>(P.k + src);
    }
  }
  if (lf & kLayerWritesQCache) {
    const int n_q_vec = P.hq * vec_per_row;
    const size_t src0 = (static_cast<size_t>(layer) * P.n_seqs + si) * P.hq * P.d;
    const size_t dst0 = (static_cast<size_t>(layer) * P.max_seqs + sq.seq_id) * P.hq * P.d;
    for (int e = threadIdx.x; e < n_q_vec; e += blockDim.x)
      reinterpret_cast<uint4*>(P.qcache + dst0)[e] = reinterpret_cast<const uint4*>(P.q + src0)[e];
  }
}

// Block roles, in grid order: n_pos * n_seqs blocks expand one (plan position, sequence) each
// into work items; housekeeping blocks apply page-table patches, reset the work counters and
// store the inline sequence descriptors for the later kernels; with fused_append, n_seqs *
// n_layers blocks do the append.  (The append reads page ids from the table, so it is only
// fused on steps without patches.)
__global__ void setup_kernel(const __grid_constant__ Params P, const __grid_constant__ StepInline inl) {
  // With claimed items the attention kernel touches nothing before its own wait, so it may be
  // scheduled while this kernel runs; under the static partition it plans its first work ahead of
  // its wait from what this kernel writes, and must not start early.
  if (!P.part_static) pdl_launch_dependents();
  pdl_wait();
  const StepSeq* seqs = P.inline_seqs ? inl.seqs : P.seqs;
  const int n_expand = P.n_pos * P.n_seqs;
  const int n_house = (max(max(P.n_patches, P.n_layers), P.n_seqs * 8) + blockDim.x - 1) / blockDim.x;
  int b = blockIdx.x;
  if (b >= n_expand + n_house) {   // append blocks
    b -= n_expand + n_house;
    const int si = b % P.n_seqs, layer = b / P.n_seqs;
    append_rows(P, seqs[si], si, layer);
    return;
  }
  if (b >= n_expand) {   // housekeeping blocks
    const int i = (b - n_expand) * blockDim.x + threadIdx.x;
    if (i < P.n_patches) P.table[P.patches[i].index] = P.patches[i].page;
    if (i < P.n_layers) P.work_counter[i] = 0;
    if (P.inline_seqs && i < P.n_seqs * 8)
      reinterpret_cast<int32_t*>(P.seqs)[i] = reinterpret_cast<const int32_t*>(inl.seqs)[i];
    return;
  }
  const int pos = b / P.n_seqs, si = b - pos * P.n_seqs;
  const StepSeq sq = seqs[si];
  const PlanJob pj = P.plan[pos];
  const Job jb = pj.job;
  const int len = jb.stream ? sq.len_vis : sq.len_text;
  const int n_chunks = jb.stream ? sq.ncv : sq.n_slots - sq.ncv;
  const int item_base = pj.vis_before * P.tot_v + pj.text_before * P.tot_t + (jb.stream ? sq.pre_v : sq.pre_t);
  const int slot_base = jb.stream ? 0 : sq.ncv;
  const int per_chunk = P.heads_per_item_dim;   // items per chunk
  const int hpi = P.heads_per_item;
  const int n_sub = (P.group + hpi - 1) / hpi;  // items per KV head
  const int total_pages = (len + kPage - 1) / kPage;
  const int n = n_chunks * per_chunk;
  for (int t = threadIdx.x; t < n; t += blockDim.x) {
    const int chunk = t / per_chunk;
    const int u = t - chunk * per_chunk;
    const int kv_head = u / n_sub, sub = u - kv_head * n_sub;
    Item it;
    it.k_layer = jb.k_layer;
    it.stream = jb.stream;
    it.n_cons = jb.n_cons;
    it.flags = jb.flags;
#pragma unroll
    for (int x = 0; x < kMaxCons; ++x) {
      it.v_layer[x] = jb.v_layer[x];
      it.q_layer[x] = jb.q_layer[x];
    }
    it.seq_id = static_cast<uint16_t>(sq.seq_id);
    it.seq_idx = static_cast<uint16_t>(si);
    it.head = static_cast<uint16_t>(kv_head * P.group + sub * hpi);
    it.slot = static_cast<uint16_t>(slot_base + chunk);
    const int first = chunk * P.chunk_pages;
    const int np = min(P.chunk_pages, total_pages - first);
    it.first_page = static_cast<uint16_t>(first);
    it.n_pages = static_cast<uint16_t>(np);
    const bool last = (first + np == total_pages);
    if (last) it.flags |= kFlagStreamEnd;
    it.n_valid_last = static_cast<uint16_t>(last ? len - (total_pages - 1) * kPage : kPage);
    it.n_heads = static_cast<uint8_t>(min(hpi, P.group - sub * hpi));
    it.skip_new = jb.skip_new;
    it.finish = jb.finish;
    it.pad1 = 0;
    it.n_pieces = 0;
    P.items[item_base + t] = it;
  }
}

// ------------------------------------------------------------------------------------------
// append: new token's k, v rows and the Q Cache refresh (separate launch on steps with patches)
// ------------------------------------------------------------------------------------------

__global__ void append_kernel(const __grid_constant__ Params P) {
  pdl_wait();
  // what the next kernel does ahead of its own wait reads nothing this kernel writes (an attention
  // worker's early tiles leave out the page that can hold the new token)
  pdl_launch_dependents();
  append_rows(P, P.seqs[blockIdx.x], blockIdx.x, P.layer_begin + blockIdx.y);   // layers of one launch group
}

// ------------------------------------------------------------------------------------------
// plan: where every worker of every statically partitioned launch of the step starts
// ------------------------------------------------------------------------------------------

__global__ void plan_kernel(const __grid_constant__ Params P, const __grid_constant__ LaunchList list) {
  pdl_wait();   // the page tables and the sequence descriptors are final
  const int g = blockIdx.y, wid = blockIdx.x * blockDim.x + threadIdx.x;
  const LaunchDesc L = list.launch[g];
  if (wid >= kPlanWorkers) return;
  WorkerDesc* out = const_cast<WorkerDesc*>(P.wdesc) + static_cast<size_t>(g) * kPlanWorkers + wid;
  PartView V = part_view(P);
  V.pos_begin = L.pos_begin, V.pos_end = L.pos_end;
  V.q = L.part_q, V.k = L.part_k, V.vw = L.part_vw, V.row_cost = L.part_row_cost;
  WorkerDesc d;
  d.item.n_pages = 0;
  RangeCursor c;
  if (wid < L.part_workers && cursor_init_scalar(c, V, wid) && cursor_next(c, V, d.item)) {
    const Item& it = d.item;
    for (int j = 0; j < 2; ++j) {
      const int pg = it.first_page + min(j, it.n_pages - 1);
      d.pids[0][j] = P.table[table_row(P, it.k_layer, it.stream, it.seq_id) + pg];
      for (int x = 0; x < kMaxCons; ++x)
        d.pids[1 + x][j] = x < it.n_cons ? P.table[table_row(P, it.v_layer[x], 2 + it.stream, it.seq_id) + pg] : 0;
    }
    d.pad[0] = d.pad[1] = 0;
    *reinterpret_cast<RangeCursor*>(d.cursor) = c;
  } else {
    d.item.n_pages = 0;
  }
  const uint4* src = reinterpret_cast<const uint4*>(&d);
  uint4* dst = reinterpret_cast<uint4*>(out);
  if (d.item.n_pages == 0) {   // no work: an all-zero item says so
    dst[0] = make_uint4(0, 0, 0, 0);
    dst[1] = make_uint4(0, 0, 0, 0);
    return;
  }
#pragma unroll
  for (int i = 0; i < 10; ++i) dst[i] = src[i];
}

// ------------------------------------------------------------------------------------------
// prefill scatter
// ------------------------------------------------------------------------------------------

__global__ void prefill_scatter_kernel(Params P, const int32_t* tok_seq, const int32_t* tok_stream,
                                       const int32_t* tok_ord, int32_t tok_stride, int32_t tok_offset) {
  const int t = blockIdx.x;
  const int layer = blockIdx.y;
  const int seq = tok_seq[t], stream = tok_stream[t], ord = tok_ord[t];
  const int pg = ord / kPage, slot = ord % kPage;
  const uint8_t lf = P.layer_flags[layer];
  // K of a lazy layer: visual rows are never kept; text rows only where the mode keeps them
  const bool keep_k = (lf & kLayerWritesQCache) || (stream == 0 && (lf & kLayerOwnsTextK));
  const int pid_v = P.table[table_row(P, layer, 2 + stream, seq) + pg];
  const int pid_k = keep_k ? P.table[table_row(P, layer, stream, seq) + pg] : -1;
  const int vec_per_row = P.d / 8;
  const int n_vec = P.hkv * vec_per_row;
  const size_t in = (static_cast<size_t>(layer) * tok_stride + tok_offset + t) * P.hkv * P.d;
  for (int e = threadIdx.x; e < n_vec; e += blockDim.x) {
    const int head = e / vec_per_row, j = e - head * vec_per_row;
    const size_t src = in + static_cast<size_t>(head) * P.d + j * 8;
    const size_t dst_v = ((static_cast<size_t>(pid_v) * P.hkv + head) * kPage + slot) * P.d + j * 8;
    *reinterpret_cast<uint4*>(P.pool + dst_v) = *reinterpret_cast<const uint4*>(P.v + src);
    if (pid_k >= 0) {
      const size_t dst_k = ((static_cast<size_t>(pid_k) * P.hkv + head) * kPage + slot) * P.d + j * 8;
      *reinterpret_cast<uint4*>(P.pool + dst_k) = *reinterpret_cast<const uint4*>(P.k + src);
    }
  }
}

// ------------------------------------------------------------------------------------------
// attend: persistent split-KV partial attention, one independent worker per warp
// ------------------------------------------------------------------------------------------

constexpr int kRing = 2;                  // tiles in flight per warp

template <int D>
struct WarpCtx {
  ItemPages ip;
  uint4 qraw[kMaxCons][D / 8];
};

// Start fetching the raw queries of the item in a context slot (asynchronous copies).
template <int D>
__device__ __forceinline__ void begin_queries(WarpCtx<D>& c, const Params& P, const Item& it, int lane) {
  const int nq = (it.flags & kFlagShared) ? 1 : it.n_cons;
  if (lane < D / 8) {
    for (int x = 0; x < nq; ++x) {
      const bool cached = (it.flags >> (kFlagCachedShift + x)) & 1;
      const uint16_t* src =
          cached ? P.qcache + ((static_cast<size_t>(it.q_layer[x]) * P.max_seqs + it.seq_id) * P.hq + it.head) * D
                 : P.q + ((static_cast<size_t>(it.q_layer[x]) * P.n_seqs + it.seq_idx) * P.hq + it.head) * D;
      cp_async_16(&c.qraw[x][lane], reinterpret_cast<const uint4*>(src) + lane);
    }
  }
}

// One item: NQ queries score the K tiles, NV value streams are accumulated.
// NQ == 1: every consumer shares the weights; NQ == NV: consumer x has its own query.
// MODE 1 (one query, one consumer) also stores the scaled scores in the logit cache; MODE 2 takes
// them from there instead of reading K tiles (the ring then carries V tiles only).
// SKIP (shared weights only): the consumers named in the item's skip_new mask leave out the
// stream's last key -- the step's new token, whose value row of a follower does not exist yet when
// its leader's launch runs (Eq. 6: V = [cached V, new v]); they get their own sum of weights.
// FOLD: the item may end its layer's text stream under the folded append (the new token's rows come
// from the step's inputs).  Launches without the folded append use the instantiation without it,
// whose page loop then carries none of this (with it in every instantiation the one-launch step was
// 3.5 % slower); under the folded append every single-consumer item of a launch takes this one
// (sending only the items that end a stream here made the workers alternate between two copies of
// the loop: 1.20 against 1.09 ms per step at config 2).
template <int D, int NQ, int NV, int MODE = 0, bool SKIP = false, bool FOLD = false>
__device__ __forceinline__ void process_item(WorkerState& st, const WarpCtx<D>* ctx, uint32_t ring, uint64_t* full,
                                             const Params& P, int lane) {
  auto ctx_of = [ctx](int k) -> const ItemPages& { return ctx[k % kCtxSlots].ip; };
  constexpr int EPL = D / 8;    // elements of a row held by one lane
  constexpr int LPR = D / 64;   // 16-byte loads per lane per row
  const WarpCtx<D>& c = ctx[st.cons_k % kCtxSlots];
  const int kg = lane >> 3;     // which of 4 keys of a pass
  const int c8 = lane & 7;      // which 16-byte chunk of the row (and of its second half)

  float qf[NQ][EPL];
#pragma unroll
  for (int x = 0; x < NQ; ++x) {
#pragma unroll
    for (int j = 0; j < LPR; ++j) {
      const uint4 raw = c.qraw[x][c8 + 8 * j];
      bf16x8_to_f32(raw, &qf[x][8 * j]);
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) qf[x][e] *= P.scale_log2;
  }

  float m[NQ], l[NQ], acc[NV][EPL];
#pragma unroll
  for (int x = 0; x < NQ; ++x) {
    m[x] = -INFINITY;
    l[x] = 0.f;
  }
#pragma unroll
  for (int v = 0; v < NV; ++v)
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[v][e] = 0.f;

  const int n_pages = c.ip.item.n_pages;
  const int n_valid_last = c.ip.item.n_valid_last;
  // SKIP: the new token is key n_valid_last - 1 of the item's last page when that page ends the stream
  const bool skip_here = SKIP && (c.ip.item.flags & kFlagStreamEnd);
  const uint32_t skip_mask = SKIP ? c.ip.item.skip_new : 0u;
  float l_skip = 0.f;       // sum of weights without the new token
  float* lg = nullptr;      // this item's first key in the logit cache
  float lg_next[4] = {0.f, 0.f, 0.f, 0.f};
  if (MODE != 0) {
    lg = logit_row(P, c.ip.item.stream, c.ip.item.seq_id, c.ip.item.head) + c.ip.item.first_page * kPage;
    if (MODE == 2) {
#pragma unroll
      for (int i = 0; i < 4; ++i) lg_next[i] = lg[4 * i + kg];
    }
  }

  constexpr bool kMayFold = FOLD || SKIP;
  const int new_pg = (kMayFold && holds_new_token(P, c.ip.item, n_pages - 1)) ? n_pages - 1 : -1;   // folded append: page of the new token
  for (int pg = 0; pg < n_pages && !st.dead; ++pg) {
    const int nvalid = (pg == n_pages - 1) ? n_valid_last : kPage;
    float p[NQ][4];
    if (MODE == 2) {
      // ---- scores of 16 keys from the logit cache; the next page's are requested now
#pragma unroll
      for (int i = 0; i < 4; ++i) p[0][i] = lg_next[i];
      if (pg + 1 < n_pages) {
#pragma unroll
        for (int i = 0; i < 4; ++i) lg_next[i] = lg[(pg + 1) * kPage + 4 * i + kg];
      }
    } else {
      // ---- K tile: scores of 16 keys
      const uint8_t* tile = static_cast<const uint8_t*>(__cvta_shared_to_generic(wait_tile<D>(st, ring, full, P, lane)));
      if (st.dead) break;
      if (kMayFold && pg == new_pg) {
        // the new token's k row comes from the step's input: into the tile, and into the pool for later steps
        const Item& it = c.ip.item;
        if (lane < D / 8) {
          const uint4 val = c.ip.new_k[lane];
          reinterpret_cast<uint4*>(const_cast<uint8_t*>(tile) + (nvalid - 1) * (D * 2))[lane] = val;
          const int pid = c.ip.pages[0][pg];
          if (static_cast<uint32_t>(pid) < static_cast<uint64_t>(P.n_pool_pages))
            reinterpret_cast<uint4*>(P.pool + ((static_cast<size_t>(pid) * P.hkv + c.ip.kv_head) * kPage + (nvalid - 1)) * D)[lane] = val;
          // an ordinary layer's query goes to the Q Cache
          if (it.q_layer[0] == it.k_layer && !((it.flags >> kFlagCachedShift) & 1) && (P.layer_flags[it.k_layer] & kLayerWritesQCache))
            reinterpret_cast<uint4*>(P.qcache + ((static_cast<size_t>(it.k_layer) * P.max_seqs + it.seq_id) * P.hq + it.head) * D)[lane] =
                c.qraw[0][lane];
        }
        __syncwarp();
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = 4 * i + kg;
        const uint4* row = reinterpret_cast<const uint4*>(tile + r * (D * 2));
        float kf[EPL];
#pragma unroll
        for (int j = 0; j < LPR; ++j) bf16x8_to_f32(row[c8 + 8 * j], &kf[8 * j]);
#pragma unroll
        for (int x = 0; x < NQ; ++x) {
          float a0 = 0.f, a1 = 0.f;
#pragma unroll
          for (int e = 0; e < EPL; e += 2) {
            a0 = fmaf(kf[e], qf[x][e], a0);
            a1 = fmaf(kf[e + 1], qf[x][e + 1], a1);
          }
          p[x][i] = a0 + a1;
        }
      }
      release_tile<kRing>(st);
      fill_ring<D, kRing, false>(st, ctx_of, ring, full, P, lane);
    }
#pragma unroll
    for (int x = 0; x < NQ; ++x) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float s = p[x][i];
        if (MODE != 2) {
          s += __shfl_xor_sync(0xffffffffu, s, 1);
          s += __shfl_xor_sync(0xffffffffu, s, 2);
          s += __shfl_xor_sync(0xffffffffu, s, 4);
        }
        if (MODE == 1 && c8 == 0 && 4 * i + kg < nvalid) lg[pg * kPage + 4 * i + kg] = s;
        p[x][i] = (4 * i + kg < nvalid) ? s : -INFINITY;
      }
      float tmax = fmaxf(fmaxf(p[x][0], p[x][1]), fmaxf(p[x][2], p[x][3]));
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 8));
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 16));
      const float m_new = fmaxf(m[x], tmax);
      const float corr = exp2f(m[x] - m_new);
      float psum = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        p[x][i] = exp2f(p[x][i] - m_new);
        psum += p[x][i];
      }
      l[x] = l[x] * corr + psum;
      if (SKIP) {
        float psum_skip = psum;
        if (skip_here && pg == n_pages - 1) {
          const int r_new = nvalid - 1;
#pragma unroll
          for (int i = 0; i < 4; ++i)
            if (4 * i + kg == r_new) psum_skip -= p[x][i];
        }
        l_skip = l_skip * corr + psum_skip;
      }
      m[x] = m_new;
      if (corr != 1.f) {
#pragma unroll
        for (int v = 0; v < NV; ++v) {
          if (NQ == 1 || v == x) {
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[v][e] *= corr;
          }
        }
      }
    }
    // ---- V tiles: weighted sums for each consumer
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const uint8_t* tile = static_cast<const uint8_t*>(__cvta_shared_to_generic(wait_tile<D>(st, ring, full, P, lane)));
      if (st.dead) break;
      const int nvalid_v = (SKIP && skip_here && pg == n_pages - 1) ? nvalid - static_cast<int>((skip_mask >> v) & 1u) : nvalid;
      if (kMayFold && pg == new_pg && nvalid_v == nvalid) {
        // this consumer's new v row, likewise
        const Item& it = c.ip.item;
        if (lane < D / 8) {
          const uint4 val = v == first_taker(it)
                                ? c.ip.new_v[lane]
                                : reinterpret_cast<const uint4*>(
                                      P.v + ((static_cast<size_t>(it.v_layer[v]) * P.n_seqs + it.seq_idx) * P.hkv + c.ip.kv_head) * D)[lane];
          reinterpret_cast<uint4*>(const_cast<uint8_t*>(tile) + (nvalid - 1) * (D * 2))[lane] = val;
          const int pid = c.ip.pages[1 + v][pg];
          if (static_cast<uint32_t>(pid) < static_cast<uint64_t>(P.n_pool_pages))
            reinterpret_cast<uint4*>(P.pool + ((static_cast<size_t>(pid) * P.hkv + c.ip.kv_head) * kPage + (nvalid - 1)) * D)[lane] = val;
        }
        __syncwarp();
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = 4 * i + kg;
        if (r < nvalid_v) {
          const uint4* row = reinterpret_cast<const uint4*>(tile + r * (D * 2));
          float vf[EPL];
#pragma unroll
          for (int j = 0; j < LPR; ++j) bf16x8_to_f32(row[c8 + 8 * j], &vf[8 * j]);
          const float pv = p[NQ == 1 ? 0 : v][i];
#pragma unroll
          for (int e = 0; e < EPL; ++e) acc[v][e] = fmaf(pv, vf[e], acc[v][e]);
        }
      }
      release_tile<kRing>(st);
      fill_ring<D, kRing, false>(st, ctx_of, ring, full, P, lane);
    }
  }
  if (st.dead) return;

  // ---- partial results: sum over the 4 key groups, then lanes 0..7 store
#pragma unroll
  for (int x = 0; x < NQ; ++x) {
    l[x] += __shfl_xor_sync(0xffffffffu, l[x], 8);
    l[x] += __shfl_xor_sync(0xffffffffu, l[x], 16);
  }
  if (SKIP) {
    l_skip += __shfl_xor_sync(0xffffffffu, l_skip, 8);
    l_skip += __shfl_xor_sync(0xffffffffu, l_skip, 16);
  }
#pragma unroll
  for (int v = 0; v < NV; ++v) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      acc[v][e] += __shfl_xor_sync(0xffffffffu, acc[v][e], 8);
      acc[v][e] += __shfl_xor_sync(0xffffffffu, acc[v][e], 16);
    }
  }
  if (kg == 0) {
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const size_t row =
          ((static_cast<size_t>(c.ip.item.v_layer[v]) * P.max_seqs + c.ip.item.seq_idx) * P.max_slots + c.ip.item.slot) *
              P.hq + c.ip.item.head;
      float* dst = P.part_acc + row * D;
#pragma unroll
      for (int j = 0; j < LPR; ++j) {
        float4* d4 = reinterpret_cast<float4*>(dst + 64 * j + 8 * c8);
        d4[0] = make_float4(acc[v][8 * j + 0], acc[v][8 * j + 1], acc[v][8 * j + 2], acc[v][8 * j + 3]);
        d4[1] = make_float4(acc[v][8 * j + 4], acc[v][8 * j + 5], acc[v][8 * j + 6], acc[v][8 * j + 7]);
      }
      const bool skipping = SKIP && ((skip_mask >> v) & 1u);
      if (c8 == 0) P.part_ml[row] = make_float2(m[NQ == 1 ? 0 : v], skipping ? l_skip : l[NQ == 1 ? 0 : v]);
    }
  }
  finish_rows<D>(P, c.ip, lane);
}

// A worker's life: take items (claimed from the list, or the pieces of its static ranges), keep
// the tile ring full across item boundaries, process each item.  While item k is processed the
// ring already fetches tiles of item k + 1 and the context of item k + 2 (descriptor, page ids,
// queries) arrives by asynchronous copies.
template <int D, bool STATIC>
__device__ __forceinline__ void attend_worker(const Params& P, WarpCtx<D>* ctx, uint32_t ring, uint64_t* full,
                                              RangeCursor* cursor, int32_t* stage, int wid, int lane) {
  auto ctx_of = [ctx](int k) -> const ItemPages& { return ctx[k % kCtxSlots].ip; };
  WorkerState st;
  worker_init(st, 0);
  st.drop_next = P.debug_drop_tile != 0;   // (test hook)
  Item it;
  int issued = 0;
  auto take = [&]() -> bool {   // the next item into `it`
    if (STATIC) return cursor_step(cursor, P, it, lane);
    const int idx = claim_take(P, issued);
    if (idx < 0) return false;
    it = load_item(P, idx);
    return true;
  };
  // ---- ahead of the wait for the previous kernel: the first items and their page ids (from the
  // launch plan, the step descriptors and the page tables, all written before that kernel
  // started), and the first tiles unless they could hold a new token that an earlier launch of the
  // step stores (with the folded append the worker patches the new token's row itself)
  Item first;
  if (STATIC && P.wdesc != nullptr) {
    // planned ahead: one read gives the first item, its first page ids and the cursor
    if (wid >= P.part_workers) return;
    if (!load_worker_desc(P, wid, ctx[0].ip, cursor, stage, lane)) return;
    first = ctx[0].ip.item;
    st.n_my = 1;
    const bool early_tiles = P.fold_append || !(first.stream == 0 && (first.flags & kFlagStreamEnd) && first.n_pages <= kRing);
    if (early_tiles) fill_ring<D, kRing, false>(st, ctx_of, ring, full, P, lane);
    begin_item_pages(ctx[0].ip, P, first, lane);   // the whole page list, while the tiles fly
  } else {
    if (STATIC) {
      if (wid >= P.part_workers) return;
      RangeCursor c;
      const bool any = cursor_init(c, part_view(P), wid, lane);
      if (lane == 0) *cursor = c;
      __syncwarp();
      if (!any) return;
    } else {
      pdl_wait();   // the item list and the work counter are the previous kernel's
      pdl_launch_dependents();
      issued = claim_issue(P, lane);
    }
    if (!take()) return;
    begin_item_pages(ctx[0].ip, P, it, lane);
    first = it;
    cp_async_wait_all();
    __syncwarp();
    st.n_my = 1;
    const bool early_tiles = P.fold_append || !(first.stream == 0 && (first.flags & kFlagStreamEnd) && first.n_pages <= kRing);
    if (early_tiles) fill_ring<D, kRing, false>(st, ctx_of, ring, full, P, lane);
  }
  if (STATIC) {
    pdl_wait();
    pdl_launch_dependents();
  }
  // ---- this layer's inputs; the rest of the first tiles; the second item's context while they fly
  begin_queries<D>(ctx[0], P, first, lane);
  begin_new_rows(ctx[0].ip, P, first, lane, D);
  fill_ring<D, kRing, false>(st, ctx_of, ring, full, P, lane);
  if (STATIC) record_row_slots(P, first, lane);
  if (!STATIC) issued = claim_issue(P, lane);
  bool more = take();
  if (more) {
    begin_item_pages(ctx[1].ip, P, it, lane);
    begin_queries<D>(ctx[1], P, it, lane);
    begin_new_rows(ctx[1].ip, P, it, lane, D);
    if (STATIC) record_row_slots(P, it, lane);
  }
  cp_async_wait_all();
  __syncwarp();
  if (more) st.n_my = 2;
  bool pending = false;   // a context is being filled for item st.n_my
  if (!STATIC && more) issued = claim_issue(P, lane);

  for (int k = 0; k < st.n_my && !st.dead; ++k) {
    const Item& cur = ctx[k % kCtxSlots].ip.item;
    const int nc = cur.n_cons;
    const bool shared = cur.flags & kFlagShared;
    if (more) {
      // the third slot is free (it held the item before this one): start filling it with the item after next
      more = take();
      if (more) {
        begin_item_pages(ctx[(k + 2) % kCtxSlots].ip, P, it, lane);
        begin_queries<D>(ctx[(k + 2) % kCtxSlots], P, it, lane);
        begin_new_rows(ctx[(k + 2) % kCtxSlots].ip, P, it, lane, D);
        if (STATIC) record_row_slots(P, it, lane);
        pending = true;
      }
    }
    if (!STATIC && more) issued = claim_issue(P, lane);   // answered by the time the next item starts
    if (nc == 1 && (cur.flags & kFlagReadLogits)) process_item<D, 1, 1, 2>(st, ctx, ring, full, P, lane);
    else if (nc == 1 && (cur.flags & kFlagWriteLogits)) process_item<D, 1, 1, 1>(st, ctx, ring, full, P, lane);
    else if (shared && cur.skip_new) {
      if (nc == 1) process_item<D, 1, 1, 0, true>(st, ctx, ring, full, P, lane);
      else if (nc == 2) process_item<D, 1, 2, 0, true>(st, ctx, ring, full, P, lane);
      else if (nc == 3) process_item<D, 1, 3, 0, true>(st, ctx, ring, full, P, lane);
      else process_item<D, 1, 4, 0, true>(st, ctx, ring, full, P, lane);
    }
    else if (nc == 1 && P.fold_append) process_item<D, 1, 1, 0, false, true>(st, ctx, ring, full, P, lane);   // (one code path per launch)
    else if (nc == 1) process_item<D, 1, 1>(st, ctx, ring, full, P, lane);
    else if (shared && nc == 2) process_item<D, 1, 2>(st, ctx, ring, full, P, lane);
    else if (shared && nc == 3) process_item<D, 1, 3>(st, ctx, ring, full, P, lane);
    else if (shared) process_item<D, 1, 4>(st, ctx, ring, full, P, lane);
    else if (nc == 2) process_item<D, 2, 2>(st, ctx, ring, full, P, lane);
    else if (nc == 3) process_item<D, 3, 3>(st, ctx, ring, full, P, lane);
    else process_item<D, 4, 4>(st, ctx, ring, full, P, lane);
    if (st.dead) break;
    if (pending) {   // the context of item k + 2 has had this item's time to arrive
      cp_async_wait_all();
      __syncwarp();
      st.n_my = k + 3;
      pending = false;
    }
    st.cons_k = k + 1;
    fill_ring<D, kRing, false>(st, ctx_of, ring, full, P, lane);
  }
  if (st.dead) {
    cp_async_wait_all();
    drain_ring<kRing>(st, full, P.debug_drop_tile ? kDebugSpinLimit : kSpinLimit);
  }
}

template <int D, bool STATIC>
__global__ void __launch_bounds__(kThreads, 1) attend_kernel(const __grid_constant__ Params P) {
  constexpr uint32_t kTile = kPage * D * 2;
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(8) uint64_t full_all[kWarps][kRing];
  __shared__ __align__(16) RangeCursor cursors[kWarps];
  __shared__ __align__(16) int32_t stages[kWarps][12];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t ring = smem_u32(smem) + static_cast<uint32_t>(warp) * kRing * kTile;
  WarpCtx<D>* ctx = reinterpret_cast<WarpCtx<D>*>(smem + static_cast<size_t>(kWarps) * kRing * kTile) + warp * kCtxSlots;
  uint64_t* full = full_all[warp];

  if (lane == 0) {
    for (int s = 0; s < kRing; ++s) mbar_init(&full[s], 1);
    fence_mbar_init();
  }
  __syncthreads();

  attend_worker<D, STATIC>(P, ctx, ring, full, &cursors[warp], stages[warp], worker_index(P, warp, kWarps), lane);
}

// ------------------------------------------------------------------------------------------
// merge: log-sum-exp combination of the partials of one (layer, sequence, head) per warp
// ------------------------------------------------------------------------------------------

// One warp per (layer, sequence, head).  Under the static partition the numbers of partial rows
// are themselves data the attention kernel wrote, so the generic merge needs three dependent
// rounds of loads (counts, then (max, sum) pairs, then rows).  When a row has at most 16 partials
// per stream (the common case: a launch per layer leaves a handful) everything is requested in
// one round instead: the counts, the pairs of the first 16 slots of either stream (lanes 0..15 /
// 16..31) and the rows that a guess at the counts names (up to 4 or 16 of the visual stream, 4 of the
// text stream); what the counts then rule out is ignored, rows beyond those take one more round
// (eight visual rows in the first round were measured slower: rows never written are not in the
// L2).  The step's sequence descriptor is read ahead of the wait for the
// attention kernel (it was written when the step began).
// NVIS = 0: the general path alone (few registers: a launch per step merges every layer's rows);
// NVIS = 4 / 16: the one-round path with up to NVIS visual rows in the first round (the host knows
// from the partition whether a row of the launch can leave more than four).
template <int D, int NVIS>
__global__ void merge_kernel(const __grid_constant__ Params P) {
  constexpr int VPL = D / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_layers = P.layer_end - P.layer_begin;
  const int idx = blockIdx.x * (blockDim.x >> 5) + warp;
  const bool live = idx < n_layers * P.n_seqs * P.hq;
  const int head = idx % P.hq;
  const int si = (idx / P.hq) % P.n_seqs;
  const int layer = P.layer_begin + idx / (P.hq * P.n_seqs);
  StepSeq sq{};
  if (live) sq = P.seqs[si];
  const size_t row = (static_cast<size_t>(layer) * P.max_seqs + si) * P.hq + head;
  // A guess at the row's piece counts, read while the attention kernel may still run: its workers
  // record the counts when they start a row, and the entry keeps the previous step's counts until
  // then, which are nearly always the same.  The guess only decides which rows the first round of
  // loads asks for (rows never written are not in the L2); the counts used are read after the wait.
  uint32_t guess = 0;
  if (NVIS > 0 && live) guess = __ldcg(reinterpret_cast<const uint32_t*>(P.row_slots + 2 * row));
  pdl_wait();
  pdl_launch_dependents();
  if (!live) return;
  if (NVIS == 0) {
    merge_row<D>(P, layer, si, head, sq, lane, P.extra_key_leader);
    return;
  }
  constexpr int NV1 = NVIS > 0 ? NVIS : 1;   // visual rows of the first round
  const int S = P.slots_per_stream;
  const size_t base = (static_cast<size_t>(layer) * P.max_seqs + si) * P.max_slots;
  const uint32_t both = __ldcg(reinterpret_cast<const uint32_t*>(P.row_slots + 2 * row));
  const int my_slot = lane < 16 ? lane : S + lane - 16;
  float2 my_ml = make_float2(-INFINITY, 0.f);
  if ((lane & 15) < S) my_ml = __ldcg(P.part_ml + (base + my_slot) * P.hq + head);
  const int gv = min(min(static_cast<int>(guess & 0xffffu), NV1), S), gt = min(static_cast<int>(guess >> 16), 4);
  float v[NV1 + 4][VPL];   // rows of visual slots 0..NV1-1 and text slots 0..3, as far as the guess goes
#pragma unroll
  for (int u = 0; u < NV1 + 4; ++u) {
    const int s = u < NV1 ? u : S + u - NV1;
    const float* src = P.part_acc + ((base + s) * P.hq + head) * D + lane * VPL;
    if ((u < NV1 ? u : u - NV1) < (u < NV1 ? gv : gt)) {
      if (VPL == 4) {
        const float4 a = __ldcg(reinterpret_cast<const float4*>(src));
        v[u][0] = a.x, v[u][1] = a.y, v[u][2 % VPL] = a.z, v[u][3 % VPL] = a.w;
      } else {
        const float2 a = __ldcg(reinterpret_cast<const float2*>(src));
        v[u][0] = a.x, v[u][1] = a.y;
      }
    } else {
#pragma unroll
      for (int e = 0; e < VPL; ++e) v[u][e] = 0.f;
    }
  }
  const int nv = sq.len_vis > 0 ? static_cast<int>(both & 0xffffu) : 0;
  const int nt = static_cast<int>(both >> 16);
  if (nv > 16 || nt > 16 || min(nv, NV1) > gv || min(nt, 4) > gt) {   // more pieces than guessed (or than this path holds)
    merge_row<D>(P, layer, si, head, sq, lane, -1);
    return;
  }
  const bool mine = lane < 16 ? lane < nv : lane - 16 < nt;
  if (!mine) my_ml = make_float2(-INFINITY, 0.f);
  float mmax = my_ml.x;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, o));
  const float my_w = my_ml.y > 0.f ? exp2f(my_ml.x - mmax) : 0.f;   // (an empty partial counts for nothing)
  float lsum = my_ml.y * my_w;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
  float acc[VPL];
#pragma unroll
  for (int e = 0; e < VPL; ++e) acc[e] = 0.f;
#pragma unroll
  for (int u = 0; u < NV1 + 4; ++u) {
    const float w = __shfl_sync(0xffffffffu, my_w, u < NV1 ? u : 16 + u - NV1);   // lanes 0..15: visual slots, 16..: text slots
    if (w > 0.f) {
#pragma unroll
      for (int e = 0; e < VPL; ++e) acc[e] = fmaf(v[u][e], w, acc[e]);
    }
  }
  // rows beyond the first round's (visual rows past NV1, text rows past four): the rest of a stream
  // in one more round of loads
#pragma unroll 1
  for (int t = (NV1 >= 16 ? 1 : 0); t < 2; ++t) {
    const int n = t ? nt : nv, first = t ? 4 : NV1;
    if (n <= first) continue;
    float r[12][VPL];
#pragma unroll
    for (int u = 0; u < 12; ++u) {
      const int s = first + u;
      const float* src = P.part_acc + ((base + (t ? S : 0) + (s < n ? s : 0)) * P.hq + head) * D + lane * VPL;
      if (VPL == 4) {
        const float4 a = __ldcg(reinterpret_cast<const float4*>(src));
        r[u][0] = a.x, r[u][1] = a.y, r[u][2 % VPL] = a.z, r[u][3 % VPL] = a.w;
      } else {
        const float2 a = __ldcg(reinterpret_cast<const float2*>(src));
        r[u][0] = a.x, r[u][1] = a.y;
      }
    }
#pragma unroll
    for (int u = 0; u < 12; ++u) {
      const int s = first + u;
      const float w = __shfl_sync(0xffffffffu, my_w, (t ? 16 : 0) + (s & 15));
      if (s < n && w > 0.f) {
#pragma unroll
        for (int e = 0; e < VPL; ++e) acc[e] = fmaf(r[u][e], w, acc[e]);
      }
    }
  }
  const float inv = 1.f / lsum;
  const size_t orow = ((static_cast<size_t>(layer) * P.n_seqs + si) * P.hq + head);
  uint16_t* dst = P.out + orow * D + lane * VPL;
  if (VPL == 4) {
    uint2 o;
    o.x = f32_to_bf16_rne(acc[0] * inv) | (static_cast<uint32_t>(f32_to_bf16_rne(acc[1] * inv)) << 16);
    o.y = f32_to_bf16_rne(acc[2 % VPL] * inv) | (static_cast<uint32_t>(f32_to_bf16_rne(acc[3 % VPL] * inv)) << 16);
    *reinterpret_cast<uint2*>(dst) = o;
  } else {
    const uint32_t o = f32_to_bf16_rne(acc[0] * inv) | (static_cast<uint32_t>(f32_to_bf16_rne(acc[1] * inv)) << 16);
    *reinterpret_cast<uint32_t*>(dst) = o;
  }
  if (P.lse != nullptr && lane == 0) P.lse[orow] = (mmax + log2f(lsum)) * 0.6931471805599453f;
}

template <int D>
constexpr int attend_smem_bytes() {
  return kWarps * kRing * kPage * D * 2 + kWarps * kCtxSlots * static_cast<int>(sizeof(WarpCtx<D>));
}

}  // namespace

// ------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------

cudaError_t configure_kernels(int* attend_smem) {
  cudaError_t e = cudaFuncSetAttribute(attend_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       attend_smem_bytes<128>());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, attend_smem_bytes<128>());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, attend_smem_bytes<64>());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, attend_smem_bytes<64>());
  if (attend_smem) *attend_smem = attend_smem_bytes<128>();
  return e;
}

cudaError_t launch_setup(const Params& p, const StepInline* inl, cudaStream_t stream) {
  constexpr int kBlock = 256;
  const int n_house = (max(max(p.n_patches, p.n_layers), p.n_seqs * 8) + kBlock - 1) / kBlock;
  const int blocks = p.n_pos * p.n_seqs + n_house + (p.fused_append ? p.n_seqs * p.n_layers : 0);
  static const StepInline kNone{};
  return launch_pdl(setup_kernel, dim3(blocks), dim3(kBlock), 0, stream, p, inl ? *inl : kNone);
}

cudaError_t launch_plan(const Params& p, const LaunchList& list, int n_launches, cudaStream_t stream) {
  if (n_launches <= 0) return cudaSuccess;
  return launch_pdl(plan_kernel, dim3(kPlanWorkers / 128, n_launches), dim3(128), 0, stream, p, list);
}

cudaError_t launch_append(const Params& p, cudaStream_t stream) {
  dim3 grid(p.n_seqs, p.layer_end - p.layer_begin);
  return launch_pdl(append_kernel, grid, dim3(128), 0, stream, p);
}

cudaError_t launch_attend(const Params& p, int n_sms, cudaStream_t stream) {
  const int n_items = p.item_end - p.item_begin;
  if (!p.part_static && n_items <= 0) return cudaSuccess;
  // static ranges: worker w is warp w / grid of CTA w % grid, so a launch with few workers still uses every SM
  const int grid = min(n_sms, ((p.part_static ? p.part_workers : n_items) + kWarps - 1) / kWarps);
  if (p.d == 128) {
    if (p.part_static)
      return launch_pdl(attend_kernel<128, true>, dim3(grid), dim3(kThreads), attend_smem_bytes<128>(), stream, p);
    return launch_pdl(attend_kernel<128, false>, dim3(grid), dim3(kThreads), attend_smem_bytes<128>(), stream, p);
  }
  if (p.part_static)
    return launch_pdl(attend_kernel<64, true>, dim3(grid), dim3(kThreads), attend_smem_bytes<64>(), stream, p);
  return launch_pdl(attend_kernel<64, false>, dim3(grid), dim3(kThreads), attend_smem_bytes<64>(), stream, p);
}

cudaError_t launch_merge(const Params& p, cudaStream_t stream) {
  const int n = (p.layer_end - p.layer_begin) * p.n_seqs * p.hq;
  if (n <= 0) return cudaSuccess;
  const int warps_per_block = 8;
  const int blocks = (n + warps_per_block - 1) / warps_per_block;
  const dim3 grid(blocks), block(warps_per_block * 32);
  // the one-round path needs the recorded piece counts of the static partition and no extra key
  const bool one_round = p.part_static && p.extra_key_leader < 0 && p.slots_per_stream >= 4;
  if (p.d == 128) {
    if (!one_round) return launch_pdl(merge_kernel<128, 0>, grid, block, 0, stream, p);
    if (p.merge_wide) return launch_pdl(merge_kernel<128, 16>, grid, block, 0, stream, p);
    return launch_pdl(merge_kernel<128, 4>, grid, block, 0, stream, p);
  }
  if (!one_round) return launch_pdl(merge_kernel<64, 0>, grid, block, 0, stream, p);
  if (p.merge_wide) return launch_pdl(merge_kernel<64, 16>, grid, block, 0, stream, p);
  return launch_pdl(merge_kernel<64, 4>, grid, block, 0, stream, p);
}

cudaError_t launch_prefill_scatter(const Params& p, const int32_t* tok_seq, const int32_t* tok_stream,
                                   const int32_t* tok_ord, int32_t n_tokens, int32_t tok_stride,
                                   int32_t tok_offset, cudaStream_t stream) {
  if (n_tokens <= 0) return cudaSuccess;
  dim3 grid(n_tokens, p.n_layers);
  prefill_scatter_kernel<<<grid, 128, 0, stream>>>(p, tok_seq, tok_stream, tok_ord, tok_stride, tok_offset);
  return cudaGetLastError();
}

}  // namespace qc
