// Split-KV partial attention for grouped-query attention (several query heads per KV head).
//
// With a query group of g heads the sweep over one KV head's keys does g times the arithmetic
// of multi-head attention on the same bytes (about g flops per byte), which the fp32 ALUs
// cannot sustain at HBM speed; the query-group tile is a small dense contraction, so it runs
// on the tensor cores:
//
//   S^T[16 keys x 8 heads] = K[16 keys x D] . Q^T[D x 8 heads]          (D/16 mma.m16n8k16)
//   O^T[D x 8 heads]      += V^T[D x 16 keys] . P^T[16 keys x 8 heads]   (D/16 mma.m16n8k16)
//
// Keys are the M dimension, so the group (padded to 8) is the N dimension and nothing but
// the padding 7 -> 8 is wasted.  The score tile comes out with keys along lane groups; an
// 8x8 register transpose (movmatrix) turns the bf16 weights into the B operand of the second
// product.  K/V page tiles arrive through a tensor map with the 128-byte swizzle, so the
// ldmatrix reads of both products (plain for K, transposed for V) are free of bank conflicts.
// Everything else is the structure of the multi-head kernel: persistent CTAs, each warp an
// independent worker with its own tile ring, online softmax in the log2 domain, fp32
// accumulation, partial (m, l, acc) per query head written for the merge kernel.
//
// Softmax weights are rounded to bf16 for the second product (the sum l uses the unrounded
// fp32 weights); accumulators stay fp32.

#include "qc_device.cuh"

namespace qc {
namespace {

constexpr int kRingTc = 2;

struct TcCtx {
  ItemPages ip;
};

// Byte offset of 16-byte chunk `chunk` (0 .. D/8-1) of row `row` inside a swizzled tile:
// the tile is stored as column halves of 64 elements, each [16 rows][128 bytes], with the
// chunk index inside a 128-byte row XORed with (row & 7).
template <int D>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  if (D == 128) return ((chunk >> 3) << 11) + (row << 7) + (((chunk & 7) ^ (row & 7)) << 4);
  return (row << 7) + ((chunk ^ (row & 7)) << 4);
}

// One item: NQ query groups score the K tiles, NV value streams are accumulated.
// NQ == 1: every consumer shares the weights; NQ == NV: consumer x has its own queries.
// MODE 1 (one query group, one consumer) also stores the scaled scores in the logit cache; MODE 2
// takes them from there instead of reading K tiles (the ring then carries V tiles only).
// SKIP (shared weights only): the consumers named in the item's skip_new mask leave out the
// stream's last key (the step's new token): they get a copy of the weights with that key's set
// to zero and their own sums.
// FOLD: the item may end its layer's text stream under the folded append (the new token's rows come
// from the step's inputs).  Launches without the folded append use the instantiation without it,
// whose page loop then carries none of this (with it in every instantiation the one-launch step was
// 3.5 % slower); under the folded append every single-consumer item of a launch takes this one
// (sending only the items that end a stream here made the workers alternate between two copies of
// the loop: 1.20 against 1.09 ms per step at config 2).
template <int D, int NQ, int NV, int MODE = 0, bool SKIP = false, bool FOLD = false>
__device__ __forceinline__ void process_item_tc(WorkerState& st, const TcCtx* ctx, uint32_t ring, uint64_t* full,
                                                const Params& P, int lane) {
  constexpr int KS = D / 16;    // k-steps of the score product = m-tiles of the value product
  auto ctx_of = [ctx](int k) -> const ItemPages& { return ctx[k % kCtxSlots].ip; };
  const Item& it = ctx[st.cons_k % kCtxSlots].ip.item;
  const int g = lane >> 2, t = lane & 3;
  const int n_heads = it.n_heads;

  // ---- query fragments (B operand of the score product): head g, d = 16 kk + 2t (+8)
  uint32_t qb[NQ][KS][2];
#pragma unroll
  for (int x = 0; x < NQ; ++x) {
    const bool cached = (it.flags >> (kFlagCachedShift + x)) & 1;
    const uint16_t* base =
        cached ? P.qcache + ((static_cast<size_t>(it.q_layer[x]) * P.max_seqs + it.seq_id) * P.hq + it.head) * D
               : P.q + ((static_cast<size_t>(it.q_layer[x]) * P.n_seqs + it.seq_idx) * P.hq + it.head) * D;
    const uint32_t* row = reinterpret_cast<const uint32_t*>(base + static_cast<size_t>(g) * D) + t;
    const bool live = g < n_heads;
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
      qb[x][kk][0] = live ? __ldg(row + 8 * kk) : 0u;
      qb[x][kk][1] = live ? __ldg(row + 8 * kk + 4) : 0u;
    }
  }

  float m[NQ][2], l[NQ][2];      // running max / partial sum of heads 2t and 2t + 1
  float o[NV][KS][4];
#pragma unroll
  for (int x = 0; x < NQ; ++x) m[x][0] = m[x][1] = -INFINITY, l[x][0] = l[x][1] = 0.f;
#pragma unroll
  for (int v = 0; v < NV; ++v)
#pragma unroll
    for (int i = 0; i < KS; ++i) o[v][i][0] = o[v][i][1] = o[v][i][2] = o[v][i][3] = 0.f;

  const int n_pages = it.n_pages;
  const int n_valid_last = it.n_valid_last;
  const bool skip_here = SKIP && (it.flags & kFlagStreamEnd);
  const uint32_t skip_mask = SKIP ? it.skip_new : 0u;
  float l_skip[2] = {0.f, 0.f};
  // ldmatrix lane roles
  const int lrow = lane & 7, lmat = lane >> 3;
  const int k_row = lrow + ((lmat & 1) << 3), k_chunk = lmat >> 1;    // K: matrices (keys lo/hi) x (chunk +0/+1)
  const int v_row = lrow + ((lmat >> 1) << 3), v_chunk = lmat & 1;    // V: matrices (chunk +0/+1) x (keys lo/hi)

  // Logit cache rows of heads 2t and 2t + 1 at this item's first key (lane (g, t) holds the scores
  // of keys g and g + 8 for those two heads).
  float* lg0 = nullptr;
  float* lg1 = nullptr;
  float lg_next[4] = {0.f, 0.f, 0.f, 0.f};
  const bool h0 = 2 * t < n_heads, h1 = 2 * t + 1 < n_heads;
  if (MODE != 0) {
    lg0 = logit_row(P, it.stream, it.seq_id, it.head + (h0 ? 2 * t : 0)) + it.first_page * kPage;
    lg1 = logit_row(P, it.stream, it.seq_id, it.head + (h1 ? 2 * t + 1 : 0)) + it.first_page * kPage;
    if (MODE == 2) {
      lg_next[0] = lg0[g], lg_next[1] = lg1[g], lg_next[2] = lg0[g + 8], lg_next[3] = lg1[g + 8];
    }
  }

  constexpr bool kMayFold = FOLD || SKIP;
  const int new_pg = (kMayFold && holds_new_token(P, it, n_pages - 1)) ? n_pages - 1 : -1;   // folded append: page of the new token
  for (int pg = 0; pg < n_pages && !st.dead; ++pg) {
    const int nvalid = (pg == n_pages - 1) ? n_valid_last : kPage;
    uint32_t pb[NQ][2];
    uint32_t pb_skip[2] = {0u, 0u};   // the weights without the new token (SKIP, last page only)
    const bool skip_page = SKIP && skip_here && pg == n_pages - 1;
    // ---- K tile: scores of 16 keys for 8 heads
    {
      float s[NQ][4];
      if (MODE == 2) {
        // the scaled scores of this page from the logit cache; the next page's are requested now
#pragma unroll
        for (int i = 0; i < 4; ++i) s[0][i] = lg_next[i];
        if (pg + 1 < n_pages) {
          const int o = (pg + 1) * kPage + g;
          lg_next[0] = lg0[o], lg_next[1] = lg1[o], lg_next[2] = lg0[o + 8], lg_next[3] = lg1[o + 8];
        }
      } else {
        const uint32_t tile = wait_tile<D>(st, ring, full, P, lane);
        if (st.dead) break;
        if (kMayFold && pg == new_pg) {
          // the new token's k row comes from the step's input: into the (swizzled) tile, and into the pool
          const ItemPages& ip = ctx[st.cons_k % kCtxSlots].ip;
          if (lane < D / 8) {
            const uint4 val = ip.new_k[lane];
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(tile + swz<D>(nvalid - 1, lane)), "r"(val.x),
                         "r"(val.y), "r"(val.z), "r"(val.w)
                         : "memory");
            const int pid = ip.pages[0][pg];
            if (static_cast<uint32_t>(pid) < static_cast<uint64_t>(P.n_pool_pages))
              reinterpret_cast<uint4*>(P.pool + ((static_cast<size_t>(pid) * P.hkv + ip.kv_head) * kPage + (nvalid - 1)) * D)[lane] = val;
          }
          // an ordinary layer's queries go to the Q Cache
          if (it.q_layer[0] == it.k_layer && !((it.flags >> kFlagCachedShift) & 1) && (P.layer_flags[it.k_layer] & kLayerWritesQCache)) {
            const uint4* src = reinterpret_cast<const uint4*>(
                P.q + ((static_cast<size_t>(it.k_layer) * P.n_seqs + it.seq_idx) * P.hq + it.head) * D);
            uint4* dst = reinterpret_cast<uint4*>(
                P.qcache + ((static_cast<size_t>(it.k_layer) * P.max_seqs + it.seq_id) * P.hq + it.head) * D);
            for (int e = lane; e < n_heads * (D / 8); e += 32) dst[e] = src[e];
          }
          __syncwarp();
        }
#pragma unroll
        for (int x = 0; x < NQ; ++x) s[x][0] = s[x][1] = s[x][2] = s[x][3] = 0.f;
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) {
          uint32_t a[4];
          ldmatrix_x4(a, tile + swz<D>(k_row, 2 * kk + k_chunk));
#pragma unroll
          for (int x = 0; x < NQ; ++x) mma_bf16_16816(s[x], a, qb[x][kk]);
        }
        release_tile<kRingTc>(st);
        fill_ring<D, kRingTc, true>(st, ctx_of, ring, full, P, lane);
#pragma unroll
        for (int x = 0; x < NQ; ++x) {
#pragma unroll
          for (int i = 0; i < 4; ++i) s[x][i] *= P.scale_log2;
        }
      }
      const bool ok_lo = g < nvalid, ok_hi = g + 8 < nvalid;
      if (MODE == 1) {
        const int o = pg * kPage + g;
        if (ok_lo && h0) lg0[o] = s[0][0];
        if (ok_lo && h1) lg1[o] = s[0][1];
        if (ok_hi && h0) lg0[o + 8] = s[0][2];
        if (ok_hi && h1) lg1[o + 8] = s[0][3];
      }
#pragma unroll
      for (int x = 0; x < NQ; ++x) {
        const float s0 = ok_lo ? s[x][0] : -INFINITY;   // key g,     head 2t
        const float s1 = ok_lo ? s[x][1] : -INFINITY;   // key g,     head 2t + 1
        const float s2 = ok_hi ? s[x][2] : -INFINITY;   // key g + 8, head 2t
        const float s3 = ok_hi ? s[x][3] : -INFINITY;   // key g + 8, head 2t + 1
        float t0 = fmaxf(s0, s2), t1 = fmaxf(s1, s3);
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
          t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, off));
          t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, off));
        }
        const float m0 = fmaxf(m[x][0], t0), m1 = fmaxf(m[x][1], t1);   // finite: key 0 is always valid
        const float c0 = exp2f(m[x][0] - m0), c1 = exp2f(m[x][1] - m1);
        const float p0 = exp2f(s0 - m0), p1 = exp2f(s1 - m1), p2 = exp2f(s2 - m0), p3 = exp2f(s3 - m1);
        l[x][0] = fmaf(l[x][0], c0, p0 + p2);
        l[x][1] = fmaf(l[x][1], c1, p1 + p3);
        m[x][0] = m0;
        m[x][1] = m1;
        // weights as the B operand of the value product: keys 2t, 2t+1 (+8), head g
        pb[x][0] = movmatrix_trans(pack_bf16x2(p0, p1));
        pb[x][1] = movmatrix_trans(pack_bf16x2(p2, p3));
        if (SKIP) {
          float q0 = p0, q1 = p1, q2 = p2, q3 = p3;
          if (skip_page) {
            const int r_new = nvalid - 1;
            if (g == r_new) q0 = q1 = 0.f;
            if (g + 8 == r_new) q2 = q3 = 0.f;
            pb_skip[0] = movmatrix_trans(pack_bf16x2(q0, q1));
            pb_skip[1] = movmatrix_trans(pack_bf16x2(q2, q3));
          }
          l_skip[0] = fmaf(l_skip[0], c0, q0 + q2);
          l_skip[1] = fmaf(l_skip[1], c1, q1 + q3);
        }
        if (__any_sync(0xffffffffu, c0 != 1.f || c1 != 1.f)) {
#pragma unroll
          for (int v = 0; v < NV; ++v) {
            if (NQ == 1 || v == x) {
#pragma unroll
              for (int i = 0; i < KS; ++i) {
                o[v][i][0] *= c0;
                o[v][i][1] *= c1;
                o[v][i][2] *= c0;
                o[v][i][3] *= c1;
              }
            }
          }
        }
      }
    }
    // ---- V tiles: O^T += V^T . P^T for each consumer
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const uint32_t tile = wait_tile<D>(st, ring, full, P, lane);
      if (st.dead) break;
      const bool skipping = SKIP && skip_page && ((skip_mask >> v) & 1u);
      const int nvalid_v = skipping ? nvalid - 1 : nvalid;
      if (kMayFold && pg == new_pg && !skipping) {
        // this consumer's new v row, likewise
        const ItemPages& ip = ctx[st.cons_k % kCtxSlots].ip;
        if (lane < D / 8) {
          const uint4 val = v == first_taker(it)
                                ? ip.new_v[lane]
                                : reinterpret_cast<const uint4*>(
                                      P.v + ((static_cast<size_t>(it.v_layer[v]) * P.n_seqs + it.seq_idx) * P.hkv + ip.kv_head) * D)[lane];
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(tile + swz<D>(nvalid - 1, lane)), "r"(val.x),
                       "r"(val.y), "r"(val.z), "r"(val.w)
                       : "memory");
          const int pid = ip.pages[1 + v][pg];
          if (static_cast<uint32_t>(pid) < static_cast<uint64_t>(P.n_pool_pages))
            reinterpret_cast<uint4*>(P.pool + ((static_cast<size_t>(pid) * P.hkv + ip.kv_head) * kPage + (nvalid - 1)) * D)[lane] = val;
        }
        fence_proxy_async();
        __syncwarp();
      }
      if (nvalid_v < kPage) {
        // rows past the end of the stream hold whatever the pool held: clear them, since a
        // zero weight does not cancel a NaN or an infinity
        const int n_seg = (kPage - nvalid_v) * (D / 64);
        for (int e = lane; e < n_seg * 8; e += 32) {
          const int seg = e >> 3, half = seg / (kPage - nvalid_v), row = nvalid_v + seg % (kPage - nvalid_v);
          asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(tile + (half << 11) + (row << 7) + ((e & 7) << 4)),
                       "r"(0u)
                       : "memory");
        }
        fence_proxy_async();   // these generic-proxy writes precede the slot's next asynchronous refill
        __syncwarp();
      }
#pragma unroll
      for (int i = 0; i < KS; ++i) {
        uint32_t a[4];
        ldmatrix_x4_trans(a, tile + swz<D>(v_row, 2 * i + v_chunk));
        if (skipping) mma_bf16_16816(o[v][i], a, pb_skip);
        else mma_bf16_16816(o[v][i], a, pb[NQ == 1 ? 0 : v]);
      }
      release_tile<kRingTc>(st);
      fill_ring<D, kRingTc, true>(st, ctx_of, ring, full, P, lane);
    }
  }
  if (st.dead) return;

  // ---- partial results.  Lane (g, t) holds O^T[d = 16 i + g (+8)][heads 2t, 2t + 1].
#pragma unroll
  for (int x = 0; x < NQ; ++x) {
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      l[x][0] += __shfl_xor_sync(0xffffffffu, l[x][0], off);
      l[x][1] += __shfl_xor_sync(0xffffffffu, l[x][1], off);
    }
  }
  if (SKIP) {
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      l_skip[0] += __shfl_xor_sync(0xffffffffu, l_skip[0], off);
      l_skip[1] += __shfl_xor_sync(0xffffffffu, l_skip[1], off);
    }
  }
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const size_t row0 =
        ((static_cast<size_t>(it.v_layer[v]) * P.max_seqs + it.seq_idx) * P.max_slots + it.slot) * P.hq + it.head +
        2 * t;
    constexpr int xq_shared = 0;
    const int xq = (NQ == 1) ? xq_shared : v;
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      if (2 * t + hh < n_heads) {
        float* dst = P.part_acc + (row0 + hh) * D + g;
#pragma unroll
        for (int i = 0; i < KS; ++i) {
          dst[16 * i] = o[v][i][hh];
          dst[16 * i + 8] = o[v][i][2 + hh];
        }
        const bool skipped = SKIP && ((skip_mask >> v) & 1u);
        if (g == 0) P.part_ml[row0 + hh] = make_float2(m[xq][hh], skipped ? l_skip[hh] : l[xq][hh]);
      }
    }
  }
  finish_rows<D>(P, ctx[st.cons_k % kCtxSlots].ip, lane);
}

// A worker's life: take items (claimed from the list, or the pieces of its static ranges), keep
// the tile ring full across item boundaries, process each item.  While item k is processed the
// ring already fetches tiles of item k + 1 and the context of item k + 2 (descriptor, page ids)
// arrives by asynchronous copies.
template <int D, bool STATIC>
__device__ __forceinline__ void attend_tc_worker(const Params& P, TcCtx* ctx, uint32_t ring, uint64_t* full,
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
    const bool early_tiles = P.fold_append || !(first.stream == 0 && (first.flags & kFlagStreamEnd) && first.n_pages <= kRingTc);
    if (early_tiles) fill_ring<D, kRingTc, true>(st, ctx_of, ring, full, P, lane);
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
    const bool early_tiles = P.fold_append || !(first.stream == 0 && (first.flags & kFlagStreamEnd) && first.n_pages <= kRingTc);
    if (early_tiles) fill_ring<D, kRingTc, true>(st, ctx_of, ring, full, P, lane);
  }
  if (STATIC) {
    pdl_wait();
    pdl_launch_dependents();
  }
  // ---- this layer's inputs; the rest of the first tiles; the second item's context while they fly
  begin_new_rows(ctx[0].ip, P, first, lane, D);
  fill_ring<D, kRingTc, true>(st, ctx_of, ring, full, P, lane);
  if (STATIC) record_row_slots(P, first, lane);
  if (!STATIC) issued = claim_issue(P, lane);
  bool more = take();
  if (more) {
    begin_item_pages(ctx[1].ip, P, it, lane);
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
        begin_new_rows(ctx[(k + 2) % kCtxSlots].ip, P, it, lane, D);
        if (STATIC) record_row_slots(P, it, lane);
        pending = true;
      }
    }
    if (!STATIC && more) issued = claim_issue(P, lane);   // answered by the time the next item starts
    if (nc == 1 && (cur.flags & kFlagReadLogits)) process_item_tc<D, 1, 1, 2>(st, ctx, ring, full, P, lane);
    else if (nc == 1 && (cur.flags & kFlagWriteLogits)) process_item_tc<D, 1, 1, 1>(st, ctx, ring, full, P, lane);
    else if (shared && cur.skip_new) {
      if (nc == 1) process_item_tc<D, 1, 1, 0, true>(st, ctx, ring, full, P, lane);
      else if (nc == 2) process_item_tc<D, 1, 2, 0, true>(st, ctx, ring, full, P, lane);
      else if (nc == 3) process_item_tc<D, 1, 3, 0, true>(st, ctx, ring, full, P, lane);
      else process_item_tc<D, 1, 4, 0, true>(st, ctx, ring, full, P, lane);
    }
    else if (nc == 1 && P.fold_append) process_item_tc<D, 1, 1, 0, false, true>(st, ctx, ring, full, P, lane);   // (one code path per launch)
    else if (nc == 1) process_item_tc<D, 1, 1>(st, ctx, ring, full, P, lane);
    else if (shared && nc == 2) process_item_tc<D, 1, 2>(st, ctx, ring, full, P, lane);
    else if (shared && nc == 3) process_item_tc<D, 1, 3>(st, ctx, ring, full, P, lane);
    else if (shared) process_item_tc<D, 1, 4>(st, ctx, ring, full, P, lane);
    else process_item_tc<D, 2, 2>(st, ctx, ring, full, P, lane);   // own-query sweeps feed at most two layers here
    if (st.dead) break;
    if (pending) {   // the context of item k + 2 has had this item's time to arrive
      cp_async_wait_all();
      __syncwarp();
      st.n_my = k + 3;
      pending = false;
    }
    st.cons_k = k + 1;
    fill_ring<D, kRingTc, true>(st, ctx_of, ring, full, P, lane);
  }
  if (st.dead) {
    cp_async_wait_all();
    drain_ring<kRingTc>(st, full, P.debug_drop_tile ? kDebugSpinLimit : kSpinLimit);
  }
}

template <int D, bool STATIC>
__global__ void __launch_bounds__(kThreads, 1) attend_tc_kernel(const __grid_constant__ Params P) {
  constexpr uint32_t kTile = kPage * D * 2;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_all[kWarps][kRingTc];
  __shared__ __align__(16) RangeCursor cursors[kWarps];
  __shared__ __align__(16) int32_t stages[kWarps][12];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // swizzled tiles must sit on 1024-byte boundaries
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t ring = base + static_cast<uint32_t>(warp) * kRingTc * kTile;
  TcCtx* ctx = reinterpret_cast<TcCtx*>(base_ptr + static_cast<size_t>(kWarps) * kRingTc * kTile) + warp * kCtxSlots;
  uint64_t* full = full_all[warp];

  if (lane == 0) {
    for (int s = 0; s < kRingTc; ++s) mbar_init(&full[s], 1);
    fence_mbar_init();
  }
  __syncthreads();

  attend_tc_worker<D, STATIC>(P, ctx, ring, full, &cursors[warp], stages[warp], worker_index(P, warp, kWarps), lane);
}

template <int D>
constexpr int attend_tc_smem_bytes() {
  return 1024 + kWarps * kRingTc * kPage * D * 2 + kWarps * kCtxSlots * static_cast<int>(sizeof(TcCtx));
}

}  // namespace

cudaError_t configure_kernels_tc(int* attend_smem) {
  cudaError_t e = cudaFuncSetAttribute(attend_tc_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       attend_tc_smem_bytes<128>());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_tc_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           attend_tc_smem_bytes<128>());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_tc_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           attend_tc_smem_bytes<64>());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_tc_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           attend_tc_smem_bytes<64>());
  if (attend_smem) *attend_smem = attend_tc_smem_bytes<128>();
  return e;
}

cudaError_t launch_attend_tc(const Params& p, int n_sms, cudaStream_t stream) {
  const int n_items = p.item_end - p.item_begin;
  if (!p.part_static && n_items <= 0) return cudaSuccess;
  const int grid = min(n_sms, ((p.part_static ? p.part_workers : n_items) + kWarps - 1) / kWarps);
  if (p.d == 128) {
    if (p.part_static)
      return launch_pdl(attend_tc_kernel<128, true>, dim3(grid), dim3(kThreads), attend_tc_smem_bytes<128>(), stream, p);
    return launch_pdl(attend_tc_kernel<128, false>, dim3(grid), dim3(kThreads), attend_tc_smem_bytes<128>(), stream, p);
  }
  if (p.part_static)
    return launch_pdl(attend_tc_kernel<64, true>, dim3(grid), dim3(kThreads), attend_tc_smem_bytes<64>(), stream, p);
  return launch_pdl(attend_tc_kernel<64, false>, dim3(grid), dim3(kThreads), attend_tc_smem_bytes<64>(), stream, p);
}

}  // namespace qc
