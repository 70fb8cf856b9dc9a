// Device-side helpers shared by the attention kernels: PTX wrappers (mbarrier, bulk and
// tensor-map asynchronous copies, ldmatrix / mma), bf16 conversion, and the per-warp tile ring
// through which a warp streams K/V page tiles from the pool.
#pragma once

#include "qc_internal.h"

#include <math.h>

#include <utility>

namespace qc {
namespace {

constexpr int kWarps = kAttendWarps;
constexpr int kThreads = kWarps * 32;
constexpr uint32_t kSpinLimit = 1u << 22; // bounded mbarrier wait

// values of the device error word (QC_ERR_* of the public header)
constexpr int kErrTimeout = 6;
constexpr int kErrBadPage = 7;
constexpr int kErrPlan = 8;   // a work range did not fit the limits the host planned it for
constexpr uint32_t kDebugSpinLimit = 1u << 12;   // wait limit under the test hook that drops a tile copy

// ------------------------------------------------------------------------------------------
// PTX helpers
// ------------------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok;
}
// 1-D bulk copy global -> this CTA's shared memory, completion counted on an mbarrier.
// Source, destination and size are multiples of 16 bytes by construction (whole page tiles).
// K/V tiles are read once per step: they are fetched with the evict-first L2 policy, so that the
// stream of tiles does not push the page tables, the queries and the partial rows out of the L2.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
  return policy;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint64_t* bar,
                                         uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          dst_smem),
      "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
// 2-D tensor-map copy global -> this CTA's shared memory (the map applies the 128-byte
// swizzle).  x is a multiple of 8 elements (16 bytes) by construction: 0 or 64.
__device__ __forceinline__ void tensor_g2s_2d(uint32_t dst_smem, const void* tmap, int32_t x, int32_t y,
                                              uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::
          "r"(dst_smem),
      "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
// the same with an L2 cache policy
__device__ __forceinline__ void tensor_g2s_2d(uint32_t dst_smem, const void* tmap, int32_t x, int32_t y,
                                              uint64_t* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, "
      "%3}], [%4], %5;" ::"r"(dst_smem),
      "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}

// Asynchronous global -> shared copies of 4 or 16 bytes (no registers held while in flight);
// cp_async_wait_all() waits for the calling thread's own copies.
__device__ __forceinline__ void cp_async_4(void* dst_smem, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_16(void* dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Programmatic dependent launch: the kernels of a decode step are launched back to back with
// the programmatic-serialization attribute.  Each one does the set-up that may run early, waits
// for its predecessor to have completed (and its writes to be visible), and only then lets its
// successor start getting scheduled.
// Every kernel of the chain executes its wait BEFORE it lets its successor start, so when a kernel
// starts running, the kernel before its predecessor -- and by induction everything earlier in
// the stream -- has completed: what a kernel does ahead of its own wait may read anything that
// was written two or more launches back (the attention kernels plan their first work items there,
// from the launch plan, the step descriptors and the page tables).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launch with the programmatic-serialization attribute (plain stream order if the predecessor
// in the stream is not a kernel).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
// 8x8 transpose of 16-bit elements held one row-pair per lane (row lane/4, columns 2*(lane%4)..)
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
// two fp32 -> packed bf16x2 (round to nearest even); `lo` lands in the low half
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

__device__ __forceinline__ void bf16x8_to_f32(const uint4& r, float* f) {
  f[0] = __uint_as_float(r.x << 16);
  f[1] = __uint_as_float(r.x & 0xffff0000u);
  f[2] = __uint_as_float(r.y << 16);
  f[3] = __uint_as_float(r.y & 0xffff0000u);
  f[4] = __uint_as_float(r.z << 16);
  f[5] = __uint_as_float(r.z & 0xffff0000u);
  f[6] = __uint_as_float(r.w << 16);
  f[7] = __uint_as_float(r.w & 0xffff0000u);
}

__device__ __forceinline__ uint16_t f32_to_bf16_rne(float x) {
  uint32_t u = __float_as_uint(x);
  if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<uint16_t>((u >> 16) | 0x40);   // NaN
  u += 0x7fffu + ((u >> 16) & 1u);
  return static_cast<uint16_t>(u >> 16);
}

// Record an error: the device word (largest code wins) and its mirror in mapped host memory.
__device__ __forceinline__ void report_error(int32_t* err, int32_t* err_host, int code) {
  atomicMax(err, code);
  if (err_host != nullptr) {
    *reinterpret_cast<volatile int32_t*>(err_host) = code;
    __threadfence_system();
  }
}

__device__ __forceinline__ size_t table_row(const Params& P, int layer, int stream, int seq_id) {
  return ((static_cast<size_t>(layer) * 4 + stream) * P.max_seqs + seq_id) * P.max_pages;
}

// ------------------------------------------------------------------------------------------
// per-warp tile ring
// ------------------------------------------------------------------------------------------
//
// A warp owns RING tile slots in shared memory and one mbarrier per slot.  Lane 0 issues the
// copies of the K tile and the V tiles of each page of the warp's current item (and of the
// next one, so the ring never drains at an item boundary; an item that takes its scores from
// the logit cache has no K tiles); all lanes wait on a slot's
// barrier before reading it.  Every wait is bounded: when it runs out the worker records the
// error, stops fetching, lets the copies in flight land (again bounded) and leaves.

// Item descriptor and page ids of one item, as the ring needs them.
struct ItemPages {
  Item item;
  StepSeq sq;          // the item's sequence
  int32_t kv_head;     // item.head / group
  int32_t pad[3];
  uint4 new_k[16];     // folded append: the new token's k row of the item's K layer and the v row of its
  uint4 new_v[16];     // first consumer that takes the new token (fetched with the queries)
  int32_t pages[1 + kMaxCons][kMaxChunkPages];   // [0]: K pages, [1 + x]: V pages of consumer x
};

struct WorkerState {
  int n_my;            // items this worker owns
  int cons_k;          // item being consumed
  int iss_k;           // item being fetched (cons_k or cons_k + 1)
  int iss_page, iss_which;
  int iss_slot, cons_slot;
  uint32_t cons_phase;
  int in_flight;
  bool dead;           // a bounded wait ran out: stop fetching, drain, leave
  bool drop_next;      // test hook: the next tile's copy is left out
};

__device__ __forceinline__ void worker_init(WorkerState& st, int n_my) {
  st.n_my = n_my;
  st.cons_k = st.iss_k = 0;
  st.iss_page = st.iss_which = 0;
  st.iss_slot = st.cons_slot = 0;
  st.cons_phase = 0;
  st.in_flight = 0;
  st.dead = false;
  st.drop_next = false;
}

// Issue the copy of the next tile.  D: head dim; RING: slots; TMAP: copy through the tensor
// map (swizzled tile: two 64-element column halves per row when D == 128) instead of one
// linear 16*D*2-byte bulk copy.  `ctx(k)` returns the ItemPages of the worker's k-th item.
template <int D, int RING, bool TMAP, typename CtxFn>
__device__ __forceinline__ bool issue_one(WorkerState& st, CtxFn ctx, uint32_t ring, uint64_t* full, const Params& P,
                                          int lane) {
  constexpr uint32_t kTile = kPage * D * 2;
  if (st.dead || st.iss_k >= st.n_my || st.iss_k > st.cons_k + 1) return false;
  const ItemPages& c = ctx(st.iss_k);
  const int n_cons = c.item.n_cons;
  if (st.iss_which == 0 && (c.item.flags & kFlagReadLogits)) st.iss_which = 1;   // scores come from the logit cache
  int pid = c.pages[st.iss_which][st.iss_page];
  if (static_cast<uint32_t>(pid) >= static_cast<uint64_t>(P.n_pool_pages)) {   // never read outside the pool
    if (lane == 0) report_error(P.err, P.err_host, kErrBadPage);
    pid = 0;
  }
  if (P.debug_drop_tile && st.drop_next) {
    // test hook: count the tile as in flight without requesting it; its wait will run out
    st.drop_next = false;
  } else if (lane == 0) {
    uint64_t* bar = &full[st.iss_slot];
    const uint32_t dst = ring + st.iss_slot * kTile;
    fence_proxy_async();   // the slot's earlier generic-proxy accesses precede this async write
    mbar_expect_tx(bar, kTile);
    const uint64_t policy = l2_evict_first_policy();
    if (TMAP) {
      const int32_t row = (pid * P.hkv + c.kv_head) * kPage;
      tensor_g2s_2d(dst, &P.tmap, 0, row, bar, policy);
      if (D == 128) tensor_g2s_2d(dst + kTile / 2, &P.tmap, 64, row, bar, policy);
    } else {
      const uint16_t* src = P.pool + (static_cast<size_t>(pid) * P.hkv + c.kv_head) * (kPage * D);
      bulk_g2s(dst, src, kTile, bar, policy);
    }
  }
  st.iss_slot = (st.iss_slot + 1 == RING) ? 0 : st.iss_slot + 1;
  st.in_flight++;
  if (++st.iss_which > n_cons) {
    st.iss_which = 0;
    if (++st.iss_page == c.item.n_pages) {
      st.iss_page = 0;
      st.iss_k++;
    }
  }
  return true;
}

template <int D, int RING, bool TMAP, typename CtxFn>
__device__ __forceinline__ void fill_ring(WorkerState& st, CtxFn ctx, uint32_t ring, uint64_t* full, const Params& P,
                                          int lane) {
  while (st.in_flight < RING) {
    if (!issue_one<D, RING, TMAP>(st, ctx, ring, full, P, lane)) break;
  }
}

// Wait until the oldest tile in flight has landed; returns its shared-memory address.
template <int D>
__device__ __forceinline__ uint32_t wait_tile(WorkerState& st, uint32_t ring, uint64_t* full, const Params& P,
                                              int lane) {
  constexpr uint32_t kTile = kPage * D * 2;
  uint64_t* bar = &full[st.cons_slot];
  uint32_t done = mbar_try_wait(bar, st.cons_phase);
  const uint32_t limit = P.debug_drop_tile ? kDebugSpinLimit : kSpinLimit;
  for (uint32_t spin = 0; !done && spin < limit; ++spin) done = mbar_try_wait(bar, st.cons_phase);
  if (!done) {
    if (lane == 0) report_error(P.err, P.err_host, kErrTimeout);
    st.dead = true;
  }
  return ring + st.cons_slot * kTile;
}

template <int RING>
__device__ __forceinline__ void release_tile(WorkerState& st) {
  __syncwarp();
  st.in_flight--;
  if (++st.cons_slot == RING) {
    st.cons_slot = 0;
    st.cons_phase ^= 1u;
  }
}

// After a failed wait: copies still in flight write into this CTA's shared memory; give them
// a bounded chance to land before the warp leaves.
template <int RING>
__device__ __forceinline__ void drain_ring(WorkerState& st, uint64_t* full, uint32_t limit = kSpinLimit) {
  while (st.in_flight > 0) {
    uint64_t* bar = &full[st.cons_slot];
    uint32_t done = 0;
    for (uint32_t spin = 0; !done && spin < limit; ++spin) done = mbar_try_wait(bar, st.cons_phase);
    st.in_flight--;
    if (++st.cons_slot == RING) {
      st.cons_slot = 0;
      st.cons_phase ^= 1u;
    }
  }
}

// A warp keeps the contexts of three items: the one it consumes, the next one (whose tiles the ring
// already fetches) and the one after, which is being filled by asynchronous copies meanwhile.
constexpr int kCtxSlots = 3;

// Start filling a context slot with an item and the page ids of its K stream and V streams
// (asynchronous copies; cp_async_wait_all() + __syncwarp() completes them).
__device__ __forceinline__ void begin_item_pages(ItemPages& c, const Params& P, const Item& it, int lane) {
  __syncwarp();   // the slot's previous item is no longer read
  if (lane == 0) {
    c.item = it;
    c.kv_head = it.head / P.group;
  }
  if (lane >= 30) cp_async_16(reinterpret_cast<uint4*>(&c.sq) + (lane - 30), reinterpret_cast<const uint4*>(P.seqs + it.seq_idx) + (lane - 30));
  if (lane < it.n_pages) {
    cp_async_4(&c.pages[0][lane], P.table + table_row(P, it.k_layer, it.stream, it.seq_id) + it.first_page + lane);
    for (int x = 0; x < it.n_cons; ++x)
      cp_async_4(&c.pages[1 + x][lane],
                 P.table + table_row(P, it.v_layer[x], 2 + it.stream, it.seq_id) + it.first_page + lane);
  }
}

// Fetch an item's descriptor from the item list.
__device__ __forceinline__ Item load_item(const Params& P, int item_idx) {
  const uint4* ip = reinterpret_cast<const uint4*>(P.items + item_idx);
  uint4 a = __ldg(ip), b = __ldg(ip + 1);
  Item it;
  reinterpret_cast<uint4*>(&it)[0] = a;
  reinterpret_cast<uint4*>(&it)[1] = b;
  return it;
}

// Items of a launch are handed out in list order (heaviest first, so the work left at the end
// comes in small pieces).  A claim is an atomic increment issued by lane 0 whose result is only
// looked at one item later, so its latency never stalls the tile pipeline.
__device__ __forceinline__ int claim_issue(const Params& P, int lane) {
  int idx = 0;
  if (lane == 0) idx = atomicAdd(P.work_counter + P.launch_index, 1);
  return idx;
}
// Where the scaled scores of (stream, sequence, head) start in the logit cache; key j of the stream
// is element j.
__device__ __forceinline__ float* logit_row(const Params& P, int stream, int seq_id, int head) {
  return P.logits + ((static_cast<size_t>(stream) * P.max_seqs + seq_id) * P.hq + head) *
                        (static_cast<size_t>(P.max_pages) * kPage);
}

// Turns the value returned by claim_issue into an item index, or -1 when the list is used up.
__device__ __forceinline__ int claim_take(const Params& P, int issued) {
  const int idx = __shfl_sync(0xffffffffu, issued, 0);
  return idx < P.item_end - P.item_begin ? P.item_begin + idx : -1;
}

// ------------------------------------------------------------------------------------------
// static partition of a launch
// ------------------------------------------------------------------------------------------
//
// The work of a launch is laid out in tiles: plan positions of the launch in order, inside a
// position the listed sequences, inside a sequence the rows (one per query head, or per query
// group with GQA), inside a row its pages, each page worth w tiles (one K tile unless the scores
// come from the logit cache, one V tile per consumer) after a fixed part_row_cost per row (what
// starting and finishing an item costs a worker).  The space of T tiles is cut into ranges of
// part_q tiles; a page belongs to the range its first tile falls into.  Physical worker i takes
// ranges i*part_k .. i*part_k + part_k - 1, which are adjacent, so it walks rows forward from one
// starting point.  The pages of a row that one range owns are one piece: an Item whose partial
// result goes to slot (range - range owning the row's first page) of the row's stream.  The host
// plans part_q so that a range is at least as long as any page (every range between a row's
// first and last owns a page of it: no slot is left unwritten), a piece has at most
// kMaxChunkPages pages and a row at most slots_per_stream pieces; T < 2^31.

struct __align__(16) RangeCursor {
  int32_t r0;        // tile offset of the current row's first page
  int32_t vw_end;    // first tile beyond the current range
  int32_t vw, vw_stop;
  int32_t pos, si, u;
  int32_t row_pages, w;     // pages of the current row; tiles per page of its job
  int32_t page;             // next page of the current row to hand out
  int32_t owner0;           // range that owns the row's first page
  int32_t len, seq_id;      // tokens of the row's stream; its sequence
  int32_t pad[3];
  Job job;
};
static_assert(sizeof(RangeCursor) == 80, "RangeCursor layout");

// What the partition of one launch is made of (the attention kernels take it from their
// parameters, the kernel that plans every launch of a step ahead from its launch list).
struct PartView {
  const PlanJob* plan;
  const StepSeq* seqs;
  int32_t* err;
  int32_t* err_host;
  int32_t pos_begin, pos_end, n_seqs;
  int32_t q, k, vw, row_cost;          // tiles per range, ranges per worker, ranges, fixed tiles per row
  int32_t tp_v, tp_t;                  // pages of the visual / text streams over the listed sequences
  int32_t rows, heads_per_item, group, slots_per_stream;   // rows per (position, sequence); query heads per row
};

__device__ __forceinline__ PartView part_view(const Params& P) {
  PartView V;
  V.plan = P.plan, V.seqs = P.seqs, V.err = P.err, V.err_host = P.err_host;
  V.pos_begin = P.pos_begin, V.pos_end = P.pos_end, V.n_seqs = P.n_seqs;
  V.q = P.part_q, V.k = P.part_k, V.vw = P.part_vw, V.row_cost = P.part_row_cost;
  V.tp_v = P.tp_v, V.tp_t = P.tp_t;
  V.rows = P.heads_per_item_dim, V.heads_per_item = P.heads_per_item, V.group = P.group;
  V.slots_per_stream = P.slots_per_stream;
  return V;
}

__device__ __forceinline__ int job_tiles_per_page(const Job& j) {
  return ((j.flags & kFlagReadLogits) ? 0 : 1) + j.n_cons;
}

// Load the job of plan position c.pos (if it changed) and the sequence c.si into the cursor.
__device__ __forceinline__ void cursor_load_segment(RangeCursor& c, const PartView& V, bool new_pos) {
  if (new_pos) {
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(V.plan + c.pos));
    *reinterpret_cast<uint4*>(&c.job) = raw;
    c.w = job_tiles_per_page(c.job);
  }
  const StepSeq sq = V.seqs[c.si];
  c.len = c.job.stream ? sq.len_vis : sq.len_text;
  c.seq_id = sq.seq_id;
  c.row_pages = (c.len + kPage - 1) / kPage;
}

// Tile offset at which the rows of a plan position start (index: its place in the launch).
__device__ __forceinline__ int32_t pos_base_of(const PartView& V, int wv_before, int wt_before, int index) {
  return V.rows * (wv_before * V.tp_v + wt_before * V.tp_t + V.row_cost * V.n_seqs * index);
}

// With position, job, sequence and its length in place: the row and page at which tile t0 falls.
__device__ __forceinline__ void cursor_place(RangeCursor& c, const PartView& V, int32_t t0, int32_t pos_base,
                                             int32_t my_pre) {
  c.w = job_tiles_per_page(c.job);
  c.row_pages = (c.len + kPage - 1) / kPage;
  const int32_t seg_base = pos_base + V.rows * (c.w * my_pre + V.row_cost * c.si);
  // a row costs its fixed part and then its pages; r0 is where its first page starts
  const int32_t row_cost = V.row_cost + c.w * c.row_pages;
  c.u = row_cost > 0 ? min(V.rows - 1, (t0 - seg_base) / row_cost) : 0;
  c.r0 = seg_base + c.u * row_cost + V.row_cost;
  c.page = t0 > c.r0 ? (t0 - c.r0 + c.w - 1) / c.w : 0;   // first page that starts at or after t0
  c.owner0 = c.r0 / V.q;
  c.pad[0] = c.pad[1] = c.pad[2] = 0;
}

// Place the cursor of worker `wid` at its first range; false if the worker has no work.  All
// lanes of a warp compute the same values.  Reads the launch plan and the step's sequence
// descriptors only, the first 32 of each in one round of loads.
__device__ __forceinline__ bool cursor_init(RangeCursor& c, const PartView& V, int wid, int lane) {
  c.vw = wid * V.k;
  c.vw_stop = min(c.vw + V.k, V.vw);
  if (c.vw >= c.vw_stop) return false;
  const int32_t t0 = c.vw * V.q;
  c.vw_end = t0 + V.q;
  const int n_pos = V.pos_end - V.pos_begin;
  uint4 pj_lo = make_uint4(0, 0, 0, 0);
  int4 pj_hi = make_int4(0, 0, 0, 0);
  int4 sq_lo = make_int4(0, 0, 0, 0), sq_hi = make_int4(0, 0, 0, 0);
  if (lane < n_pos) {
    pj_lo = __ldg(reinterpret_cast<const uint4*>(V.plan + V.pos_begin + lane));
    pj_hi = __ldg(reinterpret_cast<const int4*>(V.plan + V.pos_begin + lane) + 1);
  }
  if (lane < V.n_seqs) {
    sq_lo = reinterpret_cast<const int4*>(V.seqs + lane)[0];   // seq_id, len_text, len_vis, n_slots
    sq_hi = reinterpret_cast<const int4*>(V.seqs + lane)[1];   // pre_v, pre_t, ncv, pad
  }
  // plan position: the last one of the launch that starts at or before t0
  int n_le = __popc(__ballot_sync(0xffffffffu, lane < n_pos && pos_base_of(V, pj_hi.z, pj_hi.w, lane) <= t0));
  int32_t pos_base;
  if (n_le == 32 && n_pos > 32) {   // beyond the first round
    for (int base = V.pos_begin + 32; base < V.pos_end; base += 32) {
      const int idx = base + lane;
      bool le = false;
      if (idx < V.pos_end) {
        const int4 hi = __ldg(reinterpret_cast<const int4*>(V.plan + idx) + 1);
        le = pos_base_of(V, hi.z, hi.w, idx - V.pos_begin) <= t0;
      }
      n_le += __popc(__ballot_sync(0xffffffffu, le));
    }
    c.pos = V.pos_begin + n_le - 1;
    const PlanJob pj = V.plan[c.pos];
    c.job = pj.job;
    pos_base = pos_base_of(V, pj.wv_before, pj.wt_before, c.pos - V.pos_begin);
  } else {
    const int src = max(n_le, 1) - 1;
    c.pos = V.pos_begin + src;
    uint4 j;
    j.x = __shfl_sync(0xffffffffu, pj_lo.x, src);
    j.y = __shfl_sync(0xffffffffu, pj_lo.y, src);
    j.z = __shfl_sync(0xffffffffu, pj_lo.z, src);
    j.w = __shfl_sync(0xffffffffu, pj_lo.w, src);
    *reinterpret_cast<uint4*>(&c.job) = j;
    pos_base = pos_base_of(V, __shfl_sync(0xffffffffu, pj_hi.z, src), __shfl_sync(0xffffffffu, pj_hi.w, src), src);
  }
  const int w = job_tiles_per_page(c.job);
  // listed sequence: the last one whose rows start at or before t0
  const int32_t rc = V.row_cost;
  n_le = __popc(__ballot_sync(0xffffffffu, lane < V.n_seqs && pos_base + V.rows * (w * (c.job.stream ? sq_hi.x : sq_hi.y) + rc * lane) <= t0));
  int32_t my_pre;
  if (n_le == 32 && V.n_seqs > 32) {
    for (int base = 32; base < V.n_seqs; base += 32) {
      const int idx = base + lane;
      bool le = false;
      if (idx < V.n_seqs) le = pos_base + V.rows * (w * (c.job.stream ? V.seqs[idx].pre_v : V.seqs[idx].pre_t) + rc * idx) <= t0;
      n_le += __popc(__ballot_sync(0xffffffffu, le));
    }
    c.si = n_le - 1;
    const StepSeq sq = V.seqs[c.si];
    c.len = c.job.stream ? sq.len_vis : sq.len_text;
    c.seq_id = sq.seq_id;
    my_pre = c.job.stream ? sq.pre_v : sq.pre_t;
  } else {
    const int src = max(n_le, 1) - 1;
    c.si = src;
    c.len = __shfl_sync(0xffffffffu, c.job.stream ? sq_lo.z : sq_lo.y, src);
    c.seq_id = __shfl_sync(0xffffffffu, sq_lo.x, src);
    my_pre = __shfl_sync(0xffffffffu, c.job.stream ? sq_hi.x : sq_hi.y, src);
  }
  cursor_place(c, V, t0, pos_base, my_pre);
  return true;
}

// The same by one thread alone (the kernel that plans a step's launches ahead).
__device__ __forceinline__ bool cursor_init_scalar(RangeCursor& c, const PartView& V, int wid) {
  c.vw = wid * V.k;
  c.vw_stop = min(c.vw + V.k, V.vw);
  if (c.vw >= c.vw_stop) return false;
  const int32_t t0 = c.vw * V.q;
  c.vw_end = t0 + V.q;
  c.pos = V.pos_begin;
  int32_t pos_base = 0;
  for (int p = V.pos_begin + 1; p < V.pos_end; ++p) {
    const int4 hi = __ldg(reinterpret_cast<const int4*>(V.plan + p) + 1);
    const int32_t b = pos_base_of(V, hi.z, hi.w, p - V.pos_begin);
    if (b > t0) break;
    c.pos = p;
    pos_base = b;
  }
  c.job = V.plan[c.pos].job;
  const int w = job_tiles_per_page(c.job);
  int lo = 0, hi = V.n_seqs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    const int32_t pre = c.job.stream ? V.seqs[mid].pre_v : V.seqs[mid].pre_t;
    if (pos_base + V.rows * (w * pre + V.row_cost * mid) <= t0) lo = mid;
    else hi = mid - 1;
  }
  c.si = lo;
  const StepSeq sq = V.seqs[c.si];
  c.len = c.job.stream ? sq.len_vis : sq.len_text;
  c.seq_id = sq.seq_id;
  cursor_place(c, V, t0, pos_base, c.job.stream ? sq.pre_v : sq.pre_t);
  return true;
}

// Next piece of the worker's ranges, or false when they are used up.  Warp-uniform.
__device__ __forceinline__ bool cursor_next(RangeCursor& c, const PartView& V, Item& it) {
  for (;;) {
    if (c.vw >= c.vw_stop) return false;
    if (c.page >= c.row_pages) {   // next row
      c.r0 += c.w * c.row_pages + V.row_cost;
      c.page = 0;
      if (++c.u == V.rows) {
        c.u = 0;
        bool new_pos = false;
        if (++c.si == V.n_seqs) {
          c.si = 0;
          new_pos = true;
          if (++c.pos >= V.pos_end) {
            c.vw = c.vw_stop;
            return false;
          }
        }
        cursor_load_segment(c, V, new_pos);
      }
      c.owner0 = c.r0 / V.q;
      continue;
    }
    const int32_t d = c.vw_end - c.r0;
    const int lim = d <= 0 ? 0 : min(c.row_pages, (d + c.w - 1) / c.w);
    if (c.page < lim) {
      const int hpi = V.heads_per_item;
      const int n_sub = (V.group + hpi - 1) / hpi;
      const int kv_head = c.u / n_sub, sub = c.u - kv_head * n_sub;
      const int slot = c.vw - c.owner0;
      it.k_layer = c.job.k_layer;
      it.stream = c.job.stream;
      it.n_cons = c.job.n_cons;
      it.flags = c.job.flags;
#pragma unroll
      for (int x = 0; x < kMaxCons; ++x) {
        it.v_layer[x] = c.job.v_layer[x];
        it.q_layer[x] = c.job.q_layer[x];
      }
      it.seq_id = static_cast<uint16_t>(c.seq_id);
      it.seq_idx = static_cast<uint16_t>(c.si);
      it.head = static_cast<uint16_t>(kv_head * V.group + sub * hpi);
      it.slot = static_cast<uint16_t>((c.job.stream ? 0 : V.slots_per_stream) + slot);
      it.first_page = static_cast<uint16_t>(c.page);
      it.n_pages = static_cast<uint16_t>(lim - c.page);
      const bool last = lim == c.row_pages;
      if (last) it.flags |= kFlagStreamEnd;
      it.n_valid_last = static_cast<uint16_t>(last ? c.len - (c.row_pages - 1) * kPage : kPage);
      it.n_heads = static_cast<uint8_t>(min(hpi, V.group - sub * hpi));
      it.skip_new = c.job.skip_new;
      it.finish = c.job.finish;
      it.pad1 = 0;
      // the piece that holds a row's first page tells the merge how many pieces the row has
      it.n_pieces = c.page == 0 ? static_cast<uint16_t>((c.r0 + c.w * (c.row_pages - 1)) / V.q - c.owner0 + 1) : 0;
      if (lim - c.page > kMaxChunkPages || slot < 0 || slot >= V.slots_per_stream) {   // outside the plan's limits
        report_error(V.err, V.err_host, kErrPlan);
        c.vw = c.vw_stop;
        return false;
      }
      c.page = lim;
      return true;
    }
    // the current range owns nothing (more) of this row
    ++c.vw;
    c.vw_end += V.q;
  }
}

// One step of a worker's cursor, kept in shared memory between items.  Warp-uniform.
__device__ __forceinline__ bool cursor_step(RangeCursor* slot, const Params& P, Item& it, int lane) {
  __syncwarp();
  RangeCursor c = *slot;
  const bool ok = cursor_next(c, part_view(P), it);
  __syncwarp();
  if (lane == 0) *slot = c;
  __syncwarp();
  return ok;
}

// Folded append: is page `pg` of the item the page that receives the step's new token?
__device__ __forceinline__ bool holds_new_token(const Params& P, const Item& it, int pg) {
  return P.fold_append && it.stream == 0 && (it.flags & kFlagStreamEnd) && pg == it.n_pages - 1;
}

// Folded append: start fetching the new token's rows of an item that ends its layer's text stream
// (this layer's inputs: after the wait for the previous kernel, with the queries).
__device__ __forceinline__ int first_taker(const Item& it) {   // first consumer that does not leave out the new token
  for (int x = 0; x < it.n_cons; ++x)
    if (!((it.skip_new >> x) & 1)) return x;
  return -1;
}
__device__ __forceinline__ void begin_new_rows(ItemPages& c, const Params& P, const Item& it, int lane, int d) {
  if (!(P.fold_append && it.stream == 0 && (it.flags & kFlagStreamEnd))) return;
  const int n_vec = d / 8, kv_head = it.head / P.group;
  if (lane < n_vec)
    cp_async_16(&c.new_k[lane], reinterpret_cast<const uint4*>(
                                    P.k + ((static_cast<size_t>(it.k_layer) * P.n_seqs + it.seq_idx) * P.hkv + kv_head) * d) + lane);
  const int x = first_taker(it);
  if (x >= 0 && lane >= 16 && lane - 16 < n_vec)
    cp_async_16(&c.new_v[lane - 16],
                reinterpret_cast<const uint4*>(
                    P.v + ((static_cast<size_t>(it.v_layer[x]) * P.n_seqs + it.seq_idx) * P.hkv + kv_head) * d) + (lane - 16));
}

// Start of a worker from the descriptor planned for it when the step began: the first item goes
// into the context slot together with the page ids of its first two pages, the cursor into the
// worker's cursor slot.  False if the worker has no work.  `stage`: 48 bytes of shared memory.
__device__ __forceinline__ bool load_worker_desc(const Params& P, int wid, ItemPages& c0, RangeCursor* cursor,
                                                 int32_t* stage, int lane) {
  const uint4* d = reinterpret_cast<const uint4*>(P.wdesc + static_cast<size_t>(P.launch_index) * kPlanWorkers + wid);
  if (lane < 2) cp_async_16(reinterpret_cast<uint4*>(&c0.item) + lane, d + lane);
  else if (lane < 5) cp_async_16(reinterpret_cast<uint4*>(stage) + (lane - 2), d + lane);
  else if (lane < 10) cp_async_16(reinterpret_cast<uint4*>(cursor) + (lane - 5), d + lane);
  cp_async_wait_all();
  __syncwarp();
  if (c0.item.n_pages == 0) return false;
  if (lane < 2 * (1 + kMaxCons)) c0.pages[lane >> 1][lane & 1] = stage[lane];
  if (lane == 0) c0.kv_head = c0.item.head / P.group;
  __syncwarp();
  return true;
}

// Which worker of a launch a warp is.  Under the static partition the warps of a CTA are adjacent
// workers (adjacent ranges: the same rows, page-table lines and queries), and a launch with fewer
// workers than warps fills the first CTAs and leaves the other SMs to the next launch's early
// part.  Measured against one worker of every CTA first (same call, in-order step): config 2
// 1.117 -> 1.078 ms, configs 3 / 4 / 5 within 0.6 %; runs of adjacent workers spread over all CTAs: 1.092.
__device__ __forceinline__ int worker_index(const Params& P, int warp, int warps_per_cta) {
  if (!P.part_static) return warp * gridDim.x + blockIdx.x;
  return static_cast<int>(blockIdx.x) * warps_per_cta + warp;
}

// Under the static partition, the piece that holds a row's first page records how many pieces
// the row has: one entry per consumer layer and query head, visual and text streams side by side.
__device__ __forceinline__ void record_row_slots(const Params& P, const Item& it, int lane) {
  if (it.n_pieces == 0) return;
  const int x = lane >> 3, h = lane & 7;
  if (x < it.n_cons && h < it.n_heads) {
    const size_t row = (static_cast<size_t>(it.v_layer[x]) * P.max_seqs + it.seq_idx) * P.hq + it.head + h;
    P.row_slots[2 * row + (it.stream ? 0 : 1)] = it.n_pieces;
  }
}

// ------------------------------------------------------------------------------------------
// log-sum-exp merge of one output row's partials (one warp)
// ------------------------------------------------------------------------------------------
//
// Used by the merge kernel and by the attention workers (the worker that delivers a row's last
// partial merges it).  Partials may have been written by other SMs moments ago: they are read
// past the L1 cache.  extra_leader >= 0 adds the step's new token as one more key (merge kernel,
// rows of a GLA follower under the in-order schedule; Eq. 6).
template <int D>
__device__ __forceinline__ void merge_row(const Params& P, int layer, int si, int head, const StepSeq& sq, int lane,
                                          int extra_leader) {
  constexpr int VPL = D / 32;
  const size_t base = (static_cast<size_t>(layer) * P.max_seqs + si) * P.max_slots;
  // Partial rows of this output row: nv from the visual sweep in slots 0.., nt from the text
  // sweep in slots text0...  With claimed items both counts follow from the stream lengths; under
  // the static partition the sweeps recorded them.
  int nv = sq.ncv, nt = sq.n_slots - sq.ncv, text0 = sq.ncv;
  if (P.part_static) {
    const size_t row = (static_cast<size_t>(layer) * P.max_seqs + si) * P.hq + head;
    const uint32_t both = __ldcg(reinterpret_cast<const uint32_t*>(P.row_slots + 2 * row));
    nv = sq.len_vis > 0 ? static_cast<int>(both & 0xffffu) : 0;
    nt = static_cast<int>(both >> 16);
    text0 = P.slots_per_stream;
  }
  const int n_slots = nv + nt;
  auto phys = [&](int s) { return s < nv ? s : text0 + (s - nv); };

  // Lane s holds the (max, sum) pair of slot s; the accumulator rows do not depend on them, so
  // their loads are issued four at a time without waiting for the pairs.
  float mmax = -INFINITY;
  float2 my_ml = make_float2(-INFINITY, 0.f);
  if (lane < n_slots) my_ml = __ldcg(P.part_ml + (base + phys(lane)) * P.hq + head);
  mmax = my_ml.x;
  for (int s = lane + 32; s < n_slots; s += 32) mmax = fmaxf(mmax, __ldcg(P.part_ml + (base + phys(s)) * P.hq + head).x);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, o));

  float s_new = -INFINITY;
  const uint16_t* v_new = nullptr;
  if (extra_leader >= 0) {
    const int kvh = head / P.group;
    const uint16_t* qrow = P.qcache + ((static_cast<size_t>(extra_leader) * P.max_seqs + sq.seq_id) * P.hq + head) * D;
    // the leader's new k: the last row of its text K stream (appended before this kernel ran)
    const int pos = sq.len_text - 1;
    int pid = P.table[table_row(P, extra_leader, 0, sq.seq_id) + pos / kPage];
    if (static_cast<uint32_t>(pid) >= static_cast<uint64_t>(P.n_pool_pages)) {   // never read outside the pool
      if (lane == 0) report_error(P.err, P.err_host, kErrBadPage);
      pid = 0;
    }
    const uint16_t* krow = P.pool + ((static_cast<size_t>(pid) * P.hkv + kvh) * kPage + pos % kPage) * D;
    v_new = P.v + ((static_cast<size_t>(layer) * P.n_seqs + si) * P.hkv + kvh) * D + lane * VPL;
    float dot = 0.f;
#pragma unroll
    for (int e = 0; e < VPL; ++e)
      dot = fmaf(__uint_as_float(static_cast<uint32_t>(qrow[lane * VPL + e]) << 16),
                 __uint_as_float(static_cast<uint32_t>(krow[lane * VPL + e]) << 16), dot);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    s_new = dot * P.scale_log2;
    mmax = fmaxf(mmax, s_new);
    if (P.fold_append && head % P.group == 0) {
      // this layer's new v row has no sweep to store it: the merge warp of the KV head's first query head does
      int pid_v = P.table[table_row(P, layer, 2, sq.seq_id) + pos / kPage];
      if (static_cast<uint32_t>(pid_v) < static_cast<uint64_t>(P.n_pool_pages)) {
        uint16_t* dst_v = P.pool + ((static_cast<size_t>(pid_v) * P.hkv + kvh) * kPage + pos % kPage) * D + lane * VPL;
#pragma unroll
        for (int e = 0; e < VPL; ++e) dst_v[e] = v_new[e];
      } else if (lane == 0) {
        report_error(P.err, P.err_host, kErrBadPage);
      }
    }
  }

  float lsum = 0.f;
  float acc[VPL];
#pragma unroll
  for (int e = 0; e < VPL; ++e) acc[e] = 0.f;
  if (v_new != nullptr) {
    const float w = exp2f(s_new - mmax);
    lsum = w;
#pragma unroll
    for (int e = 0; e < VPL; ++e) acc[e] = w * __uint_as_float(static_cast<uint32_t>(v_new[e]) << 16);
  }
  for (int s0 = 0; s0 < n_slots; s0 += 4) {
    float v[4][VPL];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int s = phys(min(s0 + u, n_slots - 1));
      const float* src = P.part_acc + ((base + s) * P.hq + head) * D + lane * VPL;
      if (VPL == 4) {
        const float4 a = __ldcg(reinterpret_cast<const float4*>(src));
        v[u][0] = a.x, v[u][1] = a.y, v[u][2 % VPL] = a.z, v[u][3 % VPL] = a.w;
      } else {
        const float2 a = __ldcg(reinterpret_cast<const float2*>(src));
        v[u][0] = a.x, v[u][1] = a.y;
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int s = s0 + u;
      float2 ml;
      if (s < 32) {
        ml.x = __shfl_sync(0xffffffffu, my_ml.x, s & 31);
        ml.y = __shfl_sync(0xffffffffu, my_ml.y, s & 31);
      } else {
        ml = __ldcg(P.part_ml + (base + phys(min(s, n_slots - 1))) * P.hq + head);
      }
      if (s < n_slots && ml.y > 0.f) {   // (a sweep that left out its only key has an empty partial)
        const float w = exp2f(ml.x - mmax);
        lsum = fmaf(ml.y, w, lsum);
#pragma unroll
        for (int e = 0; e < VPL; ++e) acc[e] = fmaf(v[u][e], w, acc[e]);
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

// After an item's partial rows have been stored: count the item's pages towards the output rows
// that this launch completes (the job's finish bits), and merge a row whose count is full.  The
// count of a row is the pages of its visual and text streams, or of the item's stream alone when
// only that stream is swept for the row in this launch.  Release / acquire: every lane fences its
// stores before lane 0's atomic, and the merging warp fences again before it reads.
template <int D>
__device__ __forceinline__ void finish_rows(const Params& P, const ItemPages& c, int lane) {
  const Item& it = c.item;
  if ((it.finish & 0xf) == 0) return;
  __threadfence();
  __syncwarp();
  const StepSeq sq = c.sq;
  const int own_pages = ((it.stream ? sq.len_vis : sq.len_text) + kPage - 1) / kPage;
  const int total = (it.finish & kFinishOwnStream)
                        ? own_pages
                        : (sq.len_vis + kPage - 1) / kPage + (sq.len_text + kPage - 1) / kPage;
  // one counter per (consumer layer, sequence, first head of the item)
  int old = 0;
  if (lane < it.n_cons && ((it.finish >> lane) & 1)) {
    const size_t row = (static_cast<size_t>(it.v_layer[lane]) * P.max_seqs + it.seq_idx) * P.hq + it.head;
    old = atomicAdd(P.row_done + row, static_cast<int>(it.n_pages));
  }
  for (int x = 0; x < it.n_cons; ++x) {
    if (!((it.finish >> x) & 1)) continue;
    const int before = __shfl_sync(0xffffffffu, old, x);
    if (before + it.n_pages != total) continue;
    __threadfence();
    const size_t row = (static_cast<size_t>(it.v_layer[x]) * P.max_seqs + it.seq_idx) * P.hq + it.head;
    if (lane == 0) P.row_done[row] = 0;   // ready for the next step
    for (int h = 0; h < it.n_heads; ++h) merge_row<D>(P, it.v_layer[x], it.seq_idx, it.head + h, sq, lane, -1);
  }
}

}  // namespace
}  // namespace qc
