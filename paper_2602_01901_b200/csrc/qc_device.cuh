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

constexpr int kErrTimeout = 6;
constexpr int kErrBadPage = 5;

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
__device__ __forceinline__ void bulk_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   dst_smem),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
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

// Programmatic dependent launch: the kernels of a decode step are launched back to back with
// the programmatic-serialization attribute.  Each one first lets its successor start getting
// scheduled, does its set-up that touches no global data, and then waits for its predecessor
// to have completed (and its writes to be visible) before it reads or writes global memory.
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
};

__device__ __forceinline__ void worker_init(WorkerState& st, int n_my) {
  st.n_my = n_my;
  st.cons_k = st.iss_k = 0;
  st.iss_page = st.iss_which = 0;
  st.iss_slot = st.cons_slot = 0;
  st.cons_phase = 0;
  st.in_flight = 0;
  st.dead = false;
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
    if (lane == 0) atomicMax(P.err, kErrBadPage);
    pid = 0;
  }
  if (lane == 0) {
    uint64_t* bar = &full[st.iss_slot];
    const uint32_t dst = ring + st.iss_slot * kTile;
    fence_proxy_async();   // the slot's earlier generic-proxy accesses precede this async write
    mbar_expect_tx(bar, kTile);
    if (TMAP) {
      const int32_t row = (pid * P.hkv + c.item.kv_head) * kPage;
      tensor_g2s_2d(dst, &P.tmap, 0, row, bar);
      if (D == 128) tensor_g2s_2d(dst + kTile / 2, &P.tmap, 64, row, bar);
    } else {
      const uint16_t* src = P.pool + (static_cast<size_t>(pid) * P.hkv + c.item.kv_head) * (kPage * D);
      bulk_g2s(dst, src, kTile, bar);
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
  for (uint32_t spin = 0; !done && spin < kSpinLimit; ++spin) done = mbar_try_wait(bar, st.cons_phase);
  if (!done) {
    if (lane == 0) atomicMax(P.err, kErrTimeout);
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
__device__ __forceinline__ void drain_ring(WorkerState& st, uint64_t* full) {
  while (st.in_flight > 0) {
    uint64_t* bar = &full[st.cons_slot];
    uint32_t done = 0;
    for (uint32_t spin = 0; !done && spin < kSpinLimit; ++spin) done = mbar_try_wait(bar, st.cons_phase);
    st.in_flight--;
    if (++st.cons_slot == RING) {
      st.cons_slot = 0;
      st.cons_phase ^= 1u;
    }
  }
}

// Fetch an item's descriptor and page ids into the warp's context slot.  Returns the item.
__device__ __forceinline__ Item load_item_pages(ItemPages& c, const Params& P, int item_idx, int lane) {
  const uint4* ip = reinterpret_cast<const uint4*>(P.items + item_idx);
  uint4 a = __ldg(ip), b = __ldg(ip + 1);
  __syncwarp();
  if (lane == 0) {
    reinterpret_cast<uint4*>(&c.item)[0] = a;
    reinterpret_cast<uint4*>(&c.item)[1] = b;
  }
  Item it;
  reinterpret_cast<uint4*>(&it)[0] = a;
  reinterpret_cast<uint4*>(&it)[1] = b;
  if (lane < it.n_pages) {
    c.pages[0][lane] = P.table[table_row(P, it.k_layer, it.stream, it.seq_id) + it.first_page + lane];
    for (int x = 0; x < it.n_cons; ++x)
      c.pages[1 + x][lane] = P.table[table_row(P, it.v_layer[x], 2 + it.stream, it.seq_id) + it.first_page + lane];
  }
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

}  // namespace
}  // namespace qc
