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

__device__ __forceinline__ void load_tc_ctx(TcCtx& c, const Params& P, int item_idx, int lane) {
  load_item_pages(c.ip, P, item_idx, lane);
}

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
template <int D, int NQ, int NV, int MODE = 0>
__device__ __forceinline__ void process_item_tc(WorkerState& st, const TcCtx* ctx, uint32_t ring, uint64_t* full,
                                                const Params& P, int lane) {
  constexpr int KS = D / 16;    // k-steps of the score product = m-tiles of the value product
  auto ctx_of = [ctx](int k) -> const ItemPages& { return ctx[k & 1].ip; };
  const Item& it = ctx[st.cons_k & 1].ip.item;
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

  for (int pg = 0; pg < n_pages && !st.dead; ++pg) {
    const int nvalid = (pg == n_pages - 1) ? n_valid_last : kPage;
    uint32_t pb[NQ][2];
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
      if (nvalid < kPage) {
        // rows past the end of the stream hold whatever the pool held: clear them, since a
        // zero weight does not cancel a NaN or an infinity
        const int n_seg = (kPage - nvalid) * (D / 64);
        for (int e = lane; e < n_seg * 8; e += 32) {
          const int seg = e >> 3, half = seg / (kPage - nvalid), row = nvalid + seg % (kPage - nvalid);
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
        mma_bf16_16816(o[v][i], a, pb[NQ == 1 ? 0 : v]);
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
        if (g == 0) P.part_ml[row0 + hh] = make_float2(m[xq][hh], l[xq][hh]);
      }
    }
  }
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1) attend_tc_kernel(const __grid_constant__ Params P) {
  constexpr uint32_t kTile = kPage * D * 2;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_all[kWarps][kRingTc];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // swizzled tiles must sit on 1024-byte boundaries
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t ring = base + static_cast<uint32_t>(warp) * kRingTc * kTile;
  TcCtx* ctx = reinterpret_cast<TcCtx*>(base_ptr + static_cast<size_t>(kWarps) * kRingTc * kTile) + warp * 2;
  uint64_t* full = full_all[warp];
  auto ctx_of = [ctx](int k) -> const ItemPages& { return ctx[k & 1].ip; };

  if (lane == 0) {
    for (int s = 0; s < kRingTc; ++s) mbar_init(&full[s], 1);
    fence_mbar_init();
  }
  __syncthreads();
  pdl_launch_dependents();
  pdl_wait();

  WorkerState st;
  worker_init(st, 0);
  int next = claim_take(P, claim_issue(P, lane));
  if (next < 0) return;
  load_tc_ctx(ctx[0], P, next, lane);
  st.n_my = 1;
  next = claim_take(P, claim_issue(P, lane));
  if (next >= 0) {
    load_tc_ctx(ctx[1], P, next, lane);
    st.n_my = 2;
  }
  __syncwarp();
  fill_ring<D, kRingTc, true>(st, ctx_of, ring, full, P, lane);

  for (int k = 0; k < st.n_my && !st.dead; ++k) {
    const Item& it = ctx[k & 1].ip.item;
    const int nc = it.n_cons;
    const bool shared = it.flags & kFlagShared;
    // claim the item after next now; the answer is needed only when this item is done
    const int issued = (next >= 0) ? claim_issue(P, lane) : 0;
    if (nc == 1 && (it.flags & kFlagReadLogits)) process_item_tc<D, 1, 1, 2>(st, ctx, ring, full, P, lane);
    else if (nc == 1 && (it.flags & kFlagWriteLogits)) process_item_tc<D, 1, 1, 1>(st, ctx, ring, full, P, lane);
    else if (nc == 1) process_item_tc<D, 1, 1>(st, ctx, ring, full, P, lane);
    else if (shared && nc == 2) process_item_tc<D, 1, 2>(st, ctx, ring, full, P, lane);
    else if (shared && nc == 3) process_item_tc<D, 1, 3>(st, ctx, ring, full, P, lane);
    else if (shared) process_item_tc<D, 1, 4>(st, ctx, ring, full, P, lane);
    else process_item_tc<D, 2, 2>(st, ctx, ring, full, P, lane);   // own-query sweeps feed at most two layers here
    if (st.dead) break;
    __syncwarp();
    if (next >= 0) {
      next = claim_take(P, issued);
      if (next >= 0) {   // the context slot of the item just finished receives the item after next
        load_tc_ctx(ctx[k & 1], P, next, lane);
        __syncwarp();
        st.n_my = k + 3;
      }
    }
    st.cons_k = k + 1;
    fill_ring<D, kRingTc, true>(st, ctx_of, ring, full, P, lane);
  }
  if (st.dead) drain_ring<kRingTc>(st, full);
}

template <int D>
constexpr int attend_tc_smem_bytes() {
  return 1024 + kWarps * kRingTc * kPage * D * 2 + kWarps * 2 * static_cast<int>(sizeof(TcCtx));
}

}  // namespace

cudaError_t configure_kernels_tc(int* attend_smem) {
  cudaError_t e = cudaFuncSetAttribute(attend_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       attend_tc_smem_bytes<128>());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           attend_tc_smem_bytes<64>());
  if (attend_smem) *attend_smem = attend_tc_smem_bytes<128>();
  return e;
}

cudaError_t launch_attend_tc(const Params& p, int n_sms, cudaStream_t stream) {
  const int n_items = p.item_end - p.item_begin;
  if (n_items <= 0) return cudaSuccess;
  const int grid = min(n_sms, (n_items + kWarps - 1) / kWarps);
  if (p.d == 128)
    return launch_pdl(attend_tc_kernel<128>, dim3(grid), dim3(kThreads), attend_tc_smem_bytes<128>(), stream, p);
  return launch_pdl(attend_tc_kernel<64>, dim3(grid), dim3(kThreads), attend_tc_smem_bytes<64>(), stream, p);
}

}  // namespace qc
