// Prefill-phase attention with Lazy Attention (Eq. 1, Eq. 5, Eq. 7): causal attention over one
// prompt, all layers, where a lazy layer takes query and key rows from its block's first layer
// -- all rows in GLA (Eq. 5), the rows of visual tokens in VLA (Eq. 7) -- and keeps its own V.
// The selection happens when a tile is staged into shared memory (the source layer of a row
// is a per-token choice), so the tile arithmetic is that of ordinary causal attention.
//
// One CTA = 64 query rows of one (layer, query head); 4 warps x 16 rows.  Key/value tiles of
// 64 tokens are double-buffered through shared memory with 16-byte asynchronous copies into an
// XOR-swizzled layout (conflict-free ldmatrix).  Both products run on the tensor cores
// (mma.m16n8k16 bf16 -> fp32); the score accumulators of a warp are re-used in registers as the
// A operand of the value product.  Softmax is online, in the log2 domain, fp32.

#include "qc_device.cuh"

namespace qc {
namespace {

constexpr int kBM = 64;   // query rows per CTA
constexpr int kBN = 64;   // keys per tile
constexpr int kPrefillThreads = 128;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// byte offset of 16-byte chunk `chunk` of row `row` in a [rows][D] bf16 tile whose chunks are
// XOR-swizzled inside each 128-byte span
template <int D>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return row * (D * 2) + ((chunk & ~7) << 4) + (((chunk & 7) ^ (row & 7)) << 4);
}

struct PrefillArgs {
  // tcgen05 kernel: q / k / v as 3-D tensors {D, heads, n_layers * T}, box {64, 1, 64}; the output as a
  // 4-D tensor {D, hq, T, n_layers}, box {64, 1, 128, 1}; 128-byte swizzle
  CUtensorMap tmap_q, tmap_k, tmap_v, tmap_o;
  const PrefillPass* passes;   // device; tcgen05 kernel: what blockIdx.z stands for (null: layer blockIdx.z alone)
  CUtensorMap tmap_pool;   // the paged pool as a 2-D tensor [pages * hkv * 16 rows][D], box 16 rows x 64 elements
  int64_t n_pool_pages;    // bound for page ids read from the table
  const uint8_t* tile_code;    // [ceil(T / 64)] device: 0 = the 64-token tile is all text, 1 = all visual, 2 = mixed
  const uint16_t* q;     // [n_layers][T][hq][D]
  const uint16_t* k;     // [n_layers][T][hkv][D]
  const uint16_t* v;     // [n_layers][T][hkv][D]
  uint16_t* out;         // [n_layers][T][hq][D]
  const uint8_t* kind;   // [T] device
  const uint8_t* layer_kind;   // [n_layers] device (QC_LAYER_*)
  const uint8_t* leader;       // [n_layers] device
  int32_t T, hq, hkv, group, n_layers, gla;
  float scale_log2;
  // tokens the sequence already held before this prompt chunk: they are read from the paged cache,
  // text stream then visual stream, and are visible to every new token
  const uint16_t* pool;
  const int32_t* table;        // [n_layers][4][max_seqs][max_pages]
  const uint8_t* layer_flags;  // kLayerOwnsTextK: the layer's text K is its own
  int32_t max_seqs, max_pages, seq_id, n0_text, n0_vis;
};

// Stage rows [row0, row0 + 64) of one head of a [n_layers][T][heads][D] tensor; row t comes
// from layer `own` or, where lead_rows says so, from layer `lead`.  Rows past T are zero-filled.
template <int D>
__device__ __forceinline__ void stage_tile(uint32_t smem, const uint16_t* base, int own, int lead, bool lazy, bool gla,
                                           const uint8_t* kind, int row0, int T, int heads, int head) {
  constexpr int CH = D / 8;                         // 16-byte chunks per row
  constexpr int RPP = kPrefillThreads / CH;         // rows covered by one pass of the CTA
  constexpr int NP = kBN / RPP;
  const int c = threadIdx.x % CH, r0 = threadIdx.x / CH;
  // the source layer of each of this thread's rows first (independent loads), then the copies
  int layer_of[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int t = row0 + r0 + i * RPP;
    layer_of[i] = (lazy && (gla || (t < T && kind[t]))) ? lead : own;
  }
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int r = r0 + i * RPP, t = row0 + r;
    const uint32_t dst = smem + tile_off<D>(r, c);
    if (t < T) {
      cp_async16(dst, base + ((static_cast<size_t>(layer_of[i]) * T + t) * heads + head) * D + c * 8);
    } else {
      asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0u) : "memory");
    }
  }
}

// Stage 64 cached tokens [ord0, ord0 + 64) of one stream of (src_layer, sequence) from the paged
// pool; tokens at or past n_valid are zero-filled (their pool rows may hold anything).
template <int D>
__device__ __forceinline__ void stage_cached(uint32_t smem, const PrefillArgs& A, int src_layer, int stream, int ord0,
                                             int n_valid, int head) {
  constexpr int CH = D / 8;
  constexpr int RPP = kPrefillThreads / CH;
  constexpr int NP = kBN / RPP;
  const int c = threadIdx.x % CH, r0 = threadIdx.x / CH;
  const size_t trow = ((static_cast<size_t>(src_layer) * 4 + stream) * A.max_seqs + A.seq_id) * A.max_pages;
  int pid[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int ord = ord0 + r0 + i * RPP;
    pid[i] = ord < n_valid ? A.table[trow + ord / kPage] : -1;
  }
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int r = r0 + i * RPP, ord = ord0 + r;
    const uint32_t dst = smem + tile_off<D>(r, c);
    if (pid[i] >= 0) {
      cp_async16(dst, A.pool + ((static_cast<size_t>(pid[i]) * A.hkv + head) * kPage + ord % kPage) * D + c * 8);
    } else {
      asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0u) : "memory");
    }
  }
}

template <int D>
__global__ void __launch_bounds__(kPrefillThreads) prefill_attend_kernel(const PrefillArgs A) {
  constexpr int KS = D / 16;   // k-steps of the score product
  constexpr int NT = D / 8;    // n-tiles of the value product
  constexpr uint32_t kTileBytes = kBN * D * 2;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  const uint32_t sQ = smem_u32(smem_raw);
  const uint32_t sK = sQ + kTileBytes;              // two buffers
  const uint32_t sV = sK + 2 * kTileBytes;          // two buffers

  const int n_qtiles = (A.T + kBM - 1) / kBM;
  const int qt = n_qtiles - 1 - blockIdx.x;         // long rows first
  const int head = blockIdx.y, layer = blockIdx.z;
  const int kvh = head / A.group;
  const bool lazy = A.layer_kind[layer] != 0;
  const int lead = A.leader[layer];
  const bool gla = A.gla != 0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const int m0 = qt * kBM;
  // Key tiles, in order: the cached text tokens, the cached visual tokens (all visible, read from
  // the pool: a lazy layer's visual K -- and in GLA its text K -- are its leader's pages, which is
  // Eq. 5 / Eq. 7's selection for tokens already cached), then the new tokens 0 .. qt (causal).
  const int ct_text = (A.n0_text + kBN - 1) / kBN, ct_vis = (A.n0_vis + kBN - 1) / kBN;
  const int n_cached_tiles = ct_text + ct_vis;
  const int n_ktiles = n_cached_tiles + qt + 1;
  const int k_text_layer = (A.n0_text && !(A.layer_flags[layer] & kLayerOwnsTextK)) ? lead : layer;
  const int k_vis_layer = lazy ? lead : layer;
  auto stage_kv = [&](int i, uint32_t kdst, uint32_t vdst) {
    if (i < ct_text) {
      stage_cached<D>(kdst, A, k_text_layer, 0, i * kBN, A.n0_text, kvh);
      stage_cached<D>(vdst, A, layer, 2, i * kBN, A.n0_text, kvh);
    } else if (i < n_cached_tiles) {
      stage_cached<D>(kdst, A, k_vis_layer, 1, (i - ct_text) * kBN, A.n0_vis, kvh);
      stage_cached<D>(vdst, A, layer, 3, (i - ct_text) * kBN, A.n0_vis, kvh);
    } else {
      const int t0 = (i - n_cached_tiles) * kBN;
      stage_tile<D>(kdst, A.k, layer, lead, lazy, gla, A.kind, t0, A.T, A.hkv, kvh);
      stage_tile<D>(vdst, A.v, layer, layer, false, false, A.kind, t0, A.T, A.hkv, kvh);
    }
  };

  // stage Q and the first K/V tiles
  stage_tile<D>(sQ, A.q, layer, lead, lazy, gla, A.kind, m0, A.T, A.hq, head);
  stage_kv(0, sK, sV);
  cp_async_commit();
  cp_async_wait<0>();
  __syncthreads();

  // query fragments of this warp's 16 rows (A operand of the score product)
  uint32_t qa[KS][4];
  {
    const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) ldmatrix_x4(qa[kk], sQ + tile_off<D>(row, 2 * kk + (lane >> 4)));
  }

  float o[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};   // rows g and g + 8 of the warp's 16
  const int qrow0 = m0 + warp * 16 + g;                           // global index of row g (row g + 8: +8)

  for (int kt = 0; kt < n_ktiles; ++kt) {
    const int buf = kt & 1;
    if (kt + 1 < n_ktiles) {   // prefetch the next tiles into the other buffer
      stage_kv(kt + 1, sK + (buf ^ 1) * kTileBytes, sV + (buf ^ 1) * kTileBytes);
      cp_async_commit();
    }
    const uint32_t kb = sK + buf * kTileBytes, vb = sV + buf * kTileBytes;
    // visibility of the tile's keys: a cached tile shows its first n_show tokens to every row; a
    // tile of new tokens starts at prompt position n0 and is causal
    const bool cached_tile = kt < n_cached_tiles;
    const int n_show = !cached_tile ? 0
                       : (kt < ct_text ? min(kBN, A.n0_text - kt * kBN) : min(kBN, A.n0_vis - (kt - ct_text) * kBN));
    const int n0 = (kt - n_cached_tiles) * kBN;

    // ---- S = Q K^T for 16 rows x 64 keys
    float s[kBN / 8][4];
#pragma unroll
    for (int j = 0; j < kBN / 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
#pragma unroll
      for (int jp = 0; jp < kBN / 16; ++jp) {   // pairs of 8-key n-tiles
        uint32_t b[4];
        const int row = jp * 16 + (lane & 7) + ((lane >> 4) << 3);
        ldmatrix_x4(b, kb + tile_off<D>(row, 2 * kk + ((lane >> 3) & 1)));
        const uint32_t b0[2] = {b[0], b[1]}, b1[2] = {b[2], b[3]};
        mma_bf16_16816(s[2 * jp], qa[kk], b0);
        mma_bf16_16816(s[2 * jp + 1], qa[kk], b1);
      }
    }
    // ---- scale, causal mask, online softmax
    float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < kBN / 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int col = j * 8 + 2 * t4 + (e & 1), key = n0 + col;
        const int qrow = qrow0 + ((e >> 1) << 3);
        const bool visible = cached_tile ? col < n_show : (key <= qrow && key < A.T);
        const float x = visible ? s[j][e] * A.scale_log2 : -INFINITY;
        s[j][e] = x;
        tmax[e >> 1] = fmaxf(tmax[e >> 1], x);
      }
    }
    float corr[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 1));
      tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 2));
      const float mnew = fmaxf(mrow[r], tmax[r]);
      // a row past the end of the prompt sees no key at all: keep its numbers finite
      const float msafe = (mnew == -INFINITY) ? 0.f : mnew;
      corr[r] = exp2f(mrow[r] - msafe);
      mrow[r] = mnew;
      tmax[r] = msafe;
    }
    float psum[2] = {0.f, 0.f};
#pragma unroll
    for (int j = 0; j < kBN / 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float p = exp2f(s[j][e] - tmax[e >> 1]);
        s[j][e] = p;
        psum[e >> 1] += p;
      }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) lrow[r] = lrow[r] * corr[r] + psum[r];
#pragma unroll
    for (int i = 0; i < NT; ++i) {
      o[i][0] *= corr[0];
      o[i][1] *= corr[0];
      o[i][2] *= corr[1];
      o[i][3] *= corr[1];
    }
    // ---- O += P V: the score accumulators are the A operand, 16 keys per k-step
#pragma unroll
    for (int ks = 0; ks < kBN / 16; ++ks) {
      uint32_t pa[4];
      pa[0] = pack_bf16x2(s[2 * ks][0], s[2 * ks][1]);
      pa[1] = pack_bf16x2(s[2 * ks][2], s[2 * ks][3]);
      pa[2] = pack_bf16x2(s[2 * ks + 1][0], s[2 * ks + 1][1]);
      pa[3] = pack_bf16x2(s[2 * ks + 1][2], s[2 * ks + 1][3]);
#pragma unroll
      for (int ip = 0; ip < NT / 2; ++ip) {   // pairs of 8-column n-tiles of the head dimension
        uint32_t b[4];
        const int row = ks * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
        ldmatrix_x4_trans(b, vb + tile_off<D>(row, 2 * ip + (lane >> 4)));
        const uint32_t b0[2] = {b[0], b[1]}, b1[2] = {b[2], b[3]};
        mma_bf16_16816(o[2 * ip], pa, b0);
        mma_bf16_16816(o[2 * ip + 1], pa, b1);
      }
    }
    cp_async_wait<0>();
    __syncthreads();
  }

  // ---- normalise and store
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int tok = qrow0 + 8 * r;
    if (tok < A.T) {
      const float inv = 1.f / lrow[r];
      uint16_t* dst = A.out + ((static_cast<size_t>(layer) * A.T + tok) * A.hq + head) * D + 2 * t4;
#pragma unroll
      for (int i = 0; i < NT; ++i)
        *reinterpret_cast<uint32_t*>(dst + 8 * i) = pack_bf16x2(o[i][2 * r] * inv, o[i][2 * r + 1] * inv);
    }
  }
}

// ------------------------------------------------------------------------------------------
// The same computation on the fifth-generation tensor cores (tcgen05), head_dim 128.
//
// One CTA = 128 query rows of one (layer, query head): 128 softmax threads, one per row, plus an
// issue warp and a load warp.  Key / value tiles of 64 tokens are staged (with the per-row
// source-layer selection) into the canonical 128-byte-swizzled shared-memory layout,
// [two 64-column halves][rows][128 bytes].  One elected lane issues
//     S[128 x 64]   = Q[128 x 128] . K^T      8 x tcgen05.mma (M 128, N 64, K 16), accumulator in TMEM
//     O[128 x 128] += P[128 x 64]  . V        4 x tcgen05.mma (M 128, N 128, K 16), P read from TMEM,
//                                             V read MN-major from shared memory
// and commits to an mbarrier.  A thread reads its row of S from TMEM (one TMEM lane per row: no
// cross-thread reduction), does the online softmax, and writes the bf16 weights back into TMEM as
// the next A operand.  The running maximum is only moved when it grows by more than
// 2^8 (the weights then stay below 2^8, harmless in fp32/bf16), so the accumulator in TMEM is
// rescaled rarely (TMEM load, scale, store).  Two CTAs per SM (2 x 256 TMEM columns) overlap one
// CTA's softmax with the other's products.
// Every mbarrier wait is bounded; on expiry the CTA records the error, frees its TMEM and leaves.

constexpr int kTM = 128;        // query rows per CTA
constexpr int kTN = 64;         // keys per tile
constexpr int kTD = 128;        // head dim
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColS = 0, kColO = 128;   // scores: two buffers of 64 columns; accumulator: 128 columns
constexpr float kRescaleThreshold = 8.f;   // log2 units

__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  // start address, leading / stride byte offsets (all >> 4), descriptor version 1, 128-byte swizzle
  return static_cast<uint64_t>((saddr >> 4) & 0x3fff) | (static_cast<uint64_t>((lbo_bytes >> 4) & 0x3fff) << 16) |
         (static_cast<uint64_t>((sbo_bytes >> 4) & 0x3fff) << 32) | (1ull << 46) | (2ull << 61);
}
// S = Q K^T for one tile: eight products (k-steps of 16 along the head dimension) issued by one
// elected lane from warp-uniform code.  adesc/bdesc address k-step 0; a k-step advances the start
// address by 32 bytes inside a 128-byte swizzle row, and the second 64 elements of the head
// dimension sit one half-tile further (a_half / b_half bytes).
template <uint32_t A_HALF, uint32_t B_HALF>
__device__ __forceinline__ void umma_scores(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred e, pz, po;\n\t.reg .b64 da, db;\n\t"
      "elect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 pz, 0, 0;\n\tsetp.eq.b32 po, 0, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pz;\n\t"
      "add.u64 da, %1, 2;\n\tadd.u64 db, %2, 2;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, po;\n\t"
      "add.u64 da, %1, 4;\n\tadd.u64 db, %2, 4;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, po;\n\t"
      "add.u64 da, %1, 6;\n\tadd.u64 db, %2, 6;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, po;\n\t"
      "add.u64 da, %1, %4;\n\tadd.u64 db, %2, %5;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, po;\n\t"
      "add.u64 da, %1, %4 + 2;\n\tadd.u64 db, %2, %5 + 2;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, po;\n\t"
      "add.u64 da, %1, %4 + 4;\n\tadd.u64 db, %2, %5 + 4;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, po;\n\t"
      "add.u64 da, %1, %4 + 6;\n\tadd.u64 db, %2, %5 + 6;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, po;\n\t}"
      :: "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "n"(A_HALF >> 4), "n"(B_HALF >> 4) : "memory");
}
// O (+)= P V for one tile of 64 keys: four products (k-steps of 16 keys).  The weights are read from
// tensor memory (8 columns per k-step), the V rows MN-major from shared memory (16 rows = 2048 bytes
// per k-step).  `accumulate` = 0 starts a new accumulator.
__device__ __forceinline__ void umma_values(uint32_t tmem_d, uint32_t tmem_p, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred e, pa, po;\n\t.reg .b64 db;\n\t.reg .b32 ta;\n\t"
      "elect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 pa, %4, 0;\n\tsetp.eq.b32 po, 0, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, pa;\n\t"
      "add.u32 ta, %1, 8;\n\tadd.u64 db, %2, 128;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, po;\n\t"
      "add.u32 ta, %1, 16;\n\tadd.u64 db, %2, 256;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, po;\n\t"
      "add.u32 ta, %1, 24;\n\tadd.u64 db, %2, 384;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, po;\n\t}"
      :: "r"(tmem_d), "r"(tmem_p), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile(
      "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
      "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tc5_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc5_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
// 2^x, single MUFU instruction (2^-inf = 0)
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
         "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
         "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
         "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}

// Bounded wait on an mbarrier phase.
__device__ __forceinline__ bool bounded_wait(uint64_t* bar, uint32_t parity) {
  constexpr uint32_t kLimit = 1u << 18;
  uint32_t done = mbar_try_wait(bar, parity);
  for (uint32_t spin = 0; !done && spin < kLimit; ++spin) done = mbar_try_wait(bar, parity);
  return done != 0;
}
// one non-blocking look at an mbarrier phase
__device__ __forceinline__ uint32_t mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return done;
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tensor_g2s_3d(uint32_t dst_smem, const void* tmap, int32_t x, int32_t y, int32_t z,
                                              uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::
          "r"(dst_smem),
      "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
      : "memory");
}

__device__ __forceinline__ void tensor_s2g_4d(const void* tmap, uint32_t src_smem, int32_t x, int32_t y, int32_t z, int32_t w) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::
                   "l"(reinterpret_cast<uint64_t>(tmap)),
               "r"(src_smem), "r"(x), "r"(y), "r"(z), "r"(w)
               : "memory");
}

constexpr int kTc5Threads = kTM + 64;   // 128 softmax threads (one per query row) + an issue warp + a load warp

// Warp roles.  Warps 0-3: one thread per query row -- read the row's scores from TMEM, online
// softmax, write the bf16 weights.  Warp 4 (issue warp) issues every product: S(0), S(1), then per
// tile PV(kt) followed by S(kt+2).  Warp 5 (load warp) fetches the K and V tiles.  A product costs
// the issuing lane some tens of cycles and a look at an mbarrier about as much, so both streams
// stay off the softmax path; the issue warp runs warp-uniform code and elects the issuing lane
// inside the asm block, which lets the descriptors live in uniform registers.
// A K/V tile whose 64 rows all come from one layer -- every tile of an ordinary or GLA layer, and
// the all-text / all-visual tiles of a VLA lazy layer -- is fetched by two tensor-map copies; only
// a tile that mixes text and visual rows of a VLA lazy layer is gathered row by row with 16-byte
// copies by the 32 lanes.  Hand-offs are mbarriers only:
//   bar_k[b], bar_v[b]  copies -> issue warp        K / V tile landed in buffer b
//   bar_s[b]      tensor core -> softmax, load warp     score buffer b holds S(kt); K buffer b is free
//   bar_p[b]      softmax -> issue warp                 weights P(kt) written (one barrier per score buffer: P(kt+2)
//                 needs S(kt+2), which is issued after the issue warp has seen P(kt), so a barrier is never
//                 more than one completion ahead of its waiter -- a parity wait could not tell otherwise)
//   bar_o[b]      tensor core -> load warp, issue warp, softmax     PV(kt) done (kt & 1 == b): V buffer b and
//                 score buffer b are free and the accumulator may be rescaled
// The bf16 weights P(kt) overwrite the first 32 columns of score buffer kt & 1 in tensor memory and
// are the A operand of the value product from there: no shared-memory round trip.  S(kt+2) goes
// into the same buffer, so the issue warp waits for PV(kt) to complete before it issues S(kt+2)
// (an earlier version relied on issue order alone and produced a corrupted tile now and then).
// With two score buffers the softmax of tile kt+1 overlaps PV(kt) and S(kt+2).
// When the sequence already holds tokens, the CTA's key tiles start with those (cached text, then
// cached visual tokens, four pool pages per tile, all visible) before the prompt's own tiles.
// CACHED = false is the instantiation for a prompt that starts a sequence: no code for cached tiles.
// NV > 1 is the instantiation for shared-score passes: up to NV layers' accumulators in tensor
// memory (all 512 columns, so one CTA per SM), NV value tiles per key tile.
template <bool CACHED, int NV>
__global__ void __launch_bounds__(NV > 1 ? kTc5Threads + 32 : kTc5Threads, NV > 1 ? 1 : 2)
    prefill_attend_tcgen05_kernel(const __grid_constant__ PrefillArgs A, int32_t* err) {
  static_assert(NV == 1 || !CACHED, "shared-score passes are for prompts that start a sequence");
  constexpr uint32_t kCols = NV > 1 ? 512 : kTmemCols;
  // No static shared memory: the dynamic window then starts on the 1024-byte boundary that the
  // swizzled tiles need, and two CTAs fit an SM (2 x 112 KiB of tiles).  Checked below.
  extern __shared__ __align__(1024) uint8_t smem_dyn[];
  const uint32_t base = smem_u32(smem_dyn);
  const uint32_t sQ = base;                         // [2][128][128 B]  32 KiB
  const uint32_t sK = sQ + 2 * kTM * 128;           // two buffers of [2][64][128 B] 16 KiB
  const uint32_t sV = sK + 2 * (2 * kTN * 128);     // two buffers per consumer: consumer x, buffer b at (2 x + b)
  constexpr uint32_t kKV = 2 * kTN * 128;
  constexpr uint32_t kTiles = 2 * kTM * 128 + 2 * kKV + NV * 2 * kKV;
  uint64_t* bar_s = reinterpret_cast<uint64_t*>(smem_dyn + kTiles);          // two: one per score buffer
  uint64_t* bar_p = reinterpret_cast<uint64_t*>(smem_dyn + kTiles + 16);          // two
  uint64_t* bar_k = reinterpret_cast<uint64_t*>(smem_dyn + kTiles + 32);          // two
  uint64_t* bar_v = reinterpret_cast<uint64_t*>(smem_dyn + kTiles + 48);          // two
  uint64_t* bar_o = reinterpret_cast<uint64_t*>(smem_dyn + kTiles + 64);          // two: PV(kt) -> bar_o[kt & 1]
  uint32_t& tmem_base_slot = *reinterpret_cast<uint32_t*>(smem_dyn + kTiles + 80);
  volatile int32_t& failed = *reinterpret_cast<volatile int32_t*>(smem_dyn + kTiles + 84);
  uint64_t& bar_q = *reinterpret_cast<uint64_t*>(smem_dyn + kTiles + 88);   // the two 64-row halves of the Q tile
  uint64_t& bar_e = *reinterpret_cast<uint64_t*>(smem_dyn + kTiles + 96);   // NV > 1: an output tile is staged
  uint64_t& bar_r = *reinterpret_cast<uint64_t*>(smem_dyn + kTiles + 104);  // NV > 1: its store has read it
  if (base & 1023u) {   // cannot happen with the layout above; never run the tensor core on a misplaced tile
    if (threadIdx.x == 0) atomicMax(err, kErrBadPage);
    return;
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_qtiles = (A.T + kTM - 1) / kTM;
  const int qt = n_qtiles - 1 - blockIdx.x;         // long rows first
  const int head = blockIdx.y;
  int n_cons = 1, v_layer[NV];
  if (A.passes) {
    const PrefillPass ps = A.passes[blockIdx.z];
    n_cons = NV > 1 ? min(ps.n, NV) : 1;
#pragma unroll
    for (int x = 0; x < NV; ++x) v_layer[x] = ps.v[x < n_cons ? x : 0];
  } else {
    v_layer[0] = blockIdx.z;
  }
  const int layer = v_layer[0];   // decides where Q and K come from; with NV > 1 all consumers share that
  const int kvh = head / A.group;
  const bool lazy = A.layer_kind[layer] != 0;
  const int lead = A.leader[layer];
  const bool gla = A.gla != 0;
  const int m0 = qt * kTM;
  const int row = m0 + threadIdx.x;                 // a softmax thread's query row
  // Key tiles, in order: the cached text tokens, the cached visual tokens (all visible, read from
  // the pool: a lazy layer's visual K -- and in GLA its text K -- are its leader's pages, which is
  // Eq. 5 / Eq. 7's selection for tokens already cached), then the new tokens (causal).
  const int ct_text = CACHED ? (A.n0_text + kTN - 1) / kTN : 0, ct_vis = CACHED ? (A.n0_vis + kTN - 1) / kTN : 0;
  const int n_cached = ct_text + ct_vis;
  const int n_ktiles = n_cached + min((A.T + kTN - 1) / kTN, (m0 + kTM + kTN - 1) / kTN);

  if (threadIdx.x == 0) {
    mbar_init(&bar_s[0], 1);
    mbar_init(&bar_s[1], 1);
    mbar_init(&bar_q, 2);
    mbar_init(&bar_e, kTM);
    mbar_init(&bar_r, 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bar_k[b], 1);
      mbar_init(&bar_v[b], n_cons);
      mbar_init(&bar_o[b], 1);
      mbar_init(&bar_p[b], kTM);
    }
    fence_mbar_init();
    failed = 0;
  }
  if (warp == 4) {   // the score warp owns the TMEM allocation
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(kCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc5_fence_before();
  __syncthreads();
  tc5_fence_after();
  const uint32_t tmem = tmem_base_slot;

  // instruction descriptors: fp32 accumulate, bf16 operands, M 128; S: N 64, both K-major; PV: N 128, B MN-major
  constexpr uint32_t kIdescS = (1u << 4) | (1u << 7) | (1u << 10) | ((kTN >> 3) << 17) | ((kTM >> 4) << 24);
  constexpr uint32_t kIdescO = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((kTD >> 3) << 17) | ((kTM >> 4) << 24);

  if (warp >= 4) {
    // ------------------------------------------------------------------ tile fetch + product issue
    // Fetch key tile (is_k) or value tile kt into `dst`; completion is one phase of `bar`.
    // `which`: 0 = 64 query rows (tile index kt counts 64-row tiles), 1 = key tile, 2 = value tile.
    // The 64 rows go to `dst` and `dst + half` (the two 64-column halves).
    // The tile codes of a VLA lazy layer, read once: lane i holds tiles i, i + 32, i + 64.
    uint32_t codes[3] = {0u, 0u, 0u};
    if (warp == 5 && lazy && !gla) {
      const int n_tiles = (A.T + kTN - 1) / kTN;
#pragma unroll
      for (int i = 0; i < 3; ++i)
        if (lane + 32 * i < n_tiles) codes[i] = A.tile_code[lane + 32 * i];
    }
    auto code_of = [&](int kt) -> int {   // whole warp
      if (kt >= 96) return A.tile_code[kt];
      const uint32_t c = kt < 32 ? codes[0] : (kt < 64 ? codes[1] : codes[2]);
      return static_cast<int>(__shfl_sync(0xffffffffu, c, kt & 31));
    };
    const int k_text_layer = (CACHED && A.n0_text && !(A.layer_flags[layer] & kLayerOwnsTextK)) ? lead : layer;
    // Where cached tile kt of the key (which = 1) or value (which = 2) sequence lives: source layer,
    // stream, first token and the stream's length.
    auto cached_tile = [&](int which, int kt, int& src, int& stream, int& ord0, int& n_valid) {
      if (kt < ct_text) {
        src = which == 1 ? k_text_layer : layer, stream = which == 1 ? 0 : 2, ord0 = kt * kTN, n_valid = A.n0_text;
      } else {
        src = which == 1 ? (lazy ? lead : layer) : layer, stream = which == 1 ? 1 : 3;
        ord0 = (kt - ct_text) * kTN, n_valid = A.n0_vis;
      }
    };
    // Lanes 0..3 read the page ids of a cached tile's four pages (0 where the page holds no token).
    auto load_page_ids = [&](int which, int kt) -> int {
      int src, stream, ord0, n_valid, pid = 0;
      cached_tile(which, kt, src, stream, ord0, n_valid);
      if (lane < 4 && ord0 + 16 * lane < n_valid) {
        const size_t trow = ((static_cast<size_t>(src) * 4 + stream) * A.max_seqs + A.seq_id) * A.max_pages;
        pid = A.table[trow + ord0 / 16 + lane];
      }
      return pid;
    };
    // Fetch cached tile kt: 64 tokens of one stream of (source layer, this sequence) from the paged
    // pool, as four pages.  A page that is full arrives by two tensor-map copies; the rows of a
    // page that is not (the stream's last page, or pages past its end) are gathered or zeroed by
    // the lanes, since their pool rows may hold anything and a zero weight does not cancel a NaN.
    int ahead_tile[2] = {-1, -1}, ahead_pid[2] = {0, 0};   // page ids requested one tile ahead, per which
    auto fetch_cached = [&](int which, int kt, uint32_t dst, uint32_t half, uint64_t* bar) {
      int src, stream, ord0, n_valid;
      cached_tile(which, kt, src, stream, ord0, n_valid);
      int pid = ahead_tile[which - 1] == kt ? ahead_pid[which - 1] : load_page_ids(which, kt);
      if (kt + 1 < n_cached) {   // the next tile's ids travel while this tile is fetched and consumed
        ahead_tile[which - 1] = kt + 1;
        ahead_pid[which - 1] = load_page_ids(which, kt + 1);
      }
      if (static_cast<uint32_t>(pid) >= static_cast<uint64_t>(A.n_pool_pages)) {   // never read outside the pool
        atomicMax(err, kErrBadPage);
        pid = 0;
      }
      int n_full = 0;
      bool gathered = false;
#pragma unroll
      for (int pg = 0; pg < 4; ++pg) {
        const int p_id = __shfl_sync(0xffffffffu, pid, pg);
        const int n_tok = min(16, max(0, n_valid - (ord0 + 16 * pg)));
        if (n_tok == 16) {
          ++n_full;
          continue;
        }
        gathered = true;
        for (int e = lane; e < 16 * (kTD / 8); e += 32) {
          const int r = 16 * pg + (e >> 4), c = e & 15;
          const uint32_t d = dst + (c >> 3) * half + r * 128 + (((c & 7) ^ (r & 7)) << 4);
          if ((e >> 4) < n_tok) {
            cp_async16(d, A.pool + ((static_cast<size_t>(p_id) * A.hkv + kvh) * 16 + (e >> 4)) * kTD + c * 8);
          } else {
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(d), "r"(0u) : "memory");
          }
        }
      }
      if (gathered) {
        cp_async_commit();
        cp_async_wait<0>();
        fence_proxy_async();
        __syncwarp();
      }
      if (n_full == 0) {
        if (lane == 0) mbar_arrive(bar);
        return;
      }
      if (lane == 0) mbar_expect_tx(bar, n_full * 4096);
#pragma unroll
      for (int pg = 0; pg < 4; ++pg) {
        const int p_id = __shfl_sync(0xffffffffu, pid, pg);
        if (n_valid - (ord0 + 16 * pg) >= 16 && lane == 0) {
          const int32_t row = (p_id * A.hkv + kvh) * 16;
          tensor_g2s_2d(dst + pg * 2048, &A.tmap_pool, 0, row, bar);
          tensor_g2s_2d(dst + half + pg * 2048, &A.tmap_pool, 64, row, bar);
        }
      }
    };
    // `which`: 0 = 64 query rows (kt counts 64-row tiles of the prompt), 1 = key tile kt, 2 = value
    // tile kt of the CTA's tile sequence (cached tiles first).
    auto fetch_tile = [&](int which, int kt, uint32_t dst, uint32_t half, uint64_t* bar, int v_src = -1) {
      if (which != 0) {
        if (CACHED && kt < n_cached) {
          fetch_cached(which, kt, dst, half, bar);
          return;
        }
        kt -= n_cached;   // a tile of new tokens
      }
      int src = (which == 2 && v_src >= 0) ? v_src : layer;
      bool mixed = false;
      if (which != 2 && lazy && kt * kTN < A.T) {   // queries and keys of a lazy layer: the leader's for visual rows
        if (gla) {
          src = lead;
        } else {
          const int code = code_of(kt);
          mixed = code == 2;
          src = code == 1 ? lead : layer;
        }
      }
      if (!mixed) {
        if (lane == 0) {
          const void* tm = which == 0 ? static_cast<const void*>(&A.tmap_q)
                                      : (which == 1 ? static_cast<const void*>(&A.tmap_k) : static_cast<const void*>(&A.tmap_v));
          const int h = which == 0 ? head : kvh;
          mbar_expect_tx(bar, kKV);
          tensor_g2s_3d(dst, tm, 0, h, src * A.T + kt * kTN, bar);
          tensor_g2s_3d(dst + half, tm, 64, h, src * A.T + kt * kTN, bar);
        }
      } else {   // rows of two layers: gather with 16-byte copies (64 rows x 16 chunks over 32 lanes)
        const uint16_t* from = which == 0 ? A.q : A.k;
        const int heads = which == 0 ? A.hq : A.hkv, h = which == 0 ? head : kvh;
        for (int e = lane; e < kTN * (kTD / 8); e += 32) {
          const int r = e >> 4, c = e & 15, t = kt * kTN + r;
          const uint32_t d = dst + (c >> 3) * half + r * 128 + (((c & 7) ^ (r & 7)) << 4);
          if (t < A.T) {
            const int l = A.kind[t] ? lead : layer;
            cp_async16(d, from + ((static_cast<size_t>(l) * A.T + t) * heads + h) * kTD + c * 8);
          } else {
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(d), "r"(0u) : "memory");
          }
        }
        cp_async_commit();
        cp_async_wait<0>();
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar);
      }
    };
    bool ok = true;
    auto wait_on = [&](uint64_t* bar, uint32_t& phase) {   // warp-uniform bounded wait
      if (ok && !__all_sync(0xffffffffu, mbar_try_wait(bar, phase)))   // usually complete at the first look
        ok = __all_sync(0xffffffffu, bounded_wait(bar, phase) && !failed);
      phase ^= 1u;
    };
    if (NV > 1 && warp != 5) {
      // ---------------- shared-score passes: two issue warps.  Alone on its SM, the CTA has nothing
      // else to hide one lane's issue time behind, so the score products (warp 4) and the value
      // products of the NV consumers (warp 6) are issued in parallel; same hand-offs as below.
      uint32_t ph_k[2] = {0, 0}, ph_v[2] = {0, 0}, ph_o[2] = {0, 0}, ph_p[2] = {0, 0};
      if (warp == 4) {
        const uint64_t qd = umma_desc(sQ, 16, 1024);
        const uint64_t kd0 = umma_desc(sK, 16, 1024), kd1 = umma_desc(sK + kKV, 16, 1024);
        auto issue_scores = [&](int buf) {
          umma_scores<kTM * 128, kTN * 128>(tmem + kColS + buf * kTN, qd, buf ? kd1 : kd0, kIdescS);
          umma_commit(&bar_s[buf]);
        };
        {
          uint32_t ph_q = 0;
          wait_on(&bar_q, ph_q);
        }
        for (int kt = 0; kt < 2 && kt < n_ktiles && ok; ++kt) {
          wait_on(&bar_k[kt], ph_k[kt]);
          if (ok) {
            tc5_fence_after();
            issue_scores(kt);
          }
        }
        for (int kt = 0; kt + 2 < n_ktiles && ok; ++kt) {
          const int buf = kt & 1;
          wait_on(&bar_o[buf], ph_o[buf]);   // PV(kt) complete: the buffer's weights have been read
          wait_on(&bar_k[buf], ph_k[buf]);   // K(kt+2) landed
          if (!ok) break;
          tc5_fence_after();
          issue_scores(buf);
        }
      } else {
        uint64_t vd[NV][2];   // consumer x, buffer b
#pragma unroll
        for (int x = 0; x < NV; ++x) {
          vd[x][0] = umma_desc(sV + (2 * x) * kKV, kTN * 128, 1024);
          vd[x][1] = umma_desc(sV + (2 * x + 1) * kKV, kTN * 128, 1024);
        }
        for (int kt = 0; kt < n_ktiles && ok; ++kt) {
          const int buf = kt & 1;
          wait_on(&bar_p[buf], ph_p[buf]);   // P(kt) is in tensor memory
          wait_on(&bar_v[buf], ph_v[buf]);   // the consumers' V(kt) landed
          if (!ok) break;
          tc5_fence_after();
#pragma unroll
          for (int x = 0; x < NV; ++x)
            if (x < n_cons)
              umma_values(tmem + kColO + kTD * x, tmem + kColS + buf * kTN, buf ? vd[x][1] : vd[x][0], kIdescO,
                          kt > 0 ? 1u : 0u);
          umma_commit(&bar_o[buf]);
        }
      }
    } else if (warp == 4) {
      // ---------------- issue warp: S(kt) = Q K(kt)^T into score buffer kt & 1, O += P(kt) V(kt)
      const uint64_t qd = umma_desc(sQ, 16, 1024);
      const uint64_t kd0 = umma_desc(sK, 16, 1024), kd1 = umma_desc(sK + kKV, 16, 1024);
      uint64_t vd[NV][2];   // consumer x, buffer b
#pragma unroll
      for (int x = 0; x < NV; ++x) {
        vd[x][0] = umma_desc(sV + (2 * x) * kKV, kTN * 128, 1024);
        vd[x][1] = umma_desc(sV + (2 * x + 1) * kKV, kTN * 128, 1024);
      }
      uint32_t ph_k[2] = {0, 0}, ph_v[2] = {0, 0}, ph_o[2] = {0, 0}, ph_p[2] = {0, 0};
      auto issue_scores = [&](int buf) {   // whole warp; one elected lane issues
        umma_scores<kTM * 128, kTN * 128>(tmem + kColS + buf * kTN, qd, buf ? kd1 : kd0, kIdescS);
        umma_commit(&bar_s[buf]);
      };
      {
        uint32_t ph_q = 0;
        wait_on(&bar_q, ph_q);
      }
      for (int kt = 0; kt < 2 && kt < n_ktiles && ok; ++kt) {   // the first two score tiles have nothing to wait for but K
        wait_on(&bar_k[kt], ph_k[kt]);
        if (ok) {
          tc5_fence_after();
          issue_scores(kt);
        }
      }
      for (int kt = 0; kt < n_ktiles && ok; ++kt) {
        const int buf = kt & 1;
        wait_on(&bar_p[buf], ph_p[buf]);            // P(kt) is in tensor memory
        wait_on(&bar_v[buf], ph_v[buf]);            // V(kt) landed
        if (!ok) break;
        {
          tc5_fence_after();
#pragma unroll
          for (int x = 0; x < NV; ++x)
            if (x < n_cons)
              umma_values(tmem + kColO + kTD * x, tmem + kColS + buf * kTN, buf ? vd[x][1] : vd[x][0], kIdescO,
                          kt > 0 ? 1u : 0u);
          umma_commit(&bar_o[buf]);
        }
        if (kt + 2 < n_ktiles) {
          // S(kt+2) overwrites the buffer that holds P(kt).  Products with different accumulators are
          // not documented to run in issue order, so wait until PV(kt) has completed.
          wait_on(&bar_o[buf], ph_o[buf]);
          wait_on(&bar_k[buf], ph_k[buf]);          // K(kt+2) landed
          if (!ok) break;
          tc5_fence_after();
          issue_scores(buf);
        }
      }
    } else {
      // ---------------- load warp: K(kt) once S(kt-2) is complete, V(kt) once PV(kt-2) is complete.
      // The two streams advance independently (the products complete in the order S, S, PV, S, PV, ...),
      // so the warp polls both barriers without blocking on either.
      uint32_t ph_s[2] = {0, 0}, ph_o[2] = {0, 0};
      fetch_tile(0, 2 * qt, sQ, kTM * 128, &bar_q);
      fetch_tile(1, 0, sK, kTN * 128, &bar_k[0]);
      fetch_tile(0, 2 * qt + 1, sQ + kTN * 128, kTM * 128, &bar_q);
      auto fetch_values = [&](int kt) {   // one tile per consumer; bar_v[kt & 1] counts them all
        const int b = kt & 1;
#pragma unroll
        for (int x = 0; x < NV; ++x)
          if (x < n_cons) fetch_tile(2, kt, sV + (2 * x + b) * kKV, kTN * 128, &bar_v[b], v_layer[x]);
      };
      fetch_values(0);
      if (n_ktiles > 1) {
        fetch_tile(1, 1, sK + kKV, kTN * 128, &bar_k[1]);
        fetch_values(1);
      }
      int k_next = 2, v_next = 2;
      uint32_t idle = 0;
      while ((k_next < n_ktiles || v_next < n_ktiles) && ok) {
        bool progress = false;
        if (k_next < n_ktiles) {
          const int b = k_next & 1;
          if (__all_sync(0xffffffffu, mbar_test_wait(&bar_s[b], ph_s[b]))) {
            ph_s[b] ^= 1u;
            fetch_tile(1, k_next, sK + b * kKV, kTN * 128, &bar_k[b]);
            ++k_next;
            progress = true;
          }
        }
        if (v_next < n_ktiles) {
          const int b = v_next & 1;
          if (__all_sync(0xffffffffu, mbar_test_wait(&bar_o[b], ph_o[b]))) {
            ph_o[b] ^= 1u;
            fetch_values(v_next);
            ++v_next;
            progress = true;
          }
        }
        if (progress) {
          idle = 0;
        } else if (++idle > (1u << 20) || ((idle & 1023u) == 0 && failed)) {
          ok = false;
        }
      }
    }
    if (!ok) failed = 1;
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ softmax threads
    const uint32_t t_row = tmem + (static_cast<uint32_t>(warp * 32) << 16);   // this warp's 32 TMEM lanes
    float m_ref = -INFINITY, l_sum = 0.f;
    uint32_t ph_s[2] = {0, 0};
    bool ok = true;
    for (int kt = 0; kt < n_ktiles; ++kt) {
      const int buf = kt & 1;
      if (!__all_sync(0xffffffffu, mbar_try_wait(&bar_s[buf], ph_s[buf]))) {
        ok = bounded_wait(&bar_s[buf], ph_s[buf]) && !failed;
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      }
      ph_s[buf] ^= 1u;
      tc5_fence_after();
      // ---- this row's 64 scores (raw dot products; the scale is folded into the exponent)
      float p[kTN];
      {
        uint32_t r0[32], r1[32];
        tmem_ld32_nowait(t_row + kColS + buf * kTN, r0);
        tmem_ld32_nowait(t_row + kColS + buf * kTN + 32, r1);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int j = 0; j < 32; ++j) p[j] = __uint_as_float(r0[j]), p[32 + j] = __uint_as_float(r1[j]);
      }
      if (CACHED && kt < n_cached) {   // cached tokens: all visible; only a stream's last tile is short
        const int n_show = kt < ct_text ? A.n0_text - kt * kTN : A.n0_vis - (kt - ct_text) * kTN;
        if (n_show < kTN) {
#pragma unroll
          for (int j = 0; j < kTN; ++j)
            if (j >= n_show) p[j] = -INFINITY;
        }
      }
      const int n0 = (kt - n_cached) * kTN;
      if (kt >= n_cached && (n0 + kTN - 1 > m0 || n0 + kTN > A.T)) {   // only tiles on the diagonal or at the end of the prompt need the mask
#pragma unroll
        for (int j = 0; j < kTN; ++j) {
          const int key = n0 + j;
          if (!(key <= row && key < A.T)) p[j] = -INFINITY;
        }
      }
      float mx[4] = {p[0], p[1], p[2], p[3]};
#pragma unroll
      for (int j = 4; j < kTN; ++j) mx[j & 3] = fmaxf(mx[j & 3], p[j]);
      const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * A.scale_log2;   // the scale is positive
      float corr = 1.f;
      if (m_tile > m_ref + kRescaleThreshold || m_ref == -INFINITY) {
        if (m_tile != -INFINITY) {
          corr = exp2f(m_ref - m_tile);     // 0 on the first tile
          m_ref = m_tile;
        }
      }
      const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
      float ps[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int j = 0; j < kTN; ++j) {
        p[j] = ex2_approx(fmaf(p[j], A.scale_log2, neg_m));
        ps[j & 3] += p[j];
      }
      l_sum = l_sum * corr + ((ps[0] + ps[1]) + (ps[2] + ps[3]));
      if (kt > 0 && __any_sync(0xffffffffu, corr != 1.f)) {   // rare: move the accumulator to the new reference
        // PV(kt-1) -- and with it every earlier value product -- must be done: phase (kt-1)/2 of its barrier
        ok = bounded_wait(&bar_o[(kt - 1) & 1], ((kt - 1) >> 1) & 1) && !failed;
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
        tc5_fence_after();
#pragma unroll
        for (int x = 0; x < NV; ++x) {
          if (x < n_cons) {
#pragma unroll
            for (int c = 0; c < kTD / 32; ++c) {
              uint32_t r[32];
              tmem_ld32(t_row + kColO + kTD * x + 32 * c, r);
#pragma unroll
              for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * corr);
              tmem_st32(t_row + kColO + kTD * x + 32 * c, r);
            }
          }
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      }
      // ---- weights as the A operand, in place of the scores just read: 64 bf16 = 32 columns of this row's lane
      {
        uint32_t w[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) w[j] = pack_bf16x2(p[2 * j], p[2 * j + 1]);
        tmem_st32(t_row + kColS + buf * kTN, w);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      }
      tc5_fence_before();
      mbar_arrive(&bar_p[buf]);
    }
    if (ok) ok = bounded_wait(&bar_o[(n_ktiles - 1) & 1], ((n_ktiles - 1) >> 1) & 1) && !failed;   // the last value product
    ok = __all_sync(0xffffffffu, ok);
    // Scale the accumulator of consumer x and put the tile into the Q tile's shared memory (free: every
    // product has completed) in the swizzled layout of a 128-row box.
    auto stage_output = [&](int x, float inv) {
      const uint32_t orow = sQ + threadIdx.x * 128;
      const uint32_t sw = threadIdx.x & 7;
#pragma unroll
      for (int c = 0; c < kTD / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(t_row + kColO + kTD * x + 32 * c, r);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int chunk = 4 * c + j;   // 16-byte chunk of the 256-byte row
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(orow + (chunk >> 3) * (kTM * 128) + (((chunk & 7) ^ sw) << 4)),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * j + 0]) * inv, __uint_as_float(r[8 * j + 1]) * inv)),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * j + 2]) * inv, __uint_as_float(r[8 * j + 3]) * inv)),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * j + 4]) * inv, __uint_as_float(r[8 * j + 5]) * inv)),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * j + 6]) * inv, __uint_as_float(r[8 * j + 7]) * inv))
                       : "memory");
        }
      }
      fence_proxy_async();
    };
    if constexpr (NV > 1) {
      // One output tile per consumer, one after the other through the same staging area: the 128
      // threads arrive on bar_e when a tile is staged, thread 0 stores it and arrives on bar_r when
      // the stores have read it (bounded waits throughout, as everywhere in this kernel).
      if (ok) {
        tc5_fence_after();
        const float inv = 1.f / l_sum;
        for (int x = 0; x < n_cons; ++x) {
          if (x > 0) {
            ok = bounded_wait(&bar_r, static_cast<uint32_t>(x - 1) & 1u) && !failed;
            ok = __all_sync(0xffffffffu, ok);
          }
          if (!ok) break;
          stage_output(x, inv);
          mbar_arrive(&bar_e);
          if (threadIdx.x == 0) {
            if (bounded_wait(&bar_e, static_cast<uint32_t>(x) & 1u)) {
              tensor_s2g_4d(&A.tmap_o, sQ, 0, head, m0, v_layer[x]);
              tensor_s2g_4d(&A.tmap_o, sQ + kTM * 128, 64, head, m0, v_layer[x]);
              asm volatile("cp.async.bulk.commit_group;" ::: "memory");
              asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // (also: shared memory is released at exit)
              mbar_arrive(&bar_r);
            } else {
              failed = 1;
            }
          }
          __syncwarp();
        }
      }
      if (!ok) {
        failed = 1;
        if (lane == 0) atomicMax(err, kErrTimeout);
      }
    } else if (ok) {
      // two tensor-map stores write the staged tile (clipped at token T)
      tc5_fence_after();
      stage_output(0, 1.f / l_sum);
      asm volatile("bar.sync 1, %0;" ::"n"(kTM) : "memory");   // the 128 softmax threads
      if (threadIdx.x == 0) {
        tensor_s2g_4d(&A.tmap_o, sQ, 0, head, m0, layer);
        tensor_s2g_4d(&A.tmap_o, sQ + kTM * 128, 64, head, m0, layer);
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // shared memory is released at exit
      }
    } else {
      failed = 1;
      if (lane == 0) atomicMax(err, kErrTimeout);
      asm volatile("bar.arrive 1, %0;" ::"n"(kTM) : "memory");   // do not hold the other softmax warps
    }
  }
  tc5_fence_before();
  __syncthreads();
  if (warp == 4) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kCols) : "memory");
  }
}

// ------------------------------------------------------------------------------------------
// Two query tiles per CTA, key tiles of 128 tokens
// ------------------------------------------------------------------------------------------
//
// For prompts that start a sequence.  One CTA = 256 query rows (two tiles of 128) of one (layer,
// query head), alone on its SM with all 512 columns of tensor memory: per query tile t one score
// buffer S_t[128 x 128] and one accumulator O_t[128 x 128].  Per 128-key tile and query tile:
//     S_t = Q_t . K^T     8 x tcgen05.mma (M 128, N 128, K 16)
//     O_t += P_t . V      2 x 4 tcgen05.mma (M 128, N 128, K 16), P_t (bf16) read from the first 64 columns of S_t
// so a key costs half as many products, barrier round trips and tensor-memory transfers as with
// 64-key tiles, and a score product reads 8 KiB of shared memory for 64 cycles of arithmetic
// instead of 6 KiB for 32.  The two query tiles alternate on the tensor core: while the 128
// softmax threads of one tile work, the products of the other tile run.
// Warps 0-3 / 4-7: softmax of query tile 0 / 1, one thread per row.  Warp 8 issues the score
// products, warp 9 the value products, warp 10 fetches (warps 8-11 give registers to the others).  Hand-offs (mbarriers, all waits bounded):
//   bar_q[t]            copies -> warp 8          query tile t landed
//   bar_k[b], bar_v[b]  copies -> warps 8 / 9     K / V tile landed in buffer b
//   bar_s[t]            tensor core -> softmax t  S_t(kt) complete
//   bar_p[t], bar_pb[t] softmax t -> warp 9       the weights P_t(kt) of keys 0..63 / 64..127 are written
//   bar_o[t]            tensor core -> warp 8, softmax t    PV_t(kt) complete: S_t may be overwritten, O_t rescaled
//   bar_kf[b], bar_vf[b]  tensor core -> warp 10  both tiles' products on buffer b are complete
// No barrier can run two completions ahead of a waiter: each next completion needs something the
// waiter produces after it has seen the previous one.
constexpr int kPN = 128;                             // keys per tile
constexpr int kPairThreads = 2 * kTM + 4 * 32;   // warp 11 only completes the warpgroup whose registers are handed over
constexpr uint32_t kPairQT = 2 * kTM * 128;          // one query tile: two 64-column halves of 128 rows
constexpr uint32_t kPairKT = 2 * kPN * 128;          // one key or value tile
constexpr uint32_t kPairHalf = kPN * 128;            // distance between the two column halves of a tile (kTM == kPN)
constexpr uint32_t kPairTiles = 2 * kPairQT + 4 * kPairKT;
constexpr int prefill_pair_smem_bytes() { return kPairTiles + 176; }

__global__ void __launch_bounds__(kPairThreads, 1)
    prefill_attend_pair_kernel(const __grid_constant__ PrefillArgs A, int32_t* err) {
  extern __shared__ __align__(1024) uint8_t smem_dyn[];
  const uint32_t base = smem_u32(smem_dyn);
  const uint32_t sQ = base, sK = sQ + 2 * kPairQT, sV = sK + 2 * kPairKT;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_dyn + kPairTiles);
  uint64_t *bar_q = bars, *bar_k = bars + 2, *bar_v = bars + 4, *bar_s = bars + 6, *bar_p = bars + 8, *bar_o = bars + 10,
           *bar_kf = bars + 12, *bar_vf = bars + 14, *bar_pb = bars + 16;
  uint32_t& tmem_base_slot = *reinterpret_cast<uint32_t*>(smem_dyn + kPairTiles + 144);
  volatile int32_t& failed = *reinterpret_cast<volatile int32_t*>(smem_dyn + kPairTiles + 148);
  if (base & 1023u) {   // cannot happen with the layout above; never run the tensor core on a misplaced tile
    if (threadIdx.x == 0) atomicMax(err, kErrBadPage);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_pairs = (A.T + 2 * kTM - 1) / (2 * kTM);
  const int qp = n_pairs - 1 - blockIdx.x;          // long rows first
  const int head = blockIdx.y;
  const int layer = A.passes ? A.passes[blockIdx.z].v[0] : static_cast<int>(blockIdx.z);
  const int kvh = head / A.group;
  const bool lazy = A.layer_kind[layer] != 0;
  const int lead = A.leader[layer];
  const bool gla = A.gla != 0;
  // query tile t covers rows (2 qp + t) * 128 .. + 127 and sees key tiles 0 .. n_kt<t> - 1
  const int n_all = (A.T + kPN - 1) / kPN;
  const int n_kt0 = min(n_all, 2 * qp + 1), n_kt1 = (2 * qp + 1) * kTM < A.T ? min(n_all, 2 * qp + 2) : 0;
  const int n_ktiles = max(n_kt0, n_kt1);

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bar_q[i], 2);
      mbar_init(&bar_k[i], 2);
      mbar_init(&bar_v[i], 2);
      mbar_init(&bar_s[i], 1);
      mbar_init(&bar_p[i], kTM);
      mbar_init(&bar_pb[i], kTM);
      mbar_init(&bar_o[i], 1);
      mbar_init(&bar_kf[i], 1);
      mbar_init(&bar_vf[i], 1);
    }
    fence_mbar_init();
    failed = 0;
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc5_fence_before();
  __syncthreads();
  tc5_fence_after();
  const uint32_t tmem = tmem_base_slot;
  // tensor memory columns: S_0, S_1, O_0, O_1
  constexpr uint32_t kIdescS = (1u << 4) | (1u << 7) | (1u << 10) | ((kPN >> 3) << 17) | ((kTM >> 4) << 24);
  constexpr uint32_t kIdescO = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((kTD >> 3) << 17) | ((kTM >> 4) << 24);

  if (warp >= 8) {
    // the issuing and fetching warps need few registers; the softmax threads hold a row of 128 scores
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;" ::: "memory");
    bool ok = true;
    auto wait_on = [&](uint64_t* bar, uint32_t& phase) {   // warp-uniform bounded wait
      if (ok && !__all_sync(0xffffffffu, mbar_try_wait(bar, phase)))
        ok = __all_sync(0xffffffffu, bounded_wait(bar, phase) && !failed);
      phase ^= 1u;
    };
    if (warp == 11) {
      // nothing
    } else if (warp == 8) {
      // ---------------- score products: S_t(kt) once K(kt) has landed and PV_t(kt - 1) is complete
      const uint64_t qd0 = umma_desc(sQ, 16, 1024), qd1 = umma_desc(sQ + kPairQT, 16, 1024);
      const uint64_t kd0 = umma_desc(sK, 16, 1024), kd1 = umma_desc(sK + kPairKT, 16, 1024);
      uint32_t ph_q = 0, ph_k = 0, ph_o = 0;   // bit b / bit t: the phase of barrier b / t
      auto wait_bit = [&](uint64_t* bar, uint32_t& phases, int i) {
        uint32_t ph = (phases >> i) & 1u;
        wait_on(bar, ph);
        phases ^= 1u << i;
      };
      for (int kt = 0; kt < n_ktiles && ok; ++kt) {
        const int b = kt & 1;
        wait_bit(&bar_k[b], ph_k, b);
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (kt >= (t ? n_kt1 : n_kt0)) continue;
          if (kt == 0) wait_bit(&bar_q[t], ph_q, t);
          else wait_bit(&bar_o[t], ph_o, t);
          if (!ok) break;
          tc5_fence_after();
          umma_scores<kPairHalf, kPairHalf>(tmem + t * kPN, t ? qd1 : qd0, b ? kd1 : kd0, kIdescS);
          umma_commit(&bar_s[t]);
        }
        if (ok) umma_commit(&bar_kf[b]);
      }
    } else if (warp == 9) {
      // ---------------- value products: PV_t(kt) once P_t(kt) is written and V(kt) has landed
      const uint64_t vd0 = umma_desc(sV, kPairHalf, 1024), vd1 = umma_desc(sV + kPairKT, kPairHalf, 1024);
      uint32_t ph_p = 0, ph_pb = 0, ph_v = 0;
      auto wait_bit = [&](uint64_t* bar, uint32_t& phases, int i) {
        uint32_t ph = (phases >> i) & 1u;
        wait_on(bar, ph);
        phases ^= 1u << i;
      };
      for (int kt = 0; kt < n_ktiles && ok; ++kt) {
        const int b = kt & 1;
        bool first = true;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (kt >= (t ? n_kt1 : n_kt0)) continue;
          wait_bit(&bar_p[t], ph_p, t);
          if (first) {
            wait_bit(&bar_v[b], ph_v, b);
            first = false;
          }
          if (!ok) break;
          tc5_fence_after();
          umma_values(tmem + 2 * kPN + t * kTD, tmem + t * kPN, b ? vd1 : vd0, kIdescO, kt > 0 ? 1u : 0u);
          wait_bit(&bar_pb[t], ph_pb, t);   // the weights of keys 64..127
          if (!ok) break;
          tc5_fence_after();
          umma_values(tmem + 2 * kPN + t * kTD, tmem + t * kPN + 32, (b ? vd1 : vd0) + 512, kIdescO, 1u);
          umma_commit(&bar_o[t]);
        }
        if (ok) umma_commit(&bar_vf[b]);
      }
    } else {
      // ---------------- load warp.  64 rows per request: rows of one layer by two tensor-map copies,
      // a tile mixing text and visual rows of a VLA lazy layer row by row.
      uint32_t codes[3] = {0u, 0u, 0u};
      if (lazy && !gla) {
        const int n_tiles = (A.T + kTN - 1) / kTN;
#pragma unroll
        for (int i = 0; i < 3; ++i)
          if (lane + 32 * i < n_tiles) codes[i] = A.tile_code[lane + 32 * i];
      }
      auto code_of = [&](int kt) -> int {   // whole warp
        if (kt >= 96) return A.tile_code[kt];
        const uint32_t c = kt < 32 ? codes[0] : (kt < 64 ? codes[1] : codes[2]);
        return static_cast<int>(__shfl_sync(0xffffffffu, c, kt & 31));
      };
      // which: 0 = query rows, 1 = key rows, 2 = value rows; kt64 counts 64-token tiles of the prompt
      auto fetch64 = [&](int which, int kt64, uint32_t dst, uint64_t* bar) {
        int src = layer;
        bool mixed = false;
        if (which != 2 && lazy && kt64 * kTN < A.T) {
          if (gla) {
            src = lead;
          } else {
            const int code = code_of(kt64);
            mixed = code == 2;
            src = code == 1 ? lead : layer;
          }
        }
        if (!mixed) {
          if (lane == 0) {
            const void* tm = which == 0 ? static_cast<const void*>(&A.tmap_q)
                                        : (which == 1 ? static_cast<const void*>(&A.tmap_k) : static_cast<const void*>(&A.tmap_v));
            const int h = which == 0 ? head : kvh;
            mbar_expect_tx(bar, 2 * kTN * 128);
            tensor_g2s_3d(dst, tm, 0, h, src * A.T + kt64 * kTN, bar);
            tensor_g2s_3d(dst + kPairHalf, tm, 64, h, src * A.T + kt64 * kTN, bar);
          }
        } else {
          const uint16_t* from = which == 0 ? A.q : A.k;
          const int heads = which == 0 ? A.hq : A.hkv, h = which == 0 ? head : kvh;
          for (int e = lane; e < kTN * (kTD / 8); e += 32) {
            const int r = e >> 4, c = e & 15, t = kt64 * kTN + r;
            const uint32_t d = dst + (c >> 3) * kPairHalf + r * 128 + (((c & 7) ^ (r & 7)) << 4);
            if (t < A.T) {
              const int l = A.kind[t] ? lead : layer;
              cp_async16(d, from + ((static_cast<size_t>(l) * A.T + t) * heads + h) * kTD + c * 8);
            } else {
              asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(d), "r"(0u) : "memory");
            }
          }
          cp_async_commit();
          cp_async_wait<0>();
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar);
        }
      };
      auto fetch128 = [&](int which, int tile, uint32_t dst, uint64_t* bar) {
        fetch64(which, 2 * tile, dst, bar);
        fetch64(which, 2 * tile + 1, dst + kTN * 128, bar);
      };
      fetch128(0, 2 * qp, sQ, &bar_q[0]);
      fetch128(1, 0, sK, &bar_k[0]);
      if (n_kt1 > 0) fetch128(0, 2 * qp + 1, sQ + kPairQT, &bar_q[1]);
      fetch128(2, 0, sV, &bar_v[0]);
      if (n_ktiles > 1) {
        fetch128(1, 1, sK + kPairKT, &bar_k[1]);
        fetch128(2, 1, sV + kPairKT, &bar_v[1]);
      }
      int k_next = 2, v_next = 2;
      uint32_t ph_kf = 0, ph_vf = 0, idle = 0;   // bit b: the phase of barrier b
      while ((k_next < n_ktiles || v_next < n_ktiles) && ok) {
        bool progress = false;
        if (k_next < n_ktiles) {
          const int b = k_next & 1;
          if (__all_sync(0xffffffffu, mbar_test_wait(&bar_kf[b], (ph_kf >> b) & 1u))) {
            ph_kf ^= 1u << b;
            fetch128(1, k_next, sK + b * kPairKT, &bar_k[b]);
            ++k_next;
            progress = true;
          }
        }
        if (v_next < n_ktiles) {
          const int b = v_next & 1;
          if (__all_sync(0xffffffffu, mbar_test_wait(&bar_vf[b], (ph_vf >> b) & 1u))) {
            ph_vf ^= 1u << b;
            fetch128(2, v_next, sV + b * kPairKT, &bar_v[b]);
            ++v_next;
            progress = true;
          }
        }
        if (progress) {
          idle = 0;
        } else if (++idle > (1u << 20) || ((idle & 1023u) == 0 && failed)) {
          ok = false;
        }
      }
    }
    if (!ok) failed = 1;
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ softmax threads of query tile t
    asm volatile("setmaxnreg.inc.sync.aligned.u32 224;" ::: "memory");
    const int t = warp >> 2, tid = threadIdx.x & (kTM - 1);
    const int n_mine = t ? n_kt1 : n_kt0;
    const int m0 = (2 * qp + t) * kTM;
    const int row = m0 + tid;
    const uint32_t t_row = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);   // this warp's 32 TMEM lanes
    const uint32_t cS = t * kPN, cO = 2 * kPN + t * kTD;
    float m_ref = -INFINITY, l_sum = 0.f;
    uint32_t ph_s = 0;
    bool ok = true;
    // The two tiles take turns at the softmax arithmetic (named barriers 3 + t: tile t may start its
    // iteration kt once the other tile has finished the iteration before it in the order (0, 0),
    // (1, 0), (0, 1), (1, 1), ...), so that one tile's exponentials run while the other tile's
    // products do; left to themselves both tiles' scores complete together and the tensor core idles
    // while both compute.  A tile with no predecessor left does not wait.
    const int n_other = t ? n_kt0 : n_kt1;
    auto pass_turn = [&]() {
      if (t == 0) asm volatile("bar.arrive 4, %0;" ::"n"(2 * kTM) : "memory");
      else asm volatile("bar.arrive 3, %0;" ::"n"(2 * kTM) : "memory");
    };
    for (int kt = 0; kt < n_mine; ++kt) {
      if (failed) { ok = false; break; }
      if (!__all_sync(0xffffffffu, mbar_try_wait(&bar_s[t], ph_s))) {
        ok = bounded_wait(&bar_s[t], ph_s) && !failed;
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      }
      ph_s ^= 1u;
      if (t == 0) {
        if (kt > 0 && n_other > 0) asm volatile("bar.sync 3, %0;" ::"n"(2 * kTM) : "memory");
      } else {
        if (kt < n_other) asm volatile("bar.sync 4, %0;" ::"n"(2 * kTM) : "memory");
      }
      tc5_fence_after();
      float p[kPN];
      {
        uint32_t r0[32], r1[32], r2[32], r3[32];
        tmem_ld32_nowait(t_row + cS, r0);
        tmem_ld32_nowait(t_row + cS + 32, r1);
        tmem_ld32_nowait(t_row + cS + 64, r2);
        tmem_ld32_nowait(t_row + cS + 96, r3);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          p[j] = __uint_as_float(r0[j]), p[32 + j] = __uint_as_float(r1[j]);
          p[64 + j] = __uint_as_float(r2[j]), p[96 + j] = __uint_as_float(r3[j]);
        }
      }
      const int n0 = kt * kPN;
      if (n0 + kPN - 1 > m0 || n0 + kPN > A.T) {   // only tiles on the diagonal or at the end of the prompt need the mask
#pragma unroll
        for (int j = 0; j < kPN; ++j) {
          const int key = n0 + j;
          if (!(key <= row && key < A.T)) p[j] = -INFINITY;
        }
      }
      float mx[4] = {p[0], p[1], p[2], p[3]};
#pragma unroll
      for (int j = 4; j < kPN; ++j) mx[j & 3] = fmaxf(mx[j & 3], p[j]);
      const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * A.scale_log2;   // the scale is positive
      float corr = 1.f;
      if (m_tile > m_ref + kRescaleThreshold || m_ref == -INFINITY) {
        if (m_tile != -INFINITY) {
          corr = exp2f(m_ref - m_tile);     // 0 on the first tile
          m_ref = m_tile;
        }
      }
      const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
      if (kt > 0 && __any_sync(0xffffffffu, corr != 1.f)) {   // rare: move the accumulator to the new reference
        ok = bounded_wait(&bar_o[t], static_cast<uint32_t>(kt - 1) & 1u) && !failed;   // PV_t(kt - 1) complete
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
        tc5_fence_after();
#pragma unroll
        for (int c = 0; c < kTD / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(t_row + cO + 32 * c, r);
#pragma unroll
          for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * corr);
          tmem_st32(t_row + cO + 32 * c, r);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      }
      // ---- weights as the A operand, in place of the scores just read: 128 bf16 = 64 columns of this row's
      // lane, handed over in two halves so that the value products of keys 0..63 run during the
      // exponentials of keys 64..127
      float ps[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int h = 0; h < 2; ++h) {
#pragma unroll
        for (int j = 64 * h; j < 64 * h + 64; ++j) {
          p[j] = ex2_approx(fmaf(p[j], A.scale_log2, neg_m));
          ps[j & 3] += p[j];
        }
        if (h == 1 && (t == 0 ? n_other > 0 : kt + 1 < n_other)) pass_turn();   // the other tile's next iteration may start
        uint32_t w[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) w[j] = pack_bf16x2(p[64 * h + 2 * j], p[64 * h + 2 * j + 1]);
        tmem_st32(t_row + cS + 32 * h, w);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        tc5_fence_before();
        mbar_arrive(h ? &bar_pb[t] : &bar_p[t]);
      }
      l_sum = l_sum * corr + ((ps[0] + ps[1]) + (ps[2] + ps[3]));
    }
    if (!ok) {   // leaving early: the other tile must not wait for this one's turn
      failed = 1;
      __threadfence_block();
      pass_turn();
    }
    if (n_mine > 0) {
      if (ok) ok = bounded_wait(&bar_o[t], static_cast<uint32_t>(n_mine - 1) & 1u) && !failed;   // the last value product
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        // scale the accumulator and put the tile into query tile t's shared memory (free: every product
        // of the tile has completed) in the swizzled layout of a 128-row box; two tensor-map stores
        tc5_fence_after();
        const float inv = 1.f / l_sum;
        const uint32_t sQt = sQ + t * kPairQT;
        const uint32_t orow = sQt + tid * 128;
        const uint32_t sw = tid & 7;
#pragma unroll
        for (int c = 0; c < kTD / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(t_row + cO + 32 * c, r);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int chunk = 4 * c + j;   // 16-byte chunk of the 256-byte row
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(orow + (chunk >> 3) * kPairHalf + (((chunk & 7) ^ sw) << 4)),
                         "r"(pack_bf16x2(__uint_as_float(r[8 * j + 0]) * inv, __uint_as_float(r[8 * j + 1]) * inv)),
                         "r"(pack_bf16x2(__uint_as_float(r[8 * j + 2]) * inv, __uint_as_float(r[8 * j + 3]) * inv)),
                         "r"(pack_bf16x2(__uint_as_float(r[8 * j + 4]) * inv, __uint_as_float(r[8 * j + 5]) * inv)),
                         "r"(pack_bf16x2(__uint_as_float(r[8 * j + 6]) * inv, __uint_as_float(r[8 * j + 7]) * inv))
                         : "memory");
          }
        }
        fence_proxy_async();
        if (t == 0) asm volatile("bar.sync 1, %0;" ::"n"(kTM) : "memory");   // the tile's 128 softmax threads
        else asm volatile("bar.sync 2, %0;" ::"n"(kTM) : "memory");
        if (tid == 0) {
          tensor_s2g_4d(&A.tmap_o, sQt, 0, head, m0, layer);
          tensor_s2g_4d(&A.tmap_o, sQt + kPairHalf, 64, head, m0, layer);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // shared memory is released at exit
        }
      } else {
        failed = 1;
        if (lane == 0) atomicMax(err, kErrTimeout);
        if (t == 0) asm volatile("bar.arrive 1, %0;" ::"n"(kTM) : "memory");   // do not hold the tile's other softmax warps
        else asm volatile("bar.arrive 2, %0;" ::"n"(kTM) : "memory");
      }
    }
  }
  tc5_fence_before();
  __syncthreads();
  if (warp == 8) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

constexpr int kSharedPassLayers = kPrefillSharedLayers;   // 3 x 128 + 2 x 64 columns = all of tensor memory
constexpr int prefill_tcgen05_smem_bytes(int nv = 1) { return 2 * kTM * 128 + (2 + 2 * nv) * (2 * kTN * 128) + 128; }

template <int D>
constexpr int prefill_smem_bytes() {
  return 5 * kBN * D * 2;
}

}  // namespace

cudaError_t configure_prefill_kernels() {
  cudaError_t e = cudaFuncSetAttribute(prefill_attend_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       prefill_smem_bytes<128>());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(prefill_attend_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           prefill_smem_bytes<64>());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(prefill_attend_tcgen05_kernel<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           prefill_tcgen05_smem_bytes());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(prefill_attend_tcgen05_kernel<false, 1>, cudaFuncAttributePreferredSharedMemoryCarveout,
                           cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(prefill_attend_tcgen05_kernel<true, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           prefill_tcgen05_smem_bytes());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(prefill_attend_tcgen05_kernel<true, 1>, cudaFuncAttributePreferredSharedMemoryCarveout,
                           cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(prefill_attend_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           prefill_pair_smem_bytes());
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(prefill_attend_tcgen05_kernel<false, kSharedPassLayers>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, prefill_tcgen05_smem_bytes(kSharedPassLayers));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(prefill_attend_tcgen05_kernel<false, kSharedPassLayers>,
                              cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
}

cudaError_t launch_prefill_attend(const Params& p, const uint8_t* kind_dev, const uint8_t* layer_kind_dev,
                                  const uint8_t* leader_dev, const void* q, const void* k, const void* v, void* out,
                                  int32_t T, int32_t gla, const PrefillMaps* maps,
                                  const uint8_t* tile_code_dev, int32_t seq_id, int32_t n0_text, int32_t n0_vis,
                                  const PrefillPass* passes_dev, int32_t n_single, int32_t n_shared,
                                  int32_t pair_min_tokens, cudaStream_t stream) {
  if (T <= 0) return cudaSuccess;
  PrefillArgs a{};
  a.q = static_cast<const uint16_t*>(q);
  a.k = static_cast<const uint16_t*>(k);
  a.v = static_cast<const uint16_t*>(v);
  a.out = static_cast<uint16_t*>(out);
  a.kind = kind_dev;
  a.layer_kind = layer_kind_dev;
  a.leader = leader_dev;
  a.T = T;
  a.hq = p.hq;
  a.hkv = p.hkv;
  a.group = p.group;
  a.n_layers = p.n_layers;
  a.gla = gla;
  a.scale_log2 = p.scale_log2;
  a.pool = p.pool;
  a.table = p.table;
  a.layer_flags = p.layer_flags;
  a.max_seqs = p.max_seqs;
  a.max_pages = p.max_pages;
  a.seq_id = seq_id;
  a.n0_text = n0_text;
  a.n0_vis = n0_vis;
  if (p.d == kTD && maps) {
    a.tmap_pool = p.tmap;
    a.n_pool_pages = p.n_pool_pages;
    a.tmap_q = maps->q;
    a.tmap_k = maps->k;
    a.tmap_v = maps->v;
    a.tmap_o = maps->out;
    a.tile_code = tile_code_dev;
    const dim3 grid5((T + kTM - 1) / kTM, p.hq, p.n_layers);
    // prompts that start a sequence, from pair_min_tokens on: two query tiles per CTA, 128-key tiles
    const bool pair = pair_min_tokens > 0 && T >= pair_min_tokens;
    const dim3 gridp((T + 2 * kTM - 1) / (2 * kTM), p.hq, p.n_layers);
    if (n0_text + n0_vis > 0) {
      prefill_attend_tcgen05_kernel<true, 1><<<grid5, kTc5Threads, prefill_tcgen05_smem_bytes(), stream>>>(a, p.err);
    } else if (passes_dev && n_shared > 0) {
      // the layers that share nothing, then the shared-score passes (passes_dev lists them in that order)
      a.passes = passes_dev;
      if (n_single > 0 && pair) {
        const dim3 g1(gridp.x, gridp.y, n_single);
        prefill_attend_pair_kernel<<<g1, kPairThreads, prefill_pair_smem_bytes(), stream>>>(a, p.err);
      } else if (n_single > 0) {
        const dim3 g1(grid5.x, grid5.y, n_single);
        prefill_attend_tcgen05_kernel<false, 1><<<g1, kTc5Threads, prefill_tcgen05_smem_bytes(), stream>>>(a, p.err);
      }
      a.passes = passes_dev + n_single;
      const dim3 g3(grid5.x, grid5.y, n_shared);
      prefill_attend_tcgen05_kernel<false, kSharedPassLayers>
          <<<g3, kTc5Threads + 32, prefill_tcgen05_smem_bytes(kSharedPassLayers), stream>>>(a, p.err);
    } else if (pair) {
      prefill_attend_pair_kernel<<<gridp, kPairThreads, prefill_pair_smem_bytes(), stream>>>(a, p.err);
    } else {
      prefill_attend_tcgen05_kernel<false, 1><<<grid5, kTc5Threads, prefill_tcgen05_smem_bytes(), stream>>>(a, p.err);
    }
    return cudaGetLastError();
  }
  const dim3 grid((T + kBM - 1) / kBM, p.hq, p.n_layers);
  if (p.d == 128)
    prefill_attend_kernel<128><<<grid, kPrefillThreads, prefill_smem_bytes<128>(), stream>>>(a);
  else
    prefill_attend_kernel<64><<<grid, kPrefillThreads, prefill_smem_bytes<64>(), stream>>>(a);
  return cudaGetLastError();
}

}  // namespace qc
