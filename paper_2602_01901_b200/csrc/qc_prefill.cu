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
  const uint16_t* q;     // [n_layers][T][hq][D]
  const uint16_t* k;     // [n_layers][T][hkv][D]
  const uint16_t* v;     // [n_layers][T][hkv][D]
  uint16_t* out;         // [n_layers][T][hq][D]
  const uint8_t* kind;   // [T] device
  const uint8_t* layer_kind;   // [n_layers] device (QC_LAYER_*)
  const uint8_t* leader;       // [n_layers] device
  int32_t T, hq, hkv, group, n_layers, gla;
  float scale_log2;
};

// Stage rows [row0, row0 + 64) of one head of a [n_layers][T][heads][D] tensor; row t comes
// from layer `own` or, where lead_rows says so, from layer `lead`.  Rows past T are zero-filled.
template <int D>
__device__ __forceinline__ void stage_tile(uint32_t smem, const uint16_t* base, int own, int lead, bool lazy, bool gla,
                                           const uint8_t* kind, int row0, int T, int heads, int head) {
  constexpr int CH = D / 8;
  for (int e = threadIdx.x; e < kBN * CH; e += kPrefillThreads) {
    const int r = e / CH, c = e - r * CH;
    const int t = row0 + r;
    const uint32_t dst = smem + tile_off<D>(r, c);
    if (t < T) {
      const int layer = (lazy && (gla || kind[t])) ? lead : own;
      const uint16_t* src = base + ((static_cast<size_t>(layer) * T + t) * heads + head) * D + c * 8;
      cp_async16(dst, src);
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
  const int n_ktiles = qt + 1;                       // causal: key tiles 0 .. qt

  // stage Q and the first K/V tiles
  stage_tile<D>(sQ, A.q, layer, lead, lazy, gla, A.kind, m0, A.T, A.hq, head);
  stage_tile<D>(sK, A.k, layer, lead, lazy, gla, A.kind, 0, A.T, A.hkv, kvh);
  stage_tile<D>(sV, A.v, layer, layer, false, false, A.kind, 0, A.T, A.hkv, kvh);
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
      stage_tile<D>(sK + (buf ^ 1) * kTileBytes, A.k, layer, lead, lazy, gla, A.kind, (kt + 1) * kBN, A.T, A.hkv, kvh);
      stage_tile<D>(sV + (buf ^ 1) * kTileBytes, A.v, layer, layer, false, false, A.kind, (kt + 1) * kBN, A.T, A.hkv,
                    kvh);
      cp_async_commit();
    }
    const uint32_t kb = sK + buf * kTileBytes, vb = sV + buf * kTileBytes;
    const int n0 = kt * kBN;

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
        const int key = n0 + j * 8 + 2 * t4 + (e & 1);
        const int qrow = qrow0 + ((e >> 1) << 3);
        const float x = (key <= qrow && key < A.T) ? s[j][e] * A.scale_log2 : -INFINITY;
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

template <int D>
constexpr int prefill_smem_bytes() {
  return 5 * kBN * D * 2;
}

}  // namespace

cudaError_t configure_prefill_kernels() {
  cudaError_t e = cudaFuncSetAttribute(prefill_attend_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       prefill_smem_bytes<128>());
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(prefill_attend_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              prefill_smem_bytes<64>());
}

cudaError_t launch_prefill_attend(const Params& p, const uint8_t* kind_dev, const uint8_t* layer_kind_dev,
                                  const uint8_t* leader_dev, const void* q, const void* k, const void* v, void* out,
                                  int32_t T, int32_t gla, cudaStream_t stream) {
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
  const dim3 grid((T + kBM - 1) / kBM, p.hq, p.n_layers);
  if (p.d == 128)
    prefill_attend_kernel<128><<<grid, kPrefillThreads, prefill_smem_bytes<128>(), stream>>>(a);
  else
    prefill_attend_kernel<64><<<grid, kPrefillThreads, prefill_smem_bytes<64>(), stream>>>(a);
  return cudaGetLastError();
}

}  // namespace qc
