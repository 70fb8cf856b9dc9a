// Calibration by-product (paper section "Lazy Attention", Eq. 3): for a cache whose layers are all
// ordinary, the head-averaged attention distribution of one query token per sequence over every
// cached token, layer by layer, and the Jensen-Shannon divergence of adjacent layers'
// distributions.  A one-off analysis pass, not a hot path: plain loads, one CTA per (sequence,
// layer), logits of one head at a time in shared memory.

#include "qc_device.cuh"

namespace qc {
namespace {

constexpr int kCalibThreads = 256;

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float other = __shfl_xor_sync(0xffffffffu, v, o);
    v = is_max ? fmaxf(v, other) : v + other;
  }
  __syncthreads();   // scratch may still be read from a previous reduction
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float r = scratch[0];
  for (int w = 1; w < kCalibThreads / 32; ++w) r = is_max ? fmaxf(r, scratch[w]) : r + scratch[w];
  return r;
}

// rows[layer][si][j], j over the text stream then the visual stream: mean over query heads of
// softmax_j(scale * q_h . k_j).  Entries past the sequence's length are set to zero.
template <int D>
__global__ void __launch_bounds__(kCalibThreads) lastrow_kernel(const Params P, const int32_t* __restrict__ seq_ids,
                                                                const int32_t* __restrict__ len_text,
                                                                const int32_t* __restrict__ len_vis, float* rows,
                                                                int32_t max_len) {
  extern __shared__ float logits[];   // [max_len]
  __shared__ float scratch[kCalibThreads / 32];
  const int si = blockIdx.x, layer = blockIdx.y;
  const int seq_id = seq_ids[si], lt = len_text[si], lv = len_vis[si], L = lt + lv;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* row = rows + (static_cast<size_t>(layer) * gridDim.x + si) * max_len;
  for (int j = threadIdx.x; j < max_len; j += kCalibThreads) row[j] = 0.f;
  constexpr int EPL = D / 32;   // elements of a key row per lane
  const float scale = P.scale_log2 * 0.6931471805599453f;
  for (int h = 0; h < P.hq; ++h) {
    const int kvh = h / P.group;
    float qf[EPL];
    const uint16_t* qp = P.q + ((static_cast<size_t>(layer) * P.n_seqs + si) * P.hq + h) * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; ++e) qf[e] = __uint_as_float(static_cast<uint32_t>(qp[e]) << 16);
    for (int j = warp; j < L; j += kCalibThreads / 32) {
      const int stream = j < lt ? 0 : 1, ord = j < lt ? j : j - lt;
      const int pid = P.table[table_row(P, layer, stream, seq_id) + ord / kPage];
      const uint16_t* kp = P.pool + ((static_cast<size_t>(pid) * P.hkv + kvh) * kPage + ord % kPage) * D + lane * EPL;
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) s = fmaf(qf[e], __uint_as_float(static_cast<uint32_t>(kp[e]) << 16), s);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) logits[j] = s * scale;
    }
    __syncthreads();
    float m = -INFINITY;
    for (int j = threadIdx.x; j < L; j += kCalibThreads) m = fmaxf(m, logits[j]);
    m = block_reduce(m, true, scratch);
    float sum = 0.f;
    for (int j = threadIdx.x; j < L; j += kCalibThreads) sum += expf(logits[j] - m);
    sum = block_reduce(sum, false, scratch);
    const float w = 1.f / (sum * P.hq);
    for (int j = threadIdx.x; j < L; j += kCalibThreads) row[j] += expf(logits[j] - m) * w;   // same thread every head
    __syncthreads();
  }
}

// js[l][si] = 1/2 [KL(a || m) + KL(b || m)], m = (a + b) / 2, a = rows[l][si], b = rows[l + 1][si]
__global__ void __launch_bounds__(kCalibThreads) js_kernel(const float* __restrict__ rows, float* __restrict__ js,
                                                           int32_t max_len) {
  __shared__ float scratch[kCalibThreads / 32];
  const int si = blockIdx.x, l = blockIdx.y, n_seqs = gridDim.x;
  const float* a = rows + (static_cast<size_t>(l) * n_seqs + si) * max_len;
  const float* b = rows + (static_cast<size_t>(l + 1) * n_seqs + si) * max_len;
  float acc = 0.f;
  for (int j = threadIdx.x; j < max_len; j += kCalibThreads) {
    const float x = a[j], y = b[j], m = 0.5f * (x + y);
    if (x > 0.f) acc += x * logf(x / m);
    if (y > 0.f) acc += y * logf(y / m);
  }
  acc = block_reduce(acc, false, scratch);
  if (threadIdx.x == 0) js[l * n_seqs + si] = 0.5f * acc;
}

}  // namespace

cudaError_t launch_calibration(const Params& p, const int32_t* seq_ids_dev, const int32_t* len_text_dev,
                               const int32_t* len_vis_dev, float* rows_dev, int32_t max_len, float* js_dev,
                               cudaStream_t stream) {
  const dim3 grid(p.n_seqs, p.n_layers);
  const size_t smem = static_cast<size_t>(max_len) * sizeof(float);
  cudaError_t e;
  if (p.d == 128) {
    e = cudaFuncSetAttribute(lastrow_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    lastrow_kernel<128><<<grid, kCalibThreads, smem, stream>>>(p, seq_ids_dev, len_text_dev, len_vis_dev, rows_dev, max_len);
  } else {
    e = cudaFuncSetAttribute(lastrow_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    lastrow_kernel<64><<<grid, kCalibThreads, smem, stream>>>(p, seq_ids_dev, len_text_dev, len_vis_dev, rows_dev, max_len);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess || p.n_layers < 2) return e;
  js_kernel<<<dim3(p.n_seqs, p.n_layers - 1), kCalibThreads, 0, stream>>>(rows_dev, js_dev, max_len);
  return cudaGetLastError();
}

}  // namespace qc
