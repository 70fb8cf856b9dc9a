// qc_attend_static: split-KV decode attention whose scratch memory is part of the library image.
//
// Some users of this library run where device allocation is off the table: a serving loop
// whose memory budget was carved up at start-up and whose allocator is frozen, a plug-in
// called from inside another framework's execution callback, or code running while a memory
// pool is locked.  They cannot hand the library a freshly allocated workspace, and the
// library must not allocate one for them.  For those callers this file offers one
// self-contained call: plain decode attention (one query token per sequence against a
// contiguous K/V history) that keeps its split-KV partial results in a fixed device array
// compiled into the library.  The price is a hard size limit and no concurrency (see qc.h).
//
// The partial results (running max, sum and weighted value sum of each split) are the only
// scratch the computation needs; the merge kernel overwrites nothing else and reads only
// what the partial kernel of the same call wrote, so nothing has to be cleared between calls.

#include "../../include/qc.h"

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <mutex>

namespace {

constexpr int kMaxRows = QC_STATIC_MAX_ROWS;     // sequences x query heads
constexpr int kSplits = QC_STATIC_SPLITS;        // key ranges per row
constexpr int kMaxD = 128;
constexpr int kRowFloats = kMaxD + 2;            // acc[D], max, sum
constexpr int kWarps = 4;
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress;
// kernels receive the device address obtained from it.
static __device__ __align__(256) float g_static_scratch[kMaxRows * kSplits * kRowFloats];

std::mutex g_mutex;
float* g_scratch_ptr[kMaxDevices] = {};

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
  if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<uint16_t>((u >> 16) | 0x40);
  u += 0x7fffu + ((u >> 16) & 1u);
  return static_cast<uint16_t>(u >> 16);
}

// grid (rows, splits); 4 warps share one split's keys (warp w takes keys w, w+4, ... in
// groups of 4: 8 lanes per key), then combine through shared memory.
template <int D>
__global__ void static_partial_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                                      const uint16_t* __restrict__ v, float* __restrict__ scratch, int n_tokens,
                                      int hq, int hkv, float scale_log2) {
  constexpr int EPL = D / 8, LPR = D / 64;
  const int row = blockIdx.x, split = blockIdx.y;
  const int seq = row / hq, head = row % hq, kvh = head / (hq / hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, kg = lane >> 3, c8 = lane & 7;
  const int per = (n_tokens + kSplits - 1) / kSplits;
  const int t0 = split * per, t1 = min(n_tokens, t0 + per);

  float qf[EPL];
  const uint4* qrow = reinterpret_cast<const uint4*>(q + (static_cast<size_t>(seq) * hq + head) * D);
#pragma unroll
  for (int j = 0; j < LPR; ++j) bf16x8_to_f32(qrow[c8 + 8 * j], &qf[8 * j]);
#pragma unroll
  for (int e = 0; e < EPL; ++e) qf[e] *= scale_log2;

  float m = -INFINITY, l = 0.f, acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  const size_t tok_stride = static_cast<size_t>(hkv) * D;
  const size_t base = (static_cast<size_t>(seq) * n_tokens) * tok_stride + static_cast<size_t>(kvh) * D;
  for (int t = t0 + warp * 4; t < t1; t += kWarps * 4) {
    const int key = t + kg;
    const bool valid = key < t1;
    float kf[EPL], vf[EPL];
    float s = 0.f;
    if (valid) {
      const uint4* kr = reinterpret_cast<const uint4*>(k + base + key * tok_stride);
      const uint4* vr = reinterpret_cast<const uint4*>(v + base + key * tok_stride);
#pragma unroll
      for (int j = 0; j < LPR; ++j) {
        bf16x8_to_f32(kr[c8 + 8 * j], &kf[8 * j]);
        bf16x8_to_f32(vr[c8 + 8 * j], &vf[8 * j]);
      }
#pragma unroll
      for (int e = 0; e < EPL; ++e) s = fmaf(kf[e], qf[e], s);
    }
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    s += __shfl_xor_sync(0xffffffffu, s, 4);
    if (!valid) s = -INFINITY;
    float tmax = fmaxf(s, __shfl_xor_sync(0xffffffffu, s, 8));
    tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 16));
    const float m_new = fmaxf(m, tmax);      // finite: the first key of every group is valid
    const float corr = exp2f(m - m_new);
    const float p = exp2f(s - m_new);
    l = l * corr + p;
    m = m_new;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = valid ? fmaf(p, vf[e], acc[e] * corr) : acc[e] * corr;
  }
  // sum over the 4 key groups of the warp
  l += __shfl_xor_sync(0xffffffffu, l, 8);
  l += __shfl_xor_sync(0xffffffffu, l, 16);
#pragma unroll
  for (int e = 0; e < EPL; ++e) {
    acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 8);
    acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 16);
  }
  __shared__ float sm_acc[kWarps][kMaxD];
  __shared__ float sm_m[kWarps], sm_l[kWarps];
  if (kg == 0) {
#pragma unroll
    for (int j = 0; j < LPR; ++j)
#pragma unroll
      for (int e = 0; e < 8; ++e) sm_acc[warp][64 * j + 8 * c8 + e] = acc[8 * j + e];
    if (c8 == 0) {
      sm_m[warp] = m;
      sm_l[warp] = l;
    }
  }
  __syncthreads();
  float* dst = scratch + (static_cast<size_t>(row) * kSplits + split) * kRowFloats;
  float mm = -INFINITY;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) mm = fmaxf(mm, sm_m[w]);
  if (mm == -INFINITY) {   // an empty split: a neutral partial
    for (int d = threadIdx.x; d < D; d += blockDim.x) dst[d] = 0.f;
    if (threadIdx.x == 0) {
      dst[kMaxD] = -INFINITY;
      dst[kMaxD + 1] = 0.f;
    }
    return;
  }
  for (int d = threadIdx.x; d < D; d += blockDim.x) {
    float a = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) a += sm_acc[w][d] * exp2f(sm_m[w] - mm);
    dst[d] = a;
  }
  if (threadIdx.x == 0) {
    float ls = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) ls += sm_l[w] * exp2f(sm_m[w] - mm);
    dst[kMaxD] = mm;
    dst[kMaxD + 1] = ls;
  }
}

// one warp per row: log-sum-exp merge of the splits, bf16 output
template <int D>
__global__ void static_merge_kernel(const float* __restrict__ scratch, uint16_t* __restrict__ out, int n_rows) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  const float* src = scratch + static_cast<size_t>(row) * kSplits * kRowFloats;
  float mm = -INFINITY;
#pragma unroll
  for (int s = 0; s < kSplits; ++s) mm = fmaxf(mm, src[s * kRowFloats + kMaxD]);
  float ls = 0.f;
  float acc[D / 32];
#pragma unroll
  for (int e = 0; e < D / 32; ++e) acc[e] = 0.f;
#pragma unroll
  for (int s = 0; s < kSplits; ++s) {
    const float w = exp2f(src[s * kRowFloats + kMaxD] - mm);
    ls = fmaf(src[s * kRowFloats + kMaxD + 1], w, ls);
#pragma unroll
    for (int e = 0; e < D / 32; ++e) acc[e] = fmaf(src[s * kRowFloats + lane * (D / 32) + e], w, acc[e]);
  }
  const float inv = 1.f / ls;
#pragma unroll
  for (int e = 0; e < D / 32; ++e)
    out[static_cast<size_t>(row) * D + lane * (D / 32) + e] = f32_to_bf16_rne(acc[e] * inv);
}

}  // namespace

extern "C" int32_t qc_attend_static(int32_t device, void* cuda_stream, const void* q_dev, const void* k_dev,
                                    const void* v_dev, void* out_dev, int32_t n_seqs, int32_t n_tokens,
                                    int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, float softmax_scale) {
  if (!q_dev || !k_dev || !v_dev || !out_dev) return QC_ERR_INVALID_ARG;
  if (device < 0 || device >= kMaxDevices) return QC_ERR_INVALID_ARG;
  if (n_seqs < 1 || n_tokens < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads) return QC_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return QC_ERR_UNSUPPORTED;
  // the fixed scratch bounds the problem size: refuse anything it cannot hold
  if (static_cast<int64_t>(n_seqs) * n_q_heads > kMaxRows) return QC_ERR_INVALID_ARG;
  if (n_tokens > QC_STATIC_MAX_TOKENS) return QC_ERR_INVALID_ARG;
  if (!(softmax_scale >= 0.f) || !isfinite(softmax_scale)) return QC_ERR_INVALID_ARG;
  const void* ptrs[4] = {q_dev, k_dev, v_dev, out_dev};
  for (const void* p : ptrs)
    if (reinterpret_cast<uintptr_t>(p) & 15) return QC_ERR_INVALID_ARG;
  // launch on `device`, then give the calling thread its own current device back
  int caller_device = -1;
  if (cudaGetDevice(&caller_device) != cudaSuccess) return QC_ERR_CUDA;
  struct Restore {
    int device;
    ~Restore() { cudaSetDevice(device); }
  } restore{caller_device};
  if (cudaSetDevice(device) != cudaSuccess) return QC_ERR_CUDA;

  float* scratch = nullptr;
  {
    // first call on this device: resolve the device address of the static array (once)
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_ptr[device]) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return QC_ERR_CUDA;
      g_scratch_ptr[device] = static_cast<float*>(p);
    }
    scratch = g_scratch_ptr[device];
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(head_dim));
  const float scale_log2 = scale * 1.4426950408889634f;
  const int n_rows = n_seqs * n_q_heads;
  const dim3 grid(n_rows, kSplits);
  const uint16_t* q = static_cast<const uint16_t*>(q_dev);
  const uint16_t* k = static_cast<const uint16_t*>(k_dev);
  const uint16_t* v = static_cast<const uint16_t*>(v_dev);
  uint16_t* out = static_cast<uint16_t*>(out_dev);
  if (head_dim == 128) {
    static_partial_kernel<128><<<grid, kWarps * 32, 0, stream>>>(q, k, v, scratch, n_tokens, n_q_heads, n_kv_heads, scale_log2);
    static_merge_kernel<128><<<(n_rows + 3) / 4, 128, 0, stream>>>(scratch, out, n_rows);
  } else {
    static_partial_kernel<64><<<grid, kWarps * 32, 0, stream>>>(q, k, v, scratch, n_tokens, n_q_heads, n_kv_heads, scale_log2);
    static_merge_kernel<64><<<(n_rows + 3) / 4, 128, 0, stream>>>(scratch, out, n_rows);
  }
  return cudaGetLastError() == cudaSuccess ? QC_OK : QC_ERR_CUDA;
}
