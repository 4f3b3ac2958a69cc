// less_prompt_scores_noalloc: the H2O prompt scores (column sums of the causal
// softmax) for callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a
// serving process whose memory pool owns the whole device, in a plugin that is
// handed buffers and a stream and nothing else, or in a region of a program
// where an allocation would synchronise or fail.  Those callers can pass
// inputs and an output, but not the scratch the two-pass scoring needs (one
// row maximum and one reciprocal row sum per prompt token).  Here that scratch
// is a fixed array inside the library image itself.
//
// Consequences of that choice, all part of the contract:
//   * every GPU that loads the library holds the array (512 KB) until exit;
//   * one call handles at most LESS_NOALLOC_MAX_ROWS rows (n_inst * prompt_len);
//   * every call on a device shares the array, so two calls whose kernels can
//     overlap on the GPU (different streams, no ordering) race; calls on one
//     stream are ordered and safe;
//   * nothing in the array has to start at zero: each call overwrites the rows
//     it later reads;
//   * the first call on each device looks up the array's device address; make
//     that first call outside any stream capture.
#include <atomic>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "less.h"

namespace {

constexpr int kD = 128;
constexpr int kTile = 128;
constexpr int kStage = 32;
constexpr float kInvSqrtD = 0.08838834764831845f;
constexpr int kMaxDevices = 64;

// [0, MAX_ROWS): row maxima; [MAX_ROWS, 2*MAX_ROWS): reciprocal row sums
static __device__ __align__(256) float g_noalloc_scratch[2 * LESS_NOALLOC_MAX_ROWS];

// In host code the name above is only a handle; kernels need the address below.  Atomic, so that
// first calls from several host threads may race on the look-up: both find the same address.
std::atomic<float*> g_scratch_addr[kMaxDevices];

__device__ __forceinline__ void row_to_float(float* x, const __half* row) {
#pragma unroll
  for (int c8 = 0; c8 < 16; ++c8) {
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(row) + c8);
    const __half2* h = reinterpret_cast<const __half2*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 p = __half22float2(h[i]);
      x[c8 * 8 + 2 * i] = p.x;
      x[c8 * 8 + 2 * i + 1] = p.y;
    }
  }
}

__device__ __forceinline__ float dot_row(const float* x, const __half* row) {
  float s = 0.f;
#pragma unroll
  for (int c8 = 0; c8 < 16; ++c8) {
    const uint4 u = reinterpret_cast<const uint4*>(row)[c8];
    const __half2* h = reinterpret_cast<const __half2*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 p = __half22float2(h[i]);
      s = fmaf(x[c8 * 8 + 2 * i], p.x, s);
      s = fmaf(x[c8 * 8 + 2 * i + 1], p.y, s);
    }
  }
  return s;
}

__device__ __forceinline__ void stage_rows(__half (*dst)[kD], const __half* src, int first, int S) {
  for (int e = threadIdx.x; e < kStage * 16; e += kTile) {
    const int r = e >> 4, c = e & 15;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (first + r < S) v = __ldg(reinterpret_cast<const uint4*>(src + (size_t)(first + r) * kD) + c);
    reinterpret_cast<uint4*>(&dst[r][0])[c] = v;
  }
}

// pass 1: one thread per query row; m_i and 1/l_i of the causal row into the scratch
__global__ void __launch_bounds__(kTile) noalloc_rowstat_kernel(const __half* Q, const __half* K, int S,
                                                                float* scratch_m, float* scratch_invl) {
  __shared__ __align__(16) __half ks[kStage][kD];
  const int inst = blockIdx.y, i0 = blockIdx.x * kTile, i = i0 + threadIdx.x;
  const __half* Qi = Q + (size_t)inst * S * kD;
  const __half* Ki = K + (size_t)inst * S * kD;
  const bool live = i < S;
  float q[kD];
  if (live) row_to_float(q, Qi + (size_t)i * kD);
  else {
#pragma unroll
    for (int c = 0; c < kD; ++c) q[c] = 0.f;
  }
  float m = -INFINITY, l = 0.f;
  const int jend = min(S, i0 + kTile);
  for (int j0 = 0; j0 < jend; j0 += kStage) {
    stage_rows(ks, Ki, j0, S);
    __syncthreads();
    if (live) {
      const int jmax = min(kStage, i - j0 + 1);
      for (int jj = 0; jj < jmax; ++jj) {
        const float s = dot_row(q, &ks[jj][0]) * kInvSqrtD;
        if (s > m) { l = l * __expf(m - s) + 1.f; m = s; }
        else l += __expf(s - m);
      }
    }
    __syncthreads();
  }
  if (live) {
    scratch_m[(size_t)inst * S + i] = m;
    scratch_invl[(size_t)inst * S + i] = 1.0f / l;
  }
}

// pass 2: one thread per key column; acc_j = sum_{i >= j} exp(s_ij - m_i) / l_i
__global__ void __launch_bounds__(kTile) noalloc_colsum_kernel(const __half* Q, const __half* K, int S,
                                                               const float* scratch_m,
                                                               const float* scratch_invl, float* acc_out) {
  __shared__ __align__(16) __half qs[kStage][kD];
  __shared__ float ms[kStage], ls[kStage];
  const int inst = blockIdx.y, j0 = blockIdx.x * kTile, j = j0 + threadIdx.x;
  const __half* Qi = Q + (size_t)inst * S * kD;
  const __half* Ki = K + (size_t)inst * S * kD;
  const bool live = j < S;
  float k[kD];
  if (live) row_to_float(k, Ki + (size_t)j * kD);
  else {
#pragma unroll
    for (int c = 0; c < kD; ++c) k[c] = 0.f;
  }
  float acc = 0.f;
  for (int i0 = j0; i0 < S; i0 += kStage) {
    stage_rows(qs, Qi, i0, S);
    if (threadIdx.x < kStage) {
      const bool ok = i0 + threadIdx.x < S;
      ms[threadIdx.x] = ok ? scratch_m[(size_t)inst * S + i0 + threadIdx.x] : 0.f;
      ls[threadIdx.x] = ok ? scratch_invl[(size_t)inst * S + i0 + threadIdx.x] : 0.f;
    }
    __syncthreads();
    if (live) {
      const int iimax = min(kStage, S - i0);
      for (int ii = max(0, j - i0); ii < iimax; ++ii)
        acc += __expf(dot_row(k, &qs[ii][0]) * kInvSqrtD - ms[ii]) * ls[ii];
    }
    __syncthreads();
  }
  if (live) acc_out[(size_t)inst * S + j] = acc;
}

}  // namespace

extern "C" int less_prompt_scores_noalloc(const void* Q, const void* K, int32_t n_inst,
                                          int32_t prompt_len, float* acc_out, void* cuda_stream) {
  if (!Q || !K || !acc_out) return LESS_ERR_NULL_POINTER;
  if (((uintptr_t)Q & 15) || ((uintptr_t)K & 15) || ((uintptr_t)acc_out & 3)) return LESS_ERR_MISALIGNED;
  if (n_inst < 0 || prompt_len < 0 || n_inst > 65535) return LESS_ERR_INVALID_CONFIG;
  if ((int64_t)n_inst * prompt_len > LESS_NOALLOC_MAX_ROWS) return LESS_ERR_NOALLOC_TOO_LARGE;
  if (n_inst == 0 || prompt_len == 0) return LESS_OK;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LESS_ERR_CUDA;
  float* sm = g_scratch_addr[dev].load(std::memory_order_relaxed);
  if (!sm) {
    // once per device, with that device current: the device address of the array
    if (cudaGetSymbolAddress((void**)&sm, g_noalloc_scratch) != cudaSuccess || !sm) return LESS_ERR_CUDA;
    g_scratch_addr[dev].store(sm, std::memory_order_relaxed);
  }
  float* sl = sm + LESS_NOALLOC_MAX_ROWS;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const dim3 grid((prompt_len + kTile - 1) / kTile, n_inst);
  noalloc_rowstat_kernel<<<grid, kTile, 0, s>>>((const __half*)Q, (const __half*)K, prompt_len, sm, sl);
  noalloc_colsum_kernel<<<grid, kTile, 0, s>>>((const __half*)Q, (const __half*)K, prompt_len, sm, sl,
                                               acc_out);
  return cudaGetLastError() == cudaSuccess ? LESS_OK : LESS_ERR_CUDA;
}
