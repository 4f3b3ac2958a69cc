// The per-head feature-map MLP (Eq. 1, Eq. 2) evaluated on CUDA cores for a few
// rows at a time; shared by the decode-step kernel and the prompt state build.
#pragma once

#include "less_internal.cuh"

namespace less {

constexpr int FM_THREADS = 256;
constexpr int FM_BR = 4;

// One MLP evaluation for `nb` rows already staged in xs (fp32 [FM_BR][D], D = head dimension, a
// multiple of FM_THREADS / (Rp / 8)).
// part: [FM_THREADS / (Rp/8)][FM_BR][Rp] floats, hs: [FM_BR][Rp] floats.
// Result: lanes < R of warp b (b < nb) return feature r = lane of row b; other threads 0.
template <int R>
__device__ __forceinline__ float mlp_rows(const float* xs, float* part, float* hs, int nb,
                                          const __half* __restrict__ w1,
                                          const __half* __restrict__ w2,
                                          const __half* __restrict__ w3, float c1, float c2,
                                          int Rp, bool is_psi, int D = kHeadDim) {
  const int tid = threadIdx.x;
  const int ncg = Rp >> 3;               // column groups of 8 hidden units
  const int ndg = FM_THREADS / ncg;      // groups along d
  const int cg = tid % ncg, dg = tid / ncg;
  const int dper = D / ndg;
  float acc[FM_BR][8];
#pragma unroll
  for (int b = 0; b < FM_BR; ++b)
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[b][c] = 0.f;
  const __half* wp = w1 + (size_t)(dg * dper) * Rp + cg * 8;
#pragma unroll 8
  for (int dd = 0; dd < dper; ++dd) {
    float wf[8];
    half8_to_float(ldg_readonly(wp + (size_t)dd * Rp), wf);
    const int d = dg * dper + dd;
#pragma unroll
    for (int b = 0; b < FM_BR; ++b) {
      const float xv = xs[b * D + d];
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[b][c] = fmaf(xv, wf[c], acc[b][c]);
    }
  }
#pragma unroll
  for (int b = 0; b < FM_BR; ++b) {
    float4* dst = reinterpret_cast<float4*>(part + ((size_t)dg * FM_BR + b) * Rp + cg * 8);
    dst[0] = make_float4(acc[b][0], acc[b][1], acc[b][2], acc[b][3]);
    dst[1] = make_float4(acc[b][4], acc[b][5], acc[b][6], acc[b][7]);
  }
  __syncthreads();
  for (int e = tid; e < FM_BR * Rp; e += FM_THREADS) {
    float s = 0.f;
    for (int g = 0; g < ndg; ++g) s += part[(size_t)g * FM_BR * Rp + e];   // fixed order
    hs[e] = c1 * gelu_erf(s);
  }
  __syncthreads();
  // layer 2 (+ layer 3 for psi): warp b handles row b
  const int warp = tid >> 5, lane = tid & 31;
  float result = 0.f;
  if (warp < nb) {
    float a2[R];
#pragma unroll
    for (int r = 0; r < R; ++r) a2[r] = 0.f;
    for (int j = lane; j < Rp; j += 32) {
      const float hv = hs[warp * Rp + j];
#pragma unroll
      for (int r8 = 0; r8 < R / 8; ++r8) {
        float wf[8];
        half8_to_float(ldg_readonly(w2 + (size_t)j * R + r8 * 8), wf);
#pragma unroll
        for (int c = 0; c < 8; ++c) a2[r8 * 8 + c] = fmaf(hv, wf[c], a2[r8 * 8 + c]);
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) a2[r] += __shfl_xor_sync(0xffffffffu, a2[r], o);
      a2[r] = c2 * gelu_erf(a2[r]);
    }
    if (!is_psi) {
#pragma unroll
      for (int r = 0; r < R; ++r)
        if (lane == r) result = fabsf(a2[r]);
    } else if (lane < R) {
      float s = 0.f;
#pragma unroll
      for (int r = 0; r < R; ++r) s = fmaf(a2[r], __half2float(w3[r * R + lane]), s);
      result = fabsf(s);
    }
  }
  __syncthreads();   // part / hs may be reused by the caller
  return result;
}


// shared memory (floats) mlp_rows needs besides the FM_BR x 128 staged inputs
__host__ __device__ inline size_t mlp_smem_floats(int Rp) {
  const int ndg = FM_THREADS / (Rp / 8);
  return (size_t)FM_BR * Rp + (size_t)ndg * FM_BR * Rp;
}

}  // namespace less
