// Parameters and launcher of the streaming feature-map kernel.
#pragma once

#include "less_internal.cuh"

namespace less {

struct FmParams {
  const __half* x[2];     // q [B, L, Hh[0], D], k [B, L, Hh[1], D]
  const __half* w1[2];    // W_phi1, W_psi1             [L, Hd, D, Rp]
  const __half* w2[2];    // W_phi2, W_psi2             [L, Hd, Rp, R]
  const __half* w3;       // W_psi3                     [L, Hd, R, R]
  const float* psi_scale; // [L, Hd, 2] or null
  float* out[2];          // phi_q [B, L, Hh[0], R], psi_k [B, L, Hh[1], R]
  int B, L, Hd, Rp;
  int D;                  // head dimension (128; 64 on the general path)
  int Hh[2];              // heads of each map per layer: query heads for phi (Hd * group), KV heads for psi
  int lh0, nlh;           // (layer, KV head) range of this launch: [lh0, lh0 + nlh) of L * Hd (tensor-core kernels)
  int x_plain;            // small-batch tensor-core kernel: a warp fetches the q / k rows with plain loads (they may
                          // lie in pinned host memory) instead of TMA
  uint32_t* feat_flag;    // per-head counters to publish phi / psi through (psi's start at flag_stride), or null
  int flag_stride;
};

bool feature_gemv_supported(const Dims& d);
int launch_feature_gemv(less_ctx* c, const FmParams& p, cudaStream_t s);

// tensor-core weight-streaming kernel (feature_tc.cu)
bool feature_tc_supported(const Dims& d);
int launch_feature_tc(less_ctx* c, const FmParams& p, cudaStream_t s);

}  // namespace less
