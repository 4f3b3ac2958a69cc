// Parameters shared by the prompt-phase kernels and their launchers.
#pragma once

#include "less_internal.cuh"

namespace less {

struct PfParams {
  const __half* Q;                                      // [B, layer_count, Hd * grp, S, D]
  const __half* K; const __half* V;                     // [B, layer_count, Hd, S, D]
  float* attn_out;                                      // Q's shape or null
  Arena a;
  const __half* w_psi1; const __half* w_psi2; const __half* w_psi3;
  const float* psi_scale;
  int S, Sp, Sbx;            // prompt length, workspace row strides
  int layer0, nl;            // first model layer of this group, layers in the group
  int lj0, layer_count;      // first input layer of this group, layers in the input
  int B, L, Hd, N, Np, heavy, recent, Rp;
  int nsplit, split_tokens;
  int grp;                   // query heads per KV head (Section 3.2, multi-query attention)
  uint32_t flags;
};

struct InstMap {
  size_t in_row0;   // first row (of S) of this instance in Q/K/V, in rows of D
  size_t inst;      // global instance
  int lh;           // layer * Hd + head
};

__device__ __forceinline__ InstMap map_instance(const PfParams& p, int g) {
  const int h = g % p.Hd;
  const int lj = (g / p.Hd) % p.nl;
  const int b = g / (p.Hd * p.nl);
  InstMap m;
  m.in_row0 = (((size_t)b * p.layer_count + p.lj0 + lj) * p.Hd + h) * (size_t)p.S;
  m.inst = ((size_t)b * p.L + p.layer0 + lj) * p.Hd + h;
  m.lh = (p.layer0 + lj) * p.Hd + h;
  return m;
}

// A query head of the group: gq = instance-in-group * grp + head-in-group.  Its Q rows (and
// attention-output rows), and the K / V rows of the KV head it reads.
struct QueryMap {
  size_t q_row0, kv_row0;
};

__device__ __forceinline__ QueryMap map_query(const PfParams& p, int gq) {
  const int g = gq / p.grp, qg = gq - g * p.grp;
  const int h = g % p.Hd;
  const int lj = (g / p.Hd) % p.nl;
  const int b = g / (p.Hd * p.nl);
  const size_t bl = (size_t)b * p.layer_count + p.lj0 + lj;
  QueryMap m;
  m.q_row0 = ((bl * p.Hd + h) * p.grp + qg) * (size_t)p.S;
  m.kv_row0 = (bl * p.Hd + h) * (size_t)p.S;
  return m;
}

// launchers of the tensor-core kernels (score_tc.cu, state_tc.cu, psi_tc.cu)
bool score_tc_supported();
int launch_score_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s, bool with_column_sums);
// prompt attention output from the row statistics launch_score_tc leaves behind (attn_out_tc.cu)
int launch_attn_out_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s);
int launch_state_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s);
bool psi_tc_supported(const Dims& d);
int launch_psi_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s);
int launch_psi_state_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s);   // psi fused with the state build
int launch_phi_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s, float* out);

}  // namespace less
