// Prompt-phase kernels that run on CUDA cores, and the launcher of the whole prompt phase
// (Section 3.1: regular attention, then the policy once):
//   select_kernel    recent window + `heavy` largest (acc, pos) -> slot of every token (H2O);
//                    first tokens + window (Lambda-masking); N largest of the last row (TOVA)
//   lastrow_kernel   TOVA: the last prompt query's attention probabilities
//   gather_kernel    kept rows -> slots (K, V, position, score, cached psi)
//   finalize_kernel  fixed-order sum of the state build's partial H, z
//   rowstat_kernel, colsum_kernel, attn_out_kernel, psi_kernel
//                    fallbacks of the tensor-core kernels (score_tc.cu, attn_out_tc.cu, psi_tc.cu)
#include "feature_mlp.cuh"
#include "prefill.cuh"

namespace less {

constexpr int PF_TILE = 128;   // rows (or columns) per CTA, one per thread
constexpr int PF_KT = 32;      // rows of the other operand staged per iteration
// The CUDA-core kernels take the head dimension D as a template argument (128, or 64 on the general
// path) and any number of query heads per KV head (PfParams::grp).
template <int D>
__device__ __forceinline__ float inv_sqrt_d() { return D == 64 ? 0.125f : 0.08838834764831845f; }

template <int D>
__device__ __forceinline__ float dot_row(const float* x, const __half* row) {
  float s = 0.f;
#pragma unroll
  for (int c8 = 0; c8 < D / 8; ++c8) {
    float f[8];
    half8_to_float(*reinterpret_cast<const uint4*>(row + c8 * 8), f);
#pragma unroll
    for (int c = 0; c < 8; ++c) s = fmaf(x[c8 * 8 + c], f[c], s);
  }
  return s;
}

template <int D>
__device__ __forceinline__ void load_row(float* x, const __half* row) {
#pragma unroll
  for (int c8 = 0; c8 < D / 8; ++c8)
    half8_to_float(__ldg(reinterpret_cast<const uint4*>(row + c8 * 8)), x + c8 * 8);
}

// ---- P1: row statistics (one grid row per query head) --------------------- //
template <int D>
__global__ void __launch_bounds__(PF_TILE) rowstat_kernel(PfParams p) {
  constexpr int CH = D / 8;
  __shared__ __align__(16) __half ks[PF_KT][D];
  const int gq = blockIdx.y, i0 = blockIdx.x * PF_TILE, tid = threadIdx.x;
  const QueryMap qm = map_query(p, gq);
  const int i = i0 + tid;
  const bool live = i < p.S;
  float q[D];
  if (live) load_row<D>(q, p.Q + (qm.q_row0 + i) * D);
  else {
#pragma unroll
    for (int c = 0; c < D; ++c) q[c] = 0.f;
  }
  float m = -INFINITY, l = 0.f;
  const int jend = min(p.S, i0 + PF_TILE);
  for (int j0 = 0; j0 < jend; j0 += PF_KT) {
    for (int e = tid; e < PF_KT * CH; e += PF_TILE) {
      const int r = e / CH, c = e % CH;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (j0 + r < p.S) v = __ldg(reinterpret_cast<const uint4*>(p.K + (qm.kv_row0 + j0 + r) * D) + c);
      reinterpret_cast<uint4*>(&ks[r][0])[c] = v;
    }
    __syncthreads();
    if (live) {
      const int jmax = min(PF_KT, i - j0 + 1);
      for (int jj = 0; jj < jmax; ++jj) {
        const float s = dot_row<D>(q, &ks[jj][0]) * inv_sqrt_d<D>();
        if (s > m) { l = l * __expf(m - s) + 1.f; m = s; }
        else l += __expf(s - m);
      }
    }
    __syncthreads();
  }
  if (live) {
    p.a.ws_m[(size_t)gq * p.Sp + i] = m;
    p.a.ws_invl[(size_t)gq * p.Sp + i] = 1.0f / l;
  }
}

// ---- P2: column sums, over the rows of all query heads of the KV head ------- //
template <int D>
__global__ void __launch_bounds__(PF_TILE) colsum_kernel(PfParams p) {
  constexpr int CH = D / 8;
  __shared__ __align__(16) __half qs[PF_KT][D];
  __shared__ float ms[PF_KT], ls[PF_KT];
  const int g = blockIdx.y, j0 = blockIdx.x * PF_TILE, tid = threadIdx.x;
  const InstMap im = map_instance(p, g);
  const int j = j0 + tid;
  const bool live = j < p.S;
  float k[D];
  if (live) load_row<D>(k, p.K + (im.in_row0 + j) * D);
  else {
#pragma unroll
    for (int c = 0; c < D; ++c) k[c] = 0.f;
  }
  float acc = 0.f;
  for (int qg = 0; qg < p.grp; ++qg) {
    const int gq = g * p.grp + qg;
    const size_t q_row0 = map_query(p, gq).q_row0;
    for (int i0 = j0; i0 < p.S; i0 += PF_KT) {       // j0 is a multiple of PF_KT
      for (int e = tid; e < PF_KT * CH; e += PF_TILE) {
        const int r = e / CH, c = e % CH;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (i0 + r < p.S) v = __ldg(reinterpret_cast<const uint4*>(p.Q + (q_row0 + i0 + r) * D) + c);
        reinterpret_cast<uint4*>(&qs[r][0])[c] = v;
      }
      if (tid < PF_KT) {
        const bool ok = i0 + tid < p.S;
        ms[tid] = ok ? p.a.ws_m[(size_t)gq * p.Sp + i0 + tid] : 0.f;
        ls[tid] = ok ? p.a.ws_invl[(size_t)gq * p.Sp + i0 + tid] : 0.f;
      }
      __syncthreads();
      if (live) {
        const int iimax = min(PF_KT, p.S - i0);
        for (int ii = max(0, j - i0); ii < iimax; ++ii) {
          const float s = dot_row<D>(k, &qs[ii][0]) * inv_sqrt_d<D>();
          acc += __expf(s - ms[ii]) * ls[ii];
        }
      }
      __syncthreads();
    }
  }
  if (live) p.a.ws_acc[(size_t)g * p.Sp + j] = acc;
}

// ---- optional prompt attention output (one grid row per query head) -------- //
constexpr int AO_ROWS = 8;
template <int D>
__global__ void __launch_bounds__(PF_TILE) attn_out_kernel(PfParams p) {
  constexpr int CH = D / 8;
  __shared__ float qs[AO_ROWS][D];
  __shared__ __align__(16) __half ks[PF_KT][D];
  __shared__ __align__(16) __half vs[PF_KT][D];
  __shared__ float ps[AO_ROWS][PF_KT];
  const int gq = blockIdx.y, i0 = blockIdx.x * AO_ROWS, tid = threadIdx.x;
  const QueryMap qm = map_query(p, gq);
  for (int e = tid; e < AO_ROWS * D; e += PF_TILE) {
    const int r = e / D, c = e % D;
    qs[r][c] = (i0 + r < p.S) ? __half2float(p.Q[(qm.q_row0 + i0 + r) * D + c]) : 0.f;
  }
  float o[AO_ROWS];
#pragma unroll
  for (int r = 0; r < AO_ROWS; ++r) o[r] = 0.f;
  const int jend = min(p.S, i0 + AO_ROWS);
  for (int j0 = 0; j0 < jend; j0 += PF_KT) {
    __syncthreads();
    for (int e = tid; e < PF_KT * CH; e += PF_TILE) {
      const int r = e / CH, c = e % CH;
      uint4 kv = make_uint4(0, 0, 0, 0), vv = kv;
      if (j0 + r < p.S) {
        kv = __ldg(reinterpret_cast<const uint4*>(p.K + (qm.kv_row0 + j0 + r) * D) + c);
        vv = __ldg(reinterpret_cast<const uint4*>(p.V + (qm.kv_row0 + j0 + r) * D) + c);
      }
      reinterpret_cast<uint4*>(&ks[r][0])[c] = kv;
      reinterpret_cast<uint4*>(&vs[r][0])[c] = vv;
    }
    __syncthreads();
    for (int e = tid; e < AO_ROWS * PF_KT; e += PF_TILE) {
      const int r = e / PF_KT, jj = e % PF_KT;
      const int i = i0 + r, j = j0 + jj;
      float pr = 0.f;
      if (i < p.S && j <= i) {
        const float s = dot_row<D>(&qs[r][0], &ks[jj][0]) * inv_sqrt_d<D>();
        pr = __expf(s - p.a.ws_m[(size_t)gq * p.Sp + i]) * p.a.ws_invl[(size_t)gq * p.Sp + i];
      }
      ps[r][jj] = pr;
    }
    __syncthreads();
    if (tid < D) {
      for (int jj = 0; jj < PF_KT; ++jj) {
        const float vv = __half2float(vs[jj][tid]);
#pragma unroll
        for (int r = 0; r < AO_ROWS; ++r) o[r] = fmaf(ps[r][jj], vv, o[r]);
      }
    }
  }
  if (tid < D) {
#pragma unroll
    for (int r = 0; r < AO_ROWS; ++r)
      if (i0 + r < p.S) p.attn_out[(qm.q_row0 + i0 + r) * D + tid] = o[r];
  }
}

// ---- TOVA: the last prompt query's attention probabilities ------------------- //
// p_j = softmax_j( q_{S-1} . k_j / sqrt(D) ) over the whole prompt, into ws_acc.  One CTA per
// instance: scores, block maximum, exponentials and their block sum, normalisation in place.
constexpr int LR_THREADS = 1024;
template <int D>
__global__ void __launch_bounds__(LR_THREADS) lastrow_kernel(PfParams p) {
  __shared__ float qs[D];
  __shared__ float red[LR_THREADS / 32];
  const int g = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const InstMap im = map_instance(p, g);
  float* pr = p.a.ws_acc + (size_t)g * p.Sp;
  if (tid < D) qs[tid] = __half2float(p.Q[(im.in_row0 + p.S - 1) * D + tid]);
  __syncthreads();
  float m = -INFINITY;
  for (int j = tid; j < p.S; j += LR_THREADS) {
    const float s = dot_row<D>(qs, p.K + (im.in_row0 + j) * D) * inv_sqrt_d<D>();
    pr[j] = s;
    m = fmaxf(m, s);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) red[warp] = m;
  __syncthreads();
  m = red[0];
  for (int w = 1; w < LR_THREADS / 32; ++w) m = fmaxf(m, red[w]);
  __syncthreads();
  float l = 0.f;
  for (int j = tid; j < p.S; j += LR_THREADS) {
    const float e = __expf(pr[j] - m);
    pr[j] = e;
    l += e;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
  if (lane == 0) red[warp] = l;
  __syncthreads();
  l = 0.f;
  for (int w = 0; w < LR_THREADS / 32; ++w) l += red[w];      // fixed order
  const float inv = 1.0f / l;
  for (int j = tid; j < p.S; j += LR_THREADS) pr[j] *= inv;
}

// ---- P3: selection --------------------------------------------------------- //
constexpr int SEL_THREADS = 1024;

// exclusive block scan of one int per thread; returns the exclusive prefix and the total
__device__ __forceinline__ int block_exscan(int v, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = warp_sums[lane];
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    warp_sums[lane] = winc - w;            // exclusive
    if (lane == 31) warp_sums[32] = winc;  // total
  }
  __syncthreads();
  const int ex = inc - v + warp_sums[warp];
  *total = warp_sums[32];
  __syncthreads();
  return ex;
}

__global__ void __launch_bounds__(SEL_THREADS) select_kernel(PfParams p) {
  __shared__ int hist[256];
  __shared__ int wsum[33];
  __shared__ unsigned int s_prefix;
  __shared__ int s_need;
  const int g = blockIdx.x, tid = threadIdx.x;
  const InstMap im = map_instance(p, g);
  const float* acc = p.a.ws_acc + (size_t)g * p.Sp;
  int32_t* slot_of = p.a.ws_slot + (size_t)g * p.Sp;
  const int S = p.S, N = p.N;
  if (tid == 0) {
    p.a.count[im.inst] = min(S, N);
    p.a.ws_pmax[g] = 0;                          // the psi kernels that follow take the maximum into it
    if (g == 0) { p.a.tpos[0] = S; p.a.tpos[1] = 0; }   // the first decode token has position S
  }
  if (S <= N) {
    for (int j = tid; j < S; j += SEL_THREADS) slot_of[j] = j;
    return;
  }
  if (p.flags & LESS_POLICY_LAMBDA) {
    // Lambda-masking (Section 4): the first `heavy` positions and the last `recent` stay
    for (int j = tid; j < S; j += SEL_THREADS)
      slot_of[j] = j < p.heavy ? j : (j >= S - p.recent ? p.heavy + j - (S - p.recent) : -1);
    return;
  }
  // TOVA protects no window and ranks every position by the last query's probabilities
  const bool tova = (p.flags & LESS_POLICY_TOVA) != 0;
  const int heavy = tova ? N : p.heavy;
  const int C = tova ? S : S - p.recent;         // candidates: positions [0, C)
  unsigned int thr = 0xffffffffu;                // threshold bit pattern (acc >= 0: monotone)
  int need = 0;                                  // how many of the == threshold to keep
  if (heavy > 0) {
    // radix select: the heavy-th largest accumulated score among the candidates
    if (tid == 0) { s_prefix = 0; s_need = heavy; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      const unsigned int prefix = s_prefix;
      const unsigned int himask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
      for (int j = tid; j < C; j += SEL_THREADS) {
        const unsigned int b = __float_as_uint(acc[j]);
        if ((b & himask) == prefix) atomicAdd(&hist[(b >> shift) & 255], 1);
      }
      __syncthreads();
      if (tid == 0) {
        int k = s_need, bin = 255;
        for (; bin > 0; --bin) {
          if (hist[bin] >= k) break;
          k -= hist[bin];
        }
        s_prefix = prefix | ((unsigned int)bin << shift);
        s_need = k;
      }
      __syncthreads();
    }
    thr = s_prefix;
    need = s_need;
  }
  // ties at the threshold: the lowest positions go first (key (acc, pos) ascending),
  // so the `need` HIGHEST positions among the equals stay.
  const int per = (S + SEL_THREADS - 1) / SEL_THREADS;
  const int jb = tid * per, je = min(S, jb + per);
  int eq = 0;
  for (int j = jb; j < je; ++j) eq += (j < C && __float_as_uint(acc[j]) == thr) ? 1 : 0;
  int eq_total;
  int eq_before = block_exscan(eq, wsum, &eq_total);
  const int drop_eq = eq_total - need;           // equals with fewer than this many below them are evicted
  int kept = 0;
  for (int j = jb; j < je; ++j) {
    bool k;
    if (j >= C) k = true;
    else {
      const unsigned int b = __float_as_uint(acc[j]);
      if (b == thr) { k = eq_before >= drop_eq; ++eq_before; }
      else k = heavy > 0 && b > thr;
    }
    kept += k ? 1 : 0;
  }
  int kept_total;
  int slot = block_exscan(kept, wsum, &kept_total);
  // second walk assigns slots in ascending position
  eq_before = 0;
  {
    // recompute this thread's exclusive count of equals (block_exscan result was consumed)
    int dummy;
    eq_before = block_exscan(eq, wsum, &dummy);
  }
  for (int j = jb; j < je; ++j) {
    bool k;
    if (j >= C) k = true;
    else {
      const unsigned int b = __float_as_uint(acc[j]);
      if (b == thr) { k = eq_before >= drop_eq; ++eq_before; }
      else k = heavy > 0 && b > thr;
    }
    slot_of[j] = k ? slot++ : -1;
  }
  if (tid == 0 && kept_total != N) set_status(p.a.status, kStatusBounds, 3);
}

// ---- P5: psi(k_j) of every prompt token (CUDA-core MLP) -------------------- //
template <int R, int D>
__global__ void __launch_bounds__(FM_THREADS) psi_kernel(PfParams p) {
  extern __shared__ float bsm[];
  float* xs = bsm;                              // [FM_BR][D]
  float* hs = xs + FM_BR * D;
  float* part = hs + FM_BR * p.Rp;
  const int split = blockIdx.x, g = blockIdx.y, tid = threadIdx.x;
  const InstMap im = map_instance(p, g);
  const int jbeg = split * p.split_tokens, jend = min(p.S, jbeg + p.split_tokens);
  float c1 = 1.f, c2 = 1.f;
  if (p.psi_scale) { c1 = p.psi_scale[im.lh * 2]; c2 = p.psi_scale[im.lh * 2 + 1]; }
  const __half* w1 = p.w_psi1 + (size_t)im.lh * D * p.Rp;
  const __half* w2 = p.w_psi2 + (size_t)im.lh * p.Rp * R;
  const __half* w3 = p.w_psi3 + (size_t)im.lh * R * R;
  float* psi = p.a.ws_psi + (size_t)g * p.Sp * R;
  float pmax = 0.f;
  for (int j0 = jbeg; j0 < jend; j0 += FM_BR) {
    const int nb = min(FM_BR, jend - j0);
    for (int e = tid; e < FM_BR * D; e += FM_THREADS) {
      const int b = e / D, d = e % D;
      xs[e] = b < nb ? __half2float(p.K[(im.in_row0 + j0 + b) * D + d]) : 0.f;
    }
    __syncthreads();
    const float r = mlp_rows<R>(xs, part, hs, nb, w1, w2, w3, c1, c2, p.Rp, true, D);
    const int warp = tid >> 5, lane = tid & 31;
    if (warp < nb && lane < R) {
      psi[(size_t)(j0 + warp) * R + lane] = r;
      pmax = fmaxf(pmax, r);
    }
  }
  // psi >= 0: its bit pattern orders like an integer, and a maximum does not depend on the order
  if (pmax > 0.f && pmax < INFINITY) atomicMax(p.a.ws_pmax + g, __float_as_int(pmax));
}

// ---- P4: kept rows go to their slots (K, V, position, score, psi) ----------- //
constexpr int GA_THREADS = 256;
template <int R, int D>
__global__ void __launch_bounds__(GA_THREADS) gather_kernel(PfParams p) {
  constexpr int CH = D / 8;                          // 16-byte chunks per row
  const int g = blockIdx.y, tid = threadIdx.x;
  const InstMap im = map_instance(p, g);
  const bool use_state = !(p.flags & LESS_NO_STATE);
  const int32_t* slot_of = p.a.ws_slot + (size_t)g * p.Sp;
  const float* acc = p.a.ws_acc + (size_t)g * p.Sp;
  const float* psi = p.a.ws_psi + (size_t)g * p.Sp * R;
  // 32 threads per token: CH move the K row, CH the V row
  const int sub = tid & 31;
  for (int j = blockIdx.x * (GA_THREADS / 32) + (tid >> 5); j < p.S; j += gridDim.x * (GA_THREADS / 32)) {
    const int sl = slot_of[j];
    if (sl < 0) continue;
    if (sl >= p.N) {
      if (sub == 0) set_status(p.a.status, kStatusBounds, 4);
      continue;
    }
    const size_t dst = (im.inst * (size_t)p.N + sl) * D;
    const size_t src = (im.in_row0 + j) * D;
    if (sub < CH)
      reinterpret_cast<uint4*>(p.a.kslots + dst)[sub] = __ldg(reinterpret_cast<const uint4*>(p.K + src) + sub);
    else if (sub >= 16 && sub < 16 + CH)
      reinterpret_cast<uint4*>(p.a.vslots + dst)[sub - 16] =
          __ldg(reinterpret_cast<const uint4*>(p.V + src) + (sub - 16));
    if (sub == 0) {
      p.a.pos[im.inst * (size_t)p.Np + sl] = j;
      p.a.acc[im.inst * (size_t)p.Np + sl] = (p.flags & LESS_POLICY_LAMBDA) ? 0.f : acc[j];   // no scores under Lambda-masking
    }
    if (sub < R) p.a.psic[(im.inst * (size_t)p.N + sl) * R + sub] = use_state ? psi[(size_t)j * R + sub] : 0.f;
  }
}

template <int R, int D>
__global__ void __launch_bounds__(D) finalize_kernel(PfParams p) {
  const int g = blockIdx.x, tid = threadIdx.x;
  const InstMap im = map_instance(p, g);
  const bool use_state = !(p.flags & LESS_NO_STATE);
  const float* hp = p.a.ws_hpart + (size_t)g * kMaxSplit * (R * D + R);
  const int ns = use_state ? p.nsplit : 0;
#pragma unroll
  for (int r = 0; r < R; ++r) {
    float s = 0.f;
    for (int sp = 0; sp < ns; ++sp) s += hp[(size_t)sp * (R * D + R) + r * D + tid];
    p.a.H[(im.inst * R + r) * D + tid] = s;
  }
  if (tid < R) {
    float s = 0.f;
    for (int sp = 0; sp < ns; ++sp) s += hp[(size_t)sp * (R * D + R) + R * D + tid];
    p.a.z[im.inst * R + tid] = s;
  }
}

// ---- P6 on CUDA cores (general shapes): the split's share of Eq. 4 / Eq. 5 over D_1 ---------- //
// One CTA per (token split, instance), thread d = one column of H: H[r][d] += psi_j[r] v_j[d] over
// the split's discarded tokens in ascending position (fixed order), z[r] likewise.
template <int R, int D>
__global__ void __launch_bounds__(D) state_kernel(PfParams p) {
  const int split = blockIdx.x, g = blockIdx.y, tid = threadIdx.x;
  const InstMap im = map_instance(p, g);
  const int jbeg = split * p.split_tokens, jend = min(p.S, jbeg + p.split_tokens);
  const float* psi = p.a.ws_psi + (size_t)g * p.Sp * R;
  const int32_t* slot_of = p.a.ws_slot + (size_t)g * p.Sp;
  float h[R], z = 0.f;
#pragma unroll
  for (int r = 0; r < R; ++r) h[r] = 0.f;
  for (int j = jbeg; j < jend; ++j) {
    if (slot_of[j] >= 0) continue;                    // kept: stays in the cache
    const float v = __half2float(p.V[(im.in_row0 + j) * D + tid]);
#pragma unroll
    for (int r = 0; r < R; ++r) h[r] = fmaf(__ldg(psi + (size_t)j * R + r), v, h[r]);
    if (tid < R) z += __ldg(psi + (size_t)j * R + tid);
  }
  float* hp = p.a.ws_hpart + ((size_t)g * kMaxSplit + split) * (R * D + R);
#pragma unroll
  for (int r = 0; r < R; ++r) hp[r * D + tid] = h[r];
  if (tid < R) hp[R * D + tid] = z;
}

// The CUDA-core prompt phase for one head dimension: every step of launch_prefill_group below that
// has no tensor-core kernel for the shape at hand.
template <int R, int D>
static void launch_cuda_core_tail(less_ctx* c, const PfParams& p, int G, int S, bool with_psi, bool with_state,
                                  cudaStream_t s) {
  const Dims& d = c->d;
  if (with_psi) {
    const size_t smem = (size_t)(FM_BR * D + mlp_smem_floats(d.Rp)) * 4;
    LaunchScope scope(c, LESS_KERNEL_PSI, s, "psi_kernel");
    cudaFuncSetAttribute(psi_kernel<R, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    psi_kernel<R, D><<<dim3(p.nsplit, G), FM_THREADS, smem, s>>>(p);
  }
  if (S > 0) {
    LaunchScope scope(c, LESS_KERNEL_GATHER, s, "gather_kernel");
    const int gx = (min(S, d.N) + 63) / 64 > 0 ? (min(S, d.N) + 63) / 64 : 1;
    gather_kernel<R, D><<<dim3(gx, G), GA_THREADS, 0, s>>>(p);
  }
  if (with_state) {
    LaunchScope scope(c, LESS_KERNEL_BUILD, s, "state_kernel");
    state_kernel<R, D><<<dim3(p.nsplit, G), D, 0, s>>>(p);
  }
}

template <int D>
static void launch_cuda_core_scoring(less_ctx* c, const PfParams& p, int G, int S, bool h2o, bool with_out, cudaStream_t s) {
  const int tiles = (S + PF_TILE - 1) / PF_TILE;
  {
    LaunchScope scope(c, LESS_KERNEL_ROWSTAT, s, "rowstat_kernel");
    rowstat_kernel<D><<<dim3(tiles, G * p.grp), PF_TILE, 0, s>>>(p);
  }
  if (h2o) {
    LaunchScope scope(c, LESS_KERNEL_COLSUM, s, "colsum_kernel");
    colsum_kernel<D><<<dim3(tiles, G), PF_TILE, 0, s>>>(p);
  }
  if (with_out) {
    LaunchScope scope(c, LESS_KERNEL_ATTN_OUT, s, "attn_out_kernel");
    attn_out_kernel<D><<<dim3((S + AO_ROWS - 1) / AO_ROWS, G * p.grp), PF_TILE, 0, s>>>(p);
  }
}

int launch_prefill_group(less_ctx* c, int layer0, int nl, int lj0, int layer_count, int S,
                         const void* Q, const void* K, const void* V, void* attn_out,
                         cudaStream_t s) {
  const Dims& d = c->d;
  PfParams p;
  p.Q = (const __half*)Q; p.K = (const __half*)K; p.V = (const __half*)V;
  p.attn_out = (float*)attn_out;
  p.a = c->a;
  p.w_psi1 = (const __half*)c->w.w_psi1;
  p.w_psi2 = (const __half*)c->w.w_psi2;
  p.w_psi3 = (const __half*)c->w.w_psi3;
  p.psi_scale = c->w.psi_scale;
  p.S = S; p.Sp = d.Sp; p.Sbx = d.Sbx;
  p.layer0 = layer0; p.nl = nl; p.lj0 = lj0; p.layer_count = layer_count;
  p.B = d.B; p.L = d.L; p.Hd = d.Hd; p.N = d.N; p.Np = d.Np;
  p.heavy = d.heavy; p.recent = d.recent; p.Rp = d.Rp;
  p.flags = d.flags;
  p.grp = d.G;
  // Token splits of the state build: whole 128-token tiles, as long as they can be (the head's W1,
  // 128 KB, and the CTA's set-up are paid per split) while the grid still is several waves deep,
  // so that the last wave's imbalance stays small.
  const int G = d.B * nl * d.Hd;
  int nsplit = 0, split_tokens = 8192;
  if (S > 0) {
    while (split_tokens > 128 && (long long)G * ((S + split_tokens - 1) / split_tokens) < 8 * c->sms) split_tokens >>= 1;
    if ((S + split_tokens - 1) / split_tokens > kMaxSplit)
      split_tokens = ((S + kMaxSplit - 1) / kMaxSplit + 127) / 128 * 128;
    nsplit = (S + split_tokens - 1) / split_tokens;
  }
  p.nsplit = nsplit; p.split_tokens = split_tokens;
  // Lambda-masking needs no scores and TOVA only the last query's row; the row statistics are still
  // needed for the prompt's attention output
  const bool h2o = !(d.flags & (LESS_POLICY_LAMBDA | LESS_POLICY_TOVA));
  const bool need_scores = h2o || attn_out != nullptr;
  // tensor-core kernels: head dimension 128 and 1, 2, 4 or 8 query heads per KV head; everything else
  // (and LESS_SCORE_KERNEL=plain) runs the CUDA-core kernels, which take any of the shapes
  const bool tc_scoring = !d.general && c->score_path == 1 && score_tc_supported();
  if (S > 0 && need_scores) {
    if (tc_scoring) {
      int rc = launch_score_tc(c, p, G, s, h2o);   // column sums only where H2O ranks by them
      if (rc == LESS_OK && attn_out) rc = launch_attn_out_tc(c, p, G, s);
      if (rc != LESS_OK) return rc;
    } else if (d.D == 64) {
      launch_cuda_core_scoring<64>(c, p, G, S, h2o, attn_out != nullptr, s);
    } else {
      launch_cuda_core_scoring<kHeadDim>(c, p, G, S, h2o, attn_out != nullptr, s);
    }
  }
  if (S > 0 && (d.flags & LESS_POLICY_TOVA)) {
    LaunchScope scope(c, LESS_KERNEL_COLSUM, s, "lastrow_kernel");
    if (d.D == 64) lastrow_kernel<64><<<G, LR_THREADS, 0, s>>>(p);
    else lastrow_kernel<kHeadDim><<<G, LR_THREADS, 0, s>>>(p);
  }
  {
    LaunchScope scope(c, LESS_KERNEL_SELECT, s, "select_kernel");
    select_kernel<<<G, SEL_THREADS, 0, s>>>(p);
  }
  const bool use_state = !(d.flags & LESS_NO_STATE);
  const bool with_state = nsplit > 0 && use_state;
  const bool fused = with_state && !d.general && psi_tc_supported(d);   // psi and the state build in one kernel
  if (fused) {
    const int rc = launch_psi_state_tc(c, p, G, s);
    if (rc != LESS_OK) return rc;
  }
  // psi on CUDA cores where the fused kernel does not apply; the kept rows to their slots; the state
  // build of the general shapes
  const bool cc_state = with_state && d.general;
  if (d.D == 64) {
    if (d.R == 8) launch_cuda_core_tail<8, 64>(c, p, G, S, with_state && !fused, cc_state, s);
    else launch_cuda_core_tail<16, 64>(c, p, G, S, with_state && !fused, cc_state, s);
  } else {
    if (d.R == 8) launch_cuda_core_tail<8, kHeadDim>(c, p, G, S, with_state && !fused, cc_state, s);
    else launch_cuda_core_tail<16, kHeadDim>(c, p, G, S, with_state && !fused, cc_state, s);
  }
  if (with_state && !fused && !cc_state) {
    const int rc = launch_state_tc(c, p, G, s);
    if (rc != LESS_OK) return rc;
  }
  {
    LaunchScope scope(c, LESS_KERNEL_FINALIZE, s, "finalize_kernel");
    if (d.D == 64) {
      if (d.R == 8) finalize_kernel<8, 64><<<G, 64, 0, s>>>(p);
      else finalize_kernel<16, 64><<<G, 64, 0, s>>>(p);
    } else {
      if (d.R == 8) finalize_kernel<8, kHeadDim><<<G, kHeadDim, 0, s>>>(p);
      else finalize_kernel<16, kHeadDim><<<G, kHeadDim, 0, s>>>(p);
    }
  }
  return check_launch("the prompt-phase kernels");
}

}  // namespace less
