// Decode-step kernels (Algorithm 1):
//   feature_map_kernel  phi(q_t), psi(k_t)                         (Eq. 1, Eq. 2)
//   decode_kernel       scores over the live slots, Eq. 3, H2O score update,
//                       argmin eviction, Eq. 4 / Eq. 5, in-place slot overwrite
//   decode_group_*      the same step for G query heads per KV head
//   small_step_kernel   both in one launch for workloads of a few heads: a cluster of CTAs per head
//                       splits the two MLPs, then one CTA per batch row runs the decode step
#include <stdio.h>

#include "feature_gemv.cuh"
#include "feature_mlp.cuh"
#include "tc_common.cuh"

namespace less {

// --------------------------------------------------------------------------- //
// Feature maps, plain version (hidden widths the streaming kernel does not take).
// One CTA = one (layer, head), one map (phi or psi), up to FM_BR batch rows.
// The hidden activations never leave shared memory.
// --------------------------------------------------------------------------- //
template <int R>
__global__ void __launch_bounds__(FM_THREADS) feature_map_kernel(FmParams p, int which0) {
  extern __shared__ float fm_smem[];
  const int D = p.D;
  float* xs = fm_smem;                         // [FM_BR][D]
  float* hs = xs + FM_BR * D;                  // [FM_BR][Rp]
  float* part = hs + FM_BR * p.Rp;             // [ndg][FM_BR][Rp]
  pdl_launch_dependents();
  const int which = which0 + blockIdx.y;       // 0 phi(q), 1 psi(k)
  const int Hh = p.Hh[which];                  // heads of this map per layer
  const int lh = blockIdx.x;                   // layer * Hh + head
  const int b0 = blockIdx.z * FM_BR;
  const int nb = min(FM_BR, p.B - b0);
  const int tid = threadIdx.x;
  const int layer = lh / Hh, head = lh % Hh;
  for (int e = tid; e < FM_BR * D; e += FM_THREADS) {
    const int b = e / D, d = e % D;
    float v = 0.f;
    if (b < nb)
      v = __half2float(p.x[which][(((size_t)(b0 + b) * p.L + layer) * Hh + head) * D + d]);
    xs[e] = v;
  }
  __syncthreads();
  float c1 = 1.f, c2 = 1.f;
  if (which == 1 && p.psi_scale) {
    c1 = p.psi_scale[lh * 2];
    c2 = p.psi_scale[lh * 2 + 1];
  }
  const float r = mlp_rows<R>(xs, part, hs, nb, p.w1[which] + (size_t)lh * D * p.Rp,
                              p.w2[which] + (size_t)lh * p.Rp * R, p.w3 + (size_t)lh * R * R, c1,
                              c2, p.Rp, which == 1, D);
  const int warp = tid >> 5, lane = tid & 31;
  if (warp < nb && lane < R) {
    const size_t inst = ((size_t)(b0 + warp) * p.L + layer) * Hh + head;
    p.out[which][inst * R + lane] = r;
  }
}

template <int R>
static int launch_plain_feature_maps(less_ctx* c, const FmParams& p, dim3 grid, int which0, size_t smem, cudaStream_t s) {
  LaunchScope scope(c, LESS_KERNEL_FEATURE_MAP, s, R == 8 ? "feature_map_kernel<8>" : "feature_map_kernel<16>");
  if (cudaFuncSetAttribute(feature_map_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return fail_cuda("shared memory opt-in of feature_map_kernel");
  feature_map_kernel<R><<<grid, FM_THREADS, smem, s>>>(p, which0);
  return check_launch("feature_map_kernel");
}

int launch_feature_maps(less_ctx* c, const void* q, const void* k, cudaStream_t s) {
  const Dims& d = c->d;
  FmParams p;
  p.x[0] = (const __half*)q;
  p.x[1] = (const __half*)k;
  p.w1[0] = (const __half*)c->w.w_phi1;
  p.w1[1] = (const __half*)c->w.w_psi1;
  p.w2[0] = (const __half*)c->w.w_phi2;
  p.w2[1] = (const __half*)c->w.w_psi2;
  p.w3 = (const __half*)c->w.w_psi3;
  p.psi_scale = c->w.psi_scale;
  p.out[0] = c->a.phi_q;
  p.out[1] = c->a.psi_k;
  p.B = d.B; p.L = d.L; p.Hd = d.Hd; p.Rp = d.Rp; p.D = d.D;
  p.Hh[0] = d.Hd * d.G; p.Hh[1] = d.Hd;
  p.feat_flag = nullptr; p.flag_stride = d.L * d.Hd * d.G;
  p.x_plain = c->x_plain ? 1 : 0;
  p.lh0 = c->seg_l0 * d.Hd; p.nlh = c->seg_nl * d.Hd;
  c->flags_this_step = false;
  const int ndg = FM_THREADS / (d.Rp / 8);
  const size_t smem = (size_t)(FM_BR * d.D + FM_BR * d.Rp + ndg * FM_BR * d.Rp) * 4;
  if (d.flags & LESS_NO_STATE) return LESS_OK;   // neither phi nor psi is used
  const int nbz = (d.B + FM_BR - 1) / FM_BR;
  if (!d.general) {
    if ((c->feature_path == 2 || d.G > 1) && feature_tc_supported(d)) return launch_feature_tc(c, p, s);
    if (c->seg_nl != d.L) return LESS_ERR_INVALID_CONFIG;   // only the tensor-core kernels take a layer range
    if (d.G > 1) return LESS_ERR_INVALID_CONFIG;    // the streaming kernels below know one query head per KV head
    if (c->feature_path >= 1 && feature_gemv_supported(d)) return launch_feature_gemv(c, p, s);
    const dim3 grid(d.L * d.Hd, 2, nbz);
    return d.R == 8 ? launch_plain_feature_maps<8>(c, p, grid, 0, smem, s) : launch_plain_feature_maps<16>(c, p, grid, 0, smem, s);
  }
  // general shapes: phi over the query heads, then psi over the KV heads
  for (int which = 0; which < 2; ++which) {
    const dim3 grid(d.L * p.Hh[which], 1, nbz);
    const int rc = d.R == 8 ? launch_plain_feature_maps<8>(c, p, grid, which, smem, s)
                            : launch_plain_feature_maps<16>(c, p, grid, which, smem, s);
    if (rc != LESS_OK) return rc;
  }
  return LESS_OK;
}

// --------------------------------------------------------------------------- //
// Fused decode step: one CTA per instance.
// --------------------------------------------------------------------------- //
constexpr int DEC_THREADS = 128;
constexpr int DEC_RG = DEC_THREADS / 16;   // row groups: 16 lanes x 16 B cover one 256-B row

struct DecParams {
  const __half* q; const __half* k; const __half* v;   // [I, D]
  void* out;                                            // [I * G, D] fp32, or fp16 with LESS_OUT_F16
  int32_t* evicted_pos;                                 // [I] or null
  Arena a;
  int N, Np, heavy, recent;
  int t;             // position of this step's token (direct calls)
  uint32_t flags;
  int B, LH;         // batch, layers x KV heads
  const uint32_t* feat_flag;   // per-head counters of the feature-map kernel, or null: wait for its whole grid
  int flag_stride;             // psi counters start here (= layers x query heads)
  uint32_t flag_target[2];     // counter values that mean "this step's phi / psi of the head are written"
  int head_major;              // CTAs numbered (layer-head, batch row) instead of by instance
  int lh0;                     // first (layer, KV head) of this launch (head-major numbering only)
  int done_ctas;               // CTAs of this launch that run a decode step (captured steps count themselves out)
};

__device__ __forceinline__ float block_max(float v, float* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float r = red[0];
#pragma unroll
  for (int w = 1; w < DEC_THREADS / 32; ++w) r = fmaxf(r, red[w]);
  __syncthreads();
  return r;
}

__device__ __forceinline__ float block_sum(float v, float* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float r = red[0];
#pragma unroll
  for (int w = 1; w < DEC_THREADS / 32; ++w) r += red[w];   // fixed order
  __syncthreads();
  return r;
}

// The position of the step's token.  A direct call passes it as a kernel argument and CTA 0
// leaves position + 1 in device memory.  A step that is being captured in a CUDA graph cannot bake
// the position in: it reads it from device memory, and the CTAs count themselves out so that the
// last one advances it for the next replay (one contended atomic per CTA: the price of replaying
// without the host, paid only by captured steps).
template <bool kCaptured>
__device__ __forceinline__ void step_done(const DecParams& p) {
  int32_t* tpos = p.a.tpos;
  if (threadIdx.x != 0) return;
  if (!kCaptured) {
    if (blockIdx.x == 0) tpos[0] = p.t + 1;
  } else if (atomicAdd(tpos + 1, 1) == p.done_ctas - 1) {      // every thread read the position barriers ago
    tpos[1] = 0;
    atomicAdd(tpos, 1);
  }
}

// Where the feature maps of this step come from.  The feature-map kernel of the same step may still
// be running (programmatic dependent launch): either the whole grid is awaited (griddepcontrol.wait),
// or, when the feature kernel publishes a counter per (layer, head) and map, only this instance's
// own phi(q_t) and psi(k_t) are: thread g < G polls the counter of query head g, thread G that of
// psi, each with a bounded number of polls; a wait that runs out is recorded in the status word
// and the step goes on (its result is then flagged, never hung).
constexpr uint32_t kFlagPolls = 1u << 22;          // x 64 ns of back-off: a quarter of a second at most
template <int G>
__device__ __forceinline__ void wait_feature_maps(const DecParams& p, int lh) {
  if (p.feat_flag == nullptr) {
    pdl_wait_primary();
    return;
  }
  const int tid = threadIdx.x;
  if (tid <= G) {
    const uint32_t* f = tid < G ? p.feat_flag + (size_t)lh * G + tid : p.feat_flag + p.flag_stride + lh;
    const uint32_t want = tid < G ? p.flag_target[0] : p.flag_target[1];
    uint32_t i = 0;
    for (;;) {
      uint32_t v;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(f) : "memory");
      if ((int32_t)(v - want) >= 0) break;
      if (++i >= kFlagPolls) {
        set_status(p.a.status, kStatusTimeout, 3);
        break;
      }
      // once any wait of this context has given up, the others do not sit theirs out
      if ((i & 255u) == 0 && *reinterpret_cast<volatile int32_t*>(p.a.status) != 0) break;
      __nanosleep(64);
    }
  }
  __syncthreads();
}

__device__ __forceinline__ void store_out(const DecParams& p, size_t idx, float x) {
  if (p.flags & LESS_OUT_F16) reinterpret_cast<__half*>(p.out)[idx] = __float2half_rn(x);
  else reinterpret_cast<float*>(p.out)[idx] = x;
}

// The instance a CTA works on.  Behind a feature kernel that publishes per-head counters the CTAs
// are numbered head-major (all batch rows of a head are neighbours), so that the first CTAs need
// the first heads' feature maps; otherwise CTA = instance.
__device__ __forceinline__ size_t decode_instance(const DecParams& p) {
  if (!p.head_major) return blockIdx.x;
  const int lhi = blockIdx.x / p.B, b = blockIdx.x - lhi * p.B;
  return (size_t)b * p.LH + p.lh0 + lhi;
}

// The second half of a step, common to all decode kernels (one 128-thread CTA per KV head, thread
// d owns column d of H): H2O score update with the probabilities of the G query heads, the choice
// of the entry that leaves (policy), Eq. 4 / Eq. 5 for it, and the new pair's in-place write.
//   s_sc  [G][Ns]  e^{s - m_g} of every live entry and, at index n, of the new pair
//   inv   [G]      1 / normaliser of each head
//   hcol  [R]      column d of H as read for Eq. 3
//   D     head dimension: a slot row is D / 8 chunks of 16 bytes; threads d < D own a column of H
//   stg   copies of the instance's V rows, scores, positions and cached psi the caller holds in shared
//         memory (the one-launch step of small workloads), or all null: read them from the arena
struct TailStage {
  const __half* V = nullptr;        // [N][D]
  const float* acc = nullptr;       // [Np]
  const int32_t* pos = nullptr;     // [Np]
  const float* psic = nullptr;      // [N][R]
};
template <int R, int G, bool kCaptured, int D = kHeadDim>
__device__ __forceinline__ void decode_tail(const DecParams& p, size_t inst, int n, int t_now, const float* s_sc, int Ns,
                                            const float (&inv)[G], const float (&hcol)[R], const uint4& knew,
                                            const uint4& vnew, unsigned long long* s_key, int* s_vic,
                                            const TailStage stg = TailStage()) {
  constexpr int LPR = D / 8;                           // lanes per slot row
  const int tid = threadIdx.x, d = tid, l16 = tid % LPR, rg = tid / LPR;
  const bool own = D == DEC_THREADS || d < D;
  const int N = p.N;
  const bool use_state = !(p.flags & LESS_NO_STATE);
  float* Hb = p.a.H + inst * (size_t)R * D;
  float* zb = p.a.z + inst * R;
  const __half* Vb = stg.V ? stg.V : p.a.vslots + inst * (size_t)N * D;
  int32_t* posb = p.a.pos + inst * (size_t)p.Np;
  float* accb = p.a.acc + inst * (size_t)p.Np;
  const int32_t* pos_r = stg.V ? stg.pos : posb;        // where the step reads them (never both copies of a slot
  const float* acc_r = stg.V ? stg.acc : accb;         // after its write below: reads come first)
  const bool full = (n == N);
  const bool lambda_policy = (p.flags & LESS_POLICY_LAMBDA) != 0;
  const bool tova_policy = G == 1 && (p.flags & LESS_POLICY_TOVA) != 0;
  unsigned long long best = ~0ull;
  for (int i = tid; i < n; i += DEC_THREADS) {
    float ps_sum = 0.f;
#pragma unroll
    for (int g = 0; g < G; ++g) ps_sum = G == 1 ? s_sc[i] * inv[0] : fmaf(s_sc[g * Ns + i], inv[g], ps_sum);
    // TOVA scores an entry by this query's probability alone; H2O accumulates
    const float a = tova_policy ? ps_sum : acc_r[i] + ps_sum;
    accb[i] = a;
    if (full) {
      const int ps = pos_r[i];
      if (tova_policy) {                               // TOVA: every entry competes, nothing is protected
        const unsigned long long key = ((unsigned long long)__float_as_uint(a) << 32) | (unsigned int)ps;
        best = key < best ? key : best;
      } else if (lambda_policy) {                      // Lambda-masking: the oldest position past the first tokens
        if (ps >= p.heavy) best = (unsigned long long)(unsigned int)ps < best ? (unsigned int)ps : best;
      } else if (ps <= t_now - p.recent) {             // H2O: lowest (accumulated score, position) outside the window
        const unsigned long long key = ((unsigned long long)__float_as_uint(a) << 32) | (unsigned int)ps;
        best = key < best ? key : best;
      }
    }
  }
  float p_new = 0.f;
#pragma unroll
  for (int g = 0; g < G; ++g) p_new = G == 1 ? s_sc[n] * inv[0] : fmaf(s_sc[g * Ns + n], inv[g], p_new);
  int slot = n;                                        // next free slot
  if (full) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
      best = other < best ? other : best;
    }
    if ((tid & 31) == 0) s_key[tid >> 5] = best;
    if (tid == 0) *s_vic = -1;
    __syncthreads();
    best = s_key[0];
#pragma unroll
    for (int w = 1; w < DEC_THREADS / 32; ++w) best = s_key[w] < best ? s_key[w] : best;
    if (tova_policy) {
      // the new pair competes too; if its own probability is the lowest it never enters the
      // cache: it is absorbed into H, z at once and every slot stays as it is
      const unsigned long long key_new = ((unsigned long long)__float_as_uint(p_new) << 32) | (unsigned int)t_now;
      if (key_new < best) {                            // uniform over the CTA
        if (tid == 0 && p.evicted_pos) p.evicted_pos[inst] = t_now;
        if (use_state) {
          const float* psn = p.a.psi_k + inst * R;
          if (own) {
            const float vv = __half2float(p.v[inst * D + d]);
#pragma unroll
            for (int r = 0; r < R; ++r) Hb[r * D + d] = fmaf(__ldcg(psn + r), vv, hcol[r]);
          }
          if (tid < R) zb[tid] += __ldcg(psn + tid);
        }
        step_done<kCaptured>(p);
        return;
      }
    }
    const int vpos = (int)(unsigned int)(best & 0xffffffffull);
    for (int i = tid; i < n; i += DEC_THREADS)
      if (pos_r[i] == vpos && best != ~0ull) *s_vic = i;   // positions are unique
    __syncthreads();
    slot = *s_vic;
    if (slot < 0) {                                    // cannot happen with recent >= 1; refuse
      if (tid == 0) {
        set_status(p.a.status, kStatusBounds, 2);
        if (p.evicted_pos) p.evicted_pos[inst] = -1;
      }
      step_done<kCaptured>(p);
      return;
    }
    if (tid == 0 && p.evicted_pos) p.evicted_pos[inst] = vpos;
    // ---- Eq. 4 / Eq. 5: absorb the victim (psi acts on the key: the state is the KV head's) ----
    if (use_state) {
      const float* psv = stg.V ? stg.psic + (size_t)slot * R : p.a.psic + (inst * (size_t)N + slot) * R;
      if (own) {
        const float vv = __half2float(Vb[(size_t)slot * D + d]);
#pragma unroll
        for (int r = 0; r < R; ++r) Hb[r * D + d] = fmaf(psv[r], vv, hcol[r]);
      }
      if (tid < R) zb[tid] += psv[tid];
    }
    __syncthreads();                                   // victim row fully read before overwrite
  } else {
    if (tid == 0) {
      p.a.count[inst] = n + 1;
      if (p.evicted_pos) p.evicted_pos[inst] = -1;
    }
  }
  // ---- the new pair takes the slot in place ----
  __half* Kw = p.a.kslots + (inst * (size_t)N + slot) * D;
  __half* Vw = p.a.vslots + (inst * (size_t)N + slot) * D;
  if (rg == 0) *reinterpret_cast<uint4*>(Kw + l16 * 8) = knew;
  if (rg == 1) *reinterpret_cast<uint4*>(Vw + l16 * 8) = vnew;
  if (tid == 32) { posb[slot] = t_now; accb[slot] = p_new; }
  if (tid >= 64 && tid < 64 + R)
    p.a.psic[(inst * (size_t)N + slot) * R + (tid - 64)] = use_state ? __ldcg(p.a.psi_k + inst * R + (tid - 64)) : 0.f;
  step_done<kCaptured>(p);
}

// Eq. 3 of each of the G query heads over the KV head's shared H, z, from the heads' partial
// numerators in shared memory (s_red [G][NRED][128]), then the common second half of the step.
template <int R, int G, bool kCaptured, int NRED>
__device__ __forceinline__ void group_eq3_and_tail(const DecParams& p, size_t inst, int n, int t_now, const float* s_sc,
                                                   int Ns, const float* s_red, const float* s_m, const float* s_l,
                                                   const uint4& knew, const uint4& vnew, float* s_inv,
                                                   unsigned long long* s_key, int* s_vic) {
  const int tid = threadIdx.x, d = tid;
  const bool use_state = !(p.flags & LESS_NO_STATE);
  const float* Hb = p.a.H + inst * (size_t)R * kHeadDim;
  const float* zb = p.a.z + inst * R;
  float hcol[R], zr[R];
  if (use_state) {
    wait_feature_maps<G>(p, (int)(inst % p.LH));
#pragma unroll
    for (int r = 0; r < R; ++r) {
      hcol[r] = Hb[r * kHeadDim + d];
      zr[r] = zb[r];
    }
  }
#pragma unroll
  for (int g = 0; g < G; ++g) {
    float num = 0.f;
#pragma unroll
    for (int j = 0; j < NRED; ++j) num += s_red[(g * NRED + j) * kHeadDim + d];
    const float lg = s_l[g];                         // the heads' maxima and sums stay in shared memory: registers
    float den = lg;                                  // decide how many of these CTAs an SM holds
    if (use_state) {
      const float em = __expf(-s_m[g]);
      const float* ph = p.a.phi_q + (inst * G + g) * R;
      float lr = 0.f, lz = 0.f;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float f = __ldcg(ph + r);
        lr = fmaf(f, hcol[r], lr);
        lz = fmaf(f, zr[r], lz);
      }
      num = fmaf(em, lr, num);
      den = fmaf(em, lz, den);
    }
    store_out(p, (inst * G + g) * kHeadDim + d, num / den);
    if (tid == 0) s_inv[g] = 1.0f / ((p.flags & LESS_SCORE_NORM_SPARSE) ? lg : den);
  }
  __syncthreads();
  float inv[G];
#pragma unroll
  for (int g = 0; g < G; ++g) inv[g] = s_inv[g];
  decode_tail<R, G, kCaptured>(p, inst, n, t_now, s_sc, Ns, inv, hcol, knew, vnew, s_key, s_vic);
}

template <int R, bool kCaptured>
__global__ void __launch_bounds__(DEC_THREADS) decode_kernel(DecParams p) {
  extern __shared__ float dsm[];
  pdl_launch_dependents();                         // the next step's feature-map kernel may come up while this one runs
  float* s_sc = dsm;                               // [Np + 4] scores, then e^{s - m}
  float* s_red = s_sc + p.Np + 4;                  // [DEC_RG][128] partial numerators
  __shared__ float s_small[DEC_THREADS / 32];
  __shared__ unsigned long long s_key[DEC_THREADS / 32];
  __shared__ int s_vic;

  const int tid = threadIdx.x;
  const size_t inst = decode_instance(p);
  const int l16 = tid & 15, rg = tid >> 4;
  const int N = p.N;
  const int t_now = kCaptured ? __ldcg(p.a.tpos) : p.t;   // tokens seen = this token's position
  int n = p.a.count[inst];
  if (n < 0 || n > N) {                            // refuse a corrupt count, touch nothing
    if (tid == 0) set_status(p.a.status, kStatusBounds, 1);
    step_done<kCaptured>(p);
    return;
  }
  const bool use_state = !(p.flags & LESS_NO_STATE);
  const float scale = 0.08838834764831845f;        // 1 / sqrt(128)

  const __half* Kb = p.a.kslots + inst * (size_t)N * kHeadDim;
  const __half* Vb = p.a.vslots + inst * (size_t)N * kHeadDim;

  float qf[8];
  half8_to_float(*reinterpret_cast<const uint4*>(p.q + inst * kHeadDim + l16 * 8), qf);

  // ---- scores s_i = q . k_i / sqrt(D) over live slots, and the new pair ----
#pragma unroll 8
  for (int r0 = 0; r0 < n; r0 += DEC_RG) {         // r0 is block-uniform: shuffles stay converged
    const int r = r0 + rg;
    float dot = 0.f;
    if (r < n) {
      float kf[8];
      half8_to_float(ldg_stream(Kb + (size_t)r * kHeadDim + l16 * 8), kf);
#pragma unroll
      for (int c = 0; c < 8; ++c) dot = fmaf(qf[c], kf[c], dot);
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    if (l16 == 0 && r < n) s_sc[r] = dot * scale;
  }
  const uint4 knew = *reinterpret_cast<const uint4*>(p.k + inst * kHeadDim + l16 * 8);
  const uint4 vnew = *reinterpret_cast<const uint4*>(p.v + inst * kHeadDim + l16 * 8);
  if (tid < 32) {                                  // whole warp 0 (both halves compute the same)
    float kf[8];
    half8_to_float(knew, kf);
    float dot = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) dot = fmaf(qf[c], kf[c], dot);
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    if (tid == 0) s_sc[n] = dot * scale;
  }
  __syncthreads();

  // ---- m = max, e_i = exp(s_i - m), l = sum e_i  (entries 0..n, n = new pair) ----
  float m = -INFINITY;
  for (int i = tid; i <= n; i += DEC_THREADS) m = fmaxf(m, s_sc[i]);
  m = block_max(m, s_small);
  m = fmaxf(m, -80.f);                             // keeps e^{-m} finite for the low-rank terms
  float lsum = 0.f;
  for (int i = tid; i <= n; i += DEC_THREADS) {
    const float e = __expf(s_sc[i] - m);
    s_sc[i] = e;
    lsum += e;
  }
  lsum = block_sum(lsum, s_small);                 // also orders the s_sc writes

  // ---- u = sum e_i v_i ----
  float u[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) u[c] = 0.f;
#pragma unroll 8
  for (int r = rg; r < n; r += DEC_RG) {
    float vf[8];
    half8_to_float(ldg_stream(Vb + (size_t)r * kHeadDim + l16 * 8), vf);
    const float e = s_sc[r];
#pragma unroll
    for (int c = 0; c < 8; ++c) u[c] = fmaf(e, vf[c], u[c]);
  }
  if (rg == 0) {
    float vf[8];
    half8_to_float(vnew, vf);
    const float e = s_sc[n];
#pragma unroll
    for (int c = 0; c < 8; ++c) u[c] = fmaf(e, vf[c], u[c]);
  }
#pragma unroll
  for (int c = 0; c < 8; ++c) s_red[rg * kHeadDim + l16 * 8 + c] = u[c];
  __syncthreads();

  // ---- low-rank correction and the single normalisation (Eq. 3) ----
  const int d = tid;                               // DEC_THREADS == D: one column per thread
  float num = 0.f;
#pragma unroll
  for (int g = 0; g < DEC_RG; ++g) num += s_red[g * kHeadDim + d];
  float den = lsum;
  const float* Hb = p.a.H + inst * (size_t)R * kHeadDim;
  const float* zb = p.a.z + inst * R;
  float hcol[R];
  if (use_state) {
    wait_feature_maps<1>(p, (int)(inst % p.LH));   // phi(q_t), psi(k_t) of this step are complete from here on
    const float em = __expf(-m);
    float lr = 0.f, lz = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const float f = __ldcg(p.a.phi_q + inst * R + r);
      hcol[r] = Hb[r * kHeadDim + d];
      lr = fmaf(f, hcol[r], lr);
      lz = fmaf(f, zb[r], lz);
    }
    num = fmaf(em, lr, num);
    den = fmaf(em, lz, den);
  }
  store_out(p, inst * kHeadDim + d, num / den);
  const float inv[1] = {1.0f / ((p.flags & LESS_SCORE_NORM_SPARSE) ? lsum : den)};
  decode_tail<R, 1, kCaptured>(p, inst, n, t_now, s_sc, p.Np + 4, inv, hcol, knew, vnew, s_key, &s_vic);
}

// --------------------------------------------------------------------------- //
// A whole step in one launch, for workloads of a few heads (Algorithm 1 from phi(q_t), psi(k_t) to
// the slot overwrite).  With so little to move, a step is bound by launches and by the chain
// "weights -> hidden layer -> layer 2 -> Eq. 3" rather than by bandwidth.  One cluster per
// (layer, head): one CTA per batch row runs the decode step of its instance, and SS_FEAT more CTAs
// each take 1 / SS_FEAT of the hidden units of both MLPs for all batch rows of the head (Eq. 1,
// Eq. 2: the sums over hidden units split exactly) while the decode CTAs are busy with the scores and
// the softmax.  The feature CTAs write their partial layer-2 sums of batch row b into the shared
// memory of the decode CTA of that row (plain st.shared::cluster over distributed shared memory) and
// arrive at the cluster barrier; behind it the decode CTA adds the SS_FEAT partials in rank order,
// finishes the maps (second GELU, W3 of psi, absolute value) and goes on with Eq. 3.  The barrier
// is the hardware's (barrier.cluster): every thread that has not left reaches it on every path.
// --------------------------------------------------------------------------- //
constexpr int SS_THREADS = 512;       // threads per CTA of the small-step kernel (a decode CTA runs its step on the first 128)
constexpr int SS_FEAT = 4;           // feature-map CTAs per head
constexpr int SS_MAXB = 4;           // batch rows (decode CTAs) per head: SS_FEAT + SS_MAXB = the portable cluster size
constexpr int SS_MAXJ = 128;         // hidden units per feature CTA at the widest hidden layer (512)
constexpr int SS_STAGE_SLOTS = 128;  // up to this many slots a decode CTA keeps its instance's rows in shared memory

struct SsMaps {
  const __half* w1[2];    // W_phi1, W_psi1 [L, Hd, D, Rp]
  const __half* w2[2];    // W_phi2, W_psi2 [L, Hd, Rp, R]
  const __half* w3;       // W_psi3         [L, Hd, R, R]
  const float* psi_scale; // [L, Hd, 2] or null
  int Rp;
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
// an arrival that publishes nothing
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// writes v at `local` (an address in this CTA's shared memory) in the shared memory of CTA `rank` of the cluster
__device__ __forceinline__ void cluster_peer_store_f32(float* local, uint32_t rank, float v) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(local);
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra), "f"(v) : "memory");
}

// D += A B for one 16 x 8 x 16 tile on the tensor cores (warp-level mma: fp16 operands, fp32 accumulation)
__device__ __forceinline__ void mma_m16n8k16(float* d, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// four 8 x 8 fp16 matrices from shared memory, transposed on the way (lane l gives the address of row l & 7 of matrix l >> 3)
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, const void* row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"((uint32_t)__cvta_generic_to_shared(row)));
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
               : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// max / sum over the SS_THREADS threads of a CTA (warp tree, then the warps in order: fixed)
__device__ __forceinline__ float wide_max(float v, float* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float r = red[0];
#pragma unroll
  for (int w = 1; w < SS_THREADS / 32; ++w) r = fmaxf(r, red[w]);
  return r;                                        // `red` is not reused: no second barrier
}
__device__ __forceinline__ float wide_sum(float v, float* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float r = red[0];
#pragma unroll
  for (int w = 1; w < SS_THREADS / 32; ++w) r += red[w];
  return r;
}

// What the decode CTA of the small-step kernel knows about its cluster.
struct SsDecoder {
  const float* part;      // [SS_FEAT][2][R] the feature CTAs' partial layer-2 sums of this batch row (written by them)
  float* own;             // this CTA's: gsum [2 R], phi [R], c1, c2, (pad), then W3 [R R] as halves
  const __half* K;        // the instance's K rows in shared memory, or null: not staged (too many slots)
  TailStage tail;         // ... and what the second half of the step reads
  uint64_t* bar;          // the bulk copies of all that (and of W3) complete here
  int* abort;
};

// The decode step of one instance in the small-step kernel.  The same arithmetic as decode_kernel, laid
// out for latency instead of bandwidth: with one small CTA per multiprocessor every phase is a chain of
// dependent latencies that only more warps can shorten, so the scores, the softmax and the weighted
// sum of the V rows run on all sixteen warps (32 slot rows per pass); the twelve extra warps then
// leave, and the first four meet the feature CTAs, finish phi(q_t), psi(k_t), and run Eq. 3 and the
// common second half of the step (decode_tail).
template <int R, bool kCaptured>
__device__ __forceinline__ void small_step_decode(const DecParams& p, const size_t inst, float* dsm, const SsDecoder cl) {
  constexpr int RG = SS_THREADS / 16;              // slot rows per pass
  float* s_sc = dsm;                               // [Np + 4] scores, then e^{s - m}
  float* s_red = s_sc + p.Np + 4;                  // [RG][128] partial numerators
  __shared__ float s_w[2][SS_THREADS / 32];        // one row per reduction
  __shared__ unsigned long long s_key[DEC_THREADS / 32];
  __shared__ int s_vic;

  const int tid = threadIdx.x;
  const int l16 = tid & 15, rg = tid >> 4;
  const int N = p.N;
  const int t_now = kCaptured ? __ldcg(p.a.tpos) : p.t;
  const int n = p.a.count[inst];
  if (n < 0 || n > N) {                            // refuse a corrupt count, touch nothing; the cluster is still met
    __syncthreads();                               // the barrier's initialisation is visible
    wait_or_give_up(cl.bar, 0, cl.abort, p.a.status, 130);   // leave with no copy into this CTA's shared memory in flight
    if (tid >= DEC_THREADS) return;
    cluster_wait();                                // the start-up phase, then the one the feature CTAs arrive at
    cluster_arrive();
    cluster_wait();
    if (tid == 0) set_status(p.a.status, kStatusBounds, 1);
    step_done<kCaptured>(p);
    return;
  }
  const float scale = 0.08838834764831845f;        // 1 / sqrt(128)
  const bool staged = cl.K != nullptr;
  const __half* Kb = staged ? cl.K : p.a.kslots + inst * (size_t)N * kHeadDim;
  const __half* Vb = staged ? cl.tail.V : p.a.vslots + inst * (size_t)N * kHeadDim;
  // the state is last step's: its loads are under way long before the maps arrive
  const int d = tid & (kHeadDim - 1);
  float hcol[R], zr[R];
  if (tid < DEC_THREADS) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
      hcol[r] = p.a.H[inst * (size_t)R * kHeadDim + r * kHeadDim + d];
      zr[r] = p.a.z[inst * R + r];
    }
  }

  float qf[8];
  half8_to_float(*reinterpret_cast<const uint4*>(p.q + inst * kHeadDim + l16 * 8), qf);
  const uint4 knew = *reinterpret_cast<const uint4*>(p.k + inst * kHeadDim + l16 * 8);
  const uint4 vnew = *reinterpret_cast<const uint4*>(p.v + inst * kHeadDim + l16 * 8);
  __syncthreads();                                 // the barrier's initialisation is visible
  wait_or_give_up(cl.bar, 0, cl.abort, p.a.status, 131);   // the bulk copies of the instance's rows (and W3) have landed
  // ---- scores s_i = q . k_i / sqrt(D) over live slots, and the new pair ----
#pragma unroll 2
  for (int r0 = 0; r0 < n; r0 += RG) {             // r0 is block-uniform: shuffles stay converged
    const int r = r0 + rg;
    float dot = 0.f;
    if (r < n) {
      float kf[8];
      half8_to_float(*reinterpret_cast<const uint4*>(Kb + (size_t)r * kHeadDim + l16 * 8), kf);
#pragma unroll
      for (int c = 0; c < 8; ++c) dot = fmaf(qf[c], kf[c], dot);
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    if (l16 == 0 && r < n) s_sc[r] = dot * scale;
  }
  if (tid < 32) {                                  // whole warp 0 (both halves compute the same)
    float kf[8];
    half8_to_float(knew, kf);
    float dot = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) dot = fmaf(qf[c], kf[c], dot);
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    if (tid == 0) s_sc[n] = dot * scale;
  }
  __syncthreads();

  // ---- m = max, e_i = exp(s_i - m), l = sum e_i  (entries 0..n, n = new pair) ----
  float m = -INFINITY;
  for (int i = tid; i <= n; i += SS_THREADS) m = fmaxf(m, s_sc[i]);
  m = wide_max(m, s_w[0]);
  m = fmaxf(m, -80.f);                             // keeps e^{-m} finite for the low-rank terms
  float lsum = 0.f;
  for (int i = tid; i <= n; i += SS_THREADS) {
    const float e = __expf(s_sc[i] - m);
    s_sc[i] = e;
    lsum += e;
  }
  lsum = wide_sum(lsum, s_w[1]);                   // also orders the s_sc writes

  // ---- u = sum e_i v_i ----
  float u[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) u[c] = 0.f;
#pragma unroll 2
  for (int r = rg; r < n; r += RG) {
    float vf[8];
    half8_to_float(*reinterpret_cast<const uint4*>(Vb + (size_t)r * kHeadDim + l16 * 8), vf);
    const float e = s_sc[r];
#pragma unroll
    for (int c = 0; c < 8; ++c) u[c] = fmaf(e, vf[c], u[c]);
  }
  if (rg == 0) {
    float vf[8];
    half8_to_float(vnew, vf);
    const float e = s_sc[n];
#pragma unroll
    for (int c = 0; c < 8; ++c) u[c] = fmaf(e, vf[c], u[c]);
  }
#pragma unroll
  for (int c = 0; c < 8; c += 4)
    *reinterpret_cast<float4*>(s_red + rg * kHeadDim + l16 * 8 + c) = make_float4(u[c], u[c + 1], u[c + 2], u[c + 3]);
  __syncthreads();
  if (tid >= DEC_THREADS) return;                  // the rest of the step runs on four warps; barriers count those left

  float num = 0.f;
#pragma unroll 8
  for (int g = 0; g < RG; ++g) num += s_red[g * kHeadDim + d];   // fixed order

  // ---- phi(q_t), psi(k_t): the feature CTAs' partial layer-2 sums, in rank order (Eq. 1, Eq. 2) ----
  float* gsum = cl.own;
  float* phis = cl.own + 2 * R;
  cluster_wait();                                  // the start-up phase (complete long ago)
  cluster_arrive();                                // behind this barrier the feature CTAs' partial sums are here
  cluster_wait();
  if (tid < 2 * R) {
    const int mm = tid / R, r = tid % R;
    float g = 0.f;
#pragma unroll
    for (int c = 0; c < SS_FEAT; ++c) g += cl.part[(c * 2 + mm) * R + r];   // rank order
    const float c1 = mm ? cl.own[3 * R] : 1.f, c2 = mm ? cl.own[3 * R + 1] : 1.f;
    g = c2 * gelu_erf(c1 * g);
    gsum[tid] = g;
    if (mm == 0) {
      phis[r] = fabsf(g);
      p.a.phi_q[inst * R + r] = fabsf(g);
    }
  }
  __syncthreads();
  if (tid < R) {                                   // the third layer of psi
    const __half* w3 = reinterpret_cast<const __half*>(cl.own + 3 * R + 4);
    float sacc = 0.f;
#pragma unroll
    for (int rr = 0; rr < R; ++rr) sacc = fmaf(gsum[R + rr], __half2float(w3[rr * R + tid]), sacc);
    p.a.psi_k[inst * R + tid] = fabsf(sacc);       // decode_tail reads it from memory (behind its barriers)
  }

  // ---- low-rank correction and the single normalisation (Eq. 3) ----
  float den = lsum;
  {
    const float em = __expf(-m);
    float lr = 0.f, lz = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const float f = phis[r];
      lr = fmaf(f, hcol[r], lr);
      lz = fmaf(f, zr[r], lz);
    }
    num = fmaf(em, lr, num);
    den = fmaf(em, lz, den);
  }
  store_out(p, inst * kHeadDim + d, num / den);
  const float inv[1] = {1.0f / ((p.flags & LESS_SCORE_NORM_SPARSE) ? lsum : den)};
  decode_tail<R, 1, kCaptured>(p, inst, n, t_now, s_sc, p.Np + 4, inv, hcol, knew, vnew, s_key, &s_vic, cl.tail);
}

template <int R, bool kCaptured>
__global__ void __launch_bounds__(SS_THREADS) small_step_kernel(const __grid_constant__ CUtensorMap tm_w1phi,
                                                                const __grid_constant__ CUtensorMap tm_w1psi, DecParams p,
                                                                SsMaps mp) {
  extern __shared__ __align__(1024) float dsm[];
  float* part = dsm;                                     // [SS_FEAT][2][R]  a decode CTA's inbox for the partial layer-2 sums
  float* role = dsm + 256;                               // the rest belongs to the CTA's role (on a 1024-byte boundary:
                                                         // the feature CTAs' weight tiles are 128-byte-swizzled)
  const int tid = threadIdx.x;
  const int nb = p.B;                                    // <= SS_MAXB
  const int cs = nb + SS_FEAT;                           // CTAs per cluster
  const int rank = (int)cluster_rank();
  const int lh = blockIdx.x / cs;                        // layer * Hd + head
  // "this CTA runs": distributed shared memory may only be touched once its owner has started.  Everyone
  // arrives here at once; whoever needs the fact waits for it much later, when it has long been true.
  cluster_arrive_relaxed();
  // Programmatic dependent launch, both ways: the next kernel in the stream (the next step, typically) may
  // start while this one runs, and this one may have started while its predecessor still ran.  Whatever an
  // earlier kernel may have written - the step's q, k, v, the arena - is read only behind pdl_wait_primary();
  // the feature-map weights never change and are fetched before it.
  pdl_launch_dependents();
  // Operands come as bulk copies that complete on this barrier: a copy per contiguous piece issued by a
  // few threads, where sixteen warps of 16-byte copies took thousands of cycles just to issue.
  __shared__ uint64_t s_stage_bar;
  __shared__ int s_abort;
  if (tid == 0) {
    mbar_init(&s_stage_bar, 1);
    s_abort = 0;
    mbar_fence_init();
  }

  if (rank < nb) {
    // ---------------- decode CTA of batch row `rank` ----------------
    const size_t inst = (size_t)rank * p.LH + lh;
    SsDecoder cl;
    cl.part = part;
    cl.own = role + p.Np + 4 + (SS_THREADS / 16) * kHeadDim;   // behind the step's scores and partial sums
    // Everything the step reads of its instance, asked for at once: the step is otherwise a chain of dependent
    // round trips to L2 (slot count -> K rows -> V rows -> scores and positions -> the victim's psi and V row).
    // While the slots fit; with more of them the rows stream from the arena as in the large kernels.
    cl.K = nullptr;
    cl.tail = TailStage();
    cl.bar = &s_stage_bar; cl.abort = &s_abort;
    __half* w3s = reinterpret_cast<__half*>(cl.own + 3 * R + 4);
    const bool stage = p.N <= SS_STAGE_SLOTS;
    const size_t N = p.N;
    unsigned char* st = reinterpret_cast<unsigned char*>(w3s) + R * R * 2;   // behind W3; 16-byte aligned
    __half* Ks = reinterpret_cast<__half*>(st);
    __half* Vs = Ks + N * kHeadDim;
    float* accs = reinterpret_cast<float*>(Vs + N * kHeadDim);
    int32_t* poss = reinterpret_cast<int32_t*>(accs + p.Np);
    float* psics = reinterpret_cast<float*>(poss + p.Np);
    pdl_wait_primary();
    if (tid == 0) {
      const uint32_t kv = (uint32_t)(N * kHeadDim * 2), ap = (uint32_t)p.Np * 4, ps = (uint32_t)(N * R * 4);
      mbar_expect_tx(&s_stage_bar, (uint32_t)(R * R * 2) + (stage ? 2 * kv + 2 * ap + ps : 0u));
      bulk_g2s(w3s, mp.w3 + (size_t)lh * R * R, R * R * 2, &s_stage_bar);
      if (stage) {
        bulk_g2s(Ks, p.a.kslots + inst * N * kHeadDim, kv, &s_stage_bar);
        bulk_g2s(Vs, p.a.vslots + inst * N * kHeadDim, kv, &s_stage_bar);
        bulk_g2s(accs, p.a.acc + inst * (size_t)p.Np, ap, &s_stage_bar);
        bulk_g2s(poss, p.a.pos + inst * (size_t)p.Np, ap, &s_stage_bar);
        bulk_g2s(psics, p.a.psic + inst * N * R, ps, &s_stage_bar);
      }
    }
    if (tid >= SS_THREADS - 2)                           // psi's learnable scalars, by threads of a warp that has time to wait for them
      cl.own[3 * R + (tid & 1)] = mp.psi_scale ? mp.psi_scale[lh * 2 + (tid & 1)] : 1.f;
    if (stage) {
      cl.K = Ks;
      cl.tail.V = Vs; cl.tail.acc = accs; cl.tail.pos = poss; cl.tail.psic = psics;
    }
    small_step_decode<R, kCaptured>(p, inst, role, cl);  // the barriers inside order these writes before their use
    return;
  }

  // ---------------- feature CTA: 1 / SS_FEAT of the hidden units of both maps ----------------
  // Short rolled loops over operands staged in shared memory; 16 warps, because every phase is a
  // chain of dependent latencies that only other warps can fill.
  const int fr = rank - nb;
  const int Rp = mp.Rp, J = Rp / SS_FEAT;                // hidden units of this CTA: 128, 64 or 32
  const int lj = 31 - __clz(J);                          // J = 1 << lj
  // W1 slice of this CTA: with 64 or 128 hidden units per CTA it comes as tiled TMA loads of 128 rows x 64
  // columns (two or four per CTA; the same tensor maps the tensor-core feature kernels use), 128-byte-swizzled,
  // which the transposing loads below undo; with 32 units (hidden width 128) as 16-byte asynchronous copies into
  // rows padded by 16 bytes.  Either way the eight rows of a transposing load lie in eight different bank groups.
  const bool tiled = J >= 64;
  const int ws = tiled ? 64 : J + 8;                     // halves per staged row
  __half* w1s = reinterpret_cast<__half*>(role);         // tiled: [2 maps][J / 64 halves][128 rows][64]; else [2][128 rows][J + 8]
  __half* xh = w1s + 2 * kHeadDim * (SS_MAXJ + 8);       // [2][SS_MAXB][128] q rows, then k rows
  __half* w2h = xh + 2 * SS_MAXB * kHeadDim;             // [2][J][R] this CTA's rows of W2
  float* hs = reinterpret_cast<float*>(w2h + 2 * SS_MAXJ * R);   // [2][SS_MAXB][SS_MAXJ] gelu(hidden)
  if (tiled) {
    if (smem_misaligned(dsm, p.a.status, 133)) return;   // (a CTA that leaves is no longer waited for by its cluster)
    if (tid == 0) {
      const int halves = J >> 6;
      mbar_expect_tx(&s_stage_bar, (uint32_t)(2 * halves * kHeadDim * 128));
      for (int m = 0; m < 2; ++m)
        for (int i = 0; i < halves; ++i)
          tma_load_2d(w1s + (size_t)(m * halves + i) * kHeadDim * 64, m ? &tm_w1psi : &tm_w1phi, fr * J + i * 64,
                      lh * kHeadDim, &s_stage_bar);
    }
  } else {
    const int lpr = J / 8, llpr = lj - 3;                // 16-byte chunks per weight row of this CTA
    for (int e = tid; e < 2 * kHeadDim * lpr; e += SS_THREADS) {
      const int m = e >> (7 + llpr), d = (e >> llpr) & (kHeadDim - 1), ch = e & (lpr - 1);
      cp_async16(w1s + (size_t)(m * kHeadDim + d) * ws + ch * 8,
                 mp.w1[m] + ((size_t)lh * kHeadDim + d) * Rp + (size_t)fr * J + ch * 8);
    }
  }
  // this CTA's rows of W2 and, once the kernels before this one are done, the few q / k rows with 16-byte
  // asynchronous copies (q, k may lie in pinned host memory)
  const int w2chunks = J * R / 8;                        // 16-byte chunks of this CTA's rows of W2, per map (contiguous)
  if (tid < 2 * w2chunks) {
    const int m = tid >= w2chunks, ch = tid - m * w2chunks;
    cp_async16(w2h + (m * J * R) + ch * 8, mp.w2[m] + ((size_t)lh * Rp + (size_t)fr * J) * R + ch * 8);
  }
  pdl_wait_primary();
  if (tid < 2 * nb * 16) {
    const int m = tid / (nb * 16), b = (tid >> 4) % nb, ch = tid & 15;
    cp_async16(xh + (m * SS_MAXB + b) * kHeadDim + ch * 8,
               (m == 0 ? p.q : p.k) + ((size_t)b * p.LH + lh) * kHeadDim + ch * 8);
  }
  cp_async_wait_all();
  __syncthreads();                                       // ... which also makes the barrier's initialisation visible
  if (tiled) wait_or_give_up(&s_stage_bar, 0, &s_abort, p.a.status, 132);

  // ---- layer 1 as warp-level MMAs (fp16 operands, used exactly; fp32 sums): the head's batch rows are the
  //      first rows of the 16-row A operand (the rest zero), a tile of eight hidden units the B operand, read
  //      from the staged [d][j] rows with transposing loads.  One warp per tile; gelu on the way out. ----
  {
    const int lane = tid & 31, warp = tid >> 5;
    const int row = lane >> 2;                           // batch row of this lane's A and accumulator elements
    const bool live = row < nb;
    const int tiles = J >> 3;                            // per map
    for (int tile = warp; tile < 2 * tiles; tile += SS_THREADS / 32) {
      const int m = tile >= tiles, n0 = (tile - m * tiles) * 8;
      const __half* xrow = xh + (m * SS_MAXB + row) * kHeadDim + 2 * (lane & 3);
      // row k = 32 kk + 8 (lane >> 3) + (lane & 7) of the tile's eight columns: in a swizzled tile the 16-byte
      // chunk c of row k lies at chunk c ^ (k & 7) of its 128-byte row
      const int krow = (lane >> 3) * 8 + (lane & 7);
      const __half* wrow = tiled ? w1s + (size_t)(m * (J >> 6) + (n0 >> 6)) * kHeadDim * 64 + (size_t)krow * 64 +
                                       ((((n0 & 63) >> 3) ^ (lane & 7)) << 3)
                                 : w1s + (size_t)(m * kHeadDim + krow) * ws + n0;
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int kk = 0; kk < kHeadDim / 32; ++kk) {       // two k-steps of 16 input dimensions per pass
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(b0, b1, b2, b3, wrow + (size_t)kk * 32 * ws);
        uint32_t a[4] = {0u, 0u, 0u, 0u};
        if (live) {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) a[q4] = *reinterpret_cast<const uint32_t*>(xrow + kk * 32 + q4 * 8);
        }
        mma_m16n8k16(c, a[0], 0u, a[1], 0u, b0, b1);
        mma_m16n8k16(c, a[2], 0u, a[3], 0u, b2, b3);
      }
      if (live) {
        float* h = hs + (m * SS_MAXB + row) * SS_MAXJ + n0 + 2 * (lane & 3);
        h[0] = gelu_erf(c[0]);
        h[1] = gelu_erf(c[1]);
      }
    }
  }
  __syncthreads();
  cluster_wait();                                        // the start-up phase: every decode CTA of the cluster runs
  // ---- layer 2, this CTA's share: sum_j gelu(h_j) W2[j][r] into the inbox of the decode CTA of batch row b;
  //      eight lanes per output, each over every eighth hidden unit, then a fixed shuffle tree ----
#pragma unroll 1
  for (int e0 = 0; e0 < 2 * nb * R; e0 += SS_THREADS / 8) {   // uniform over the CTA: the shuffles stay converged
    const int e = e0 + (tid >> 3), jp = tid & 7;
    const bool on = e < 2 * nb * R;
    const int m = e >= nb * R, rem = e - m * nb * R, b = rem / R, r = rem % R;
    float a = 0.f;
    if (on) {
      const float* h = hs + (m * SS_MAXB + b) * SS_MAXJ;
      const __half* w = w2h + m * J * R + r;
#pragma unroll 4
      for (int j = jp; j < J; j += 8) a = fmaf(h[j], __half2float(w[j * R]), a);
    }
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if (on && jp == 0) cluster_peer_store_f32(part + (fr * 2 + m) * R + r, (uint32_t)b, a);
  }
  cluster_arrive();                                      // releases the stores above to the decode CTAs; nothing to wait for
}

// --------------------------------------------------------------------------- //
// Grouped query heads (Section 3.2, multi-query attention): G query heads share one KV head.
// One 128-thread CTA per KV head; every query head has its own phi and its own Eq. 3 (own
// normaliser) over the shared slots and the shared H, z; then the G heads' probabilities are
// added into the entries' H2O scores and one entry leaves for all heads.
// CUDA-core version: every K / V row is loaded and converted once and meets the G queries in
// registers.
// --------------------------------------------------------------------------- //
template <int R, int G, bool kCaptured>
__global__ void __launch_bounds__(DEC_THREADS) decode_group_rows_kernel(DecParams p) {
  extern __shared__ float dsm[];
  pdl_launch_dependents();                         // the next step's feature-map kernel may come up while this one runs
  const int Ns = p.Np + 4;
  float* s_sc = dsm;                               // [G][Np + 4] scores, then e^{s - m_g}
  float* s_red = s_sc + G * Ns;                    // [G][DEC_RG][128] partial numerators
  __shared__ float s_small[DEC_THREADS / 32];
  __shared__ unsigned long long s_key[DEC_THREADS / 32];
  __shared__ int s_vic;
  __shared__ float s_inv[G];

  const int tid = threadIdx.x;
  const size_t inst = decode_instance(p);
  const int l16 = tid & 15, rg = tid >> 4;
  const int N = p.N;
  const int t_now = kCaptured ? __ldcg(p.a.tpos) : p.t;
  int n = p.a.count[inst];
  if (n < 0 || n > N) {
    if (tid == 0) set_status(p.a.status, kStatusBounds, 1);
    step_done<kCaptured>(p);
    return;
  }
  const bool use_state = !(p.flags & LESS_NO_STATE);
  const float scale = 0.08838834764831845f;        // 1 / sqrt(128)

  const __half* Kb = p.a.kslots + inst * (size_t)N * kHeadDim;
  const __half* Vb = p.a.vslots + inst * (size_t)N * kHeadDim;

  float qf[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g)
    half8_to_float(*reinterpret_cast<const uint4*>(p.q + (inst * G + g) * kHeadDim + l16 * 8), qf[g]);

  // ---- scores of the G heads against every live slot (each K row is read once) ----
#pragma unroll 2
  for (int r0 = 0; r0 < n; r0 += DEC_RG) {
    const int r = r0 + rg;
    float dot[G];
#pragma unroll
    for (int g = 0; g < G; ++g) dot[g] = 0.f;
    if (r < n) {
      float kf[8];
      half8_to_float(ldg_stream(Kb + (size_t)r * kHeadDim + l16 * 8), kf);
#pragma unroll
      for (int g = 0; g < G; ++g)
#pragma unroll
        for (int c = 0; c < 8; ++c) dot[g] = fmaf(qf[g][c], kf[c], dot[g]);
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) dot[g] += __shfl_xor_sync(0xffffffffu, dot[g], o);
      if (l16 == 0 && r < n) s_sc[g * Ns + r] = dot[g] * scale;
    }
  }
  const uint4 knew = *reinterpret_cast<const uint4*>(p.k + inst * kHeadDim + l16 * 8);
  const uint4 vnew = *reinterpret_cast<const uint4*>(p.v + inst * kHeadDim + l16 * 8);
  if (tid < 32) {
    float kf[8];
    half8_to_float(knew, kf);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float dot = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) dot = fmaf(qf[g][c], kf[c], dot);
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      if (tid == 0) s_sc[g * Ns + n] = dot * scale;
    }
  }
  __syncthreads();

  // ---- per head: m_g, e_i = exp(s_i - m_g), l_g ----
  __shared__ float s_ml[2][G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    float* sc = s_sc + g * Ns;
    float m = -INFINITY;
    for (int i = tid; i <= n; i += DEC_THREADS) m = fmaxf(m, sc[i]);
    m = block_max(m, s_small);
    m = fmaxf(m, -80.f);
    float lsum = 0.f;
    for (int i = tid; i <= n; i += DEC_THREADS) {
      const float e = __expf(sc[i] - m);
      sc[i] = e;
      lsum += e;
    }
    lsum = block_sum(lsum, s_small);
    if (tid == 0) { s_ml[0][g] = m; s_ml[1][g] = lsum; }
  }

  // ---- u_g = sum e_{g,i} v_i (each V row is read once) ----
  float u[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int c = 0; c < 8; ++c) u[g][c] = 0.f;
#pragma unroll 2
  for (int r = rg; r < n; r += DEC_RG) {
    float vf[8];
    half8_to_float(ldg_stream(Vb + (size_t)r * kHeadDim + l16 * 8), vf);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float e = s_sc[g * Ns + r];
#pragma unroll
      for (int c = 0; c < 8; ++c) u[g][c] = fmaf(e, vf[c], u[g][c]);
    }
  }
  if (rg == 0) {
    float vf[8];
    half8_to_float(vnew, vf);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float e = s_sc[g * Ns + n];
#pragma unroll
      for (int c = 0; c < 8; ++c) u[g][c] = fmaf(e, vf[c], u[g][c]);
    }
  }
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int c = 0; c < 8; ++c) s_red[(g * DEC_RG + rg) * kHeadDim + l16 * 8 + c] = u[g][c];
  __syncthreads();

  group_eq3_and_tail<R, G, kCaptured, DEC_RG>(p, inst, n, t_now, s_sc, Ns, s_red, s_ml[0], s_ml[1], knew, vnew, s_inv, s_key, &s_vic);
}


__device__ __forceinline__ uint32_t word_of(const uint4& v, int w) {
  return w == 0 ? v.x : w == 1 ? v.y : w == 2 ? v.z : v.w;
}

constexpr int kMmaRed = DEC_THREADS / 32 + 1;   // partial numerators per head in the mma kernel

// The same step with the two contractions on the tensor cores.  With G query heads per KV head the
// scores are a [slots x 128] x [128 x G] product and the numerators a [128 x slots] x [slots x G] one:
// dense, but only G <= 8 wide and bound by the K / V stream, so the warp-level mma (m16n8k16, fp16
// inputs used exactly, fp32 accumulation, N = 8 = the heads) fits: its fragments load straight from
// global memory with no staging, four warps split the 16-slot tiles.  The probabilities enter the
// second product rounded to fp16 (relative 4.9e-4, like the prompt-output kernel); the H2O scores
// use the fp32 values.
template <int R, int G, bool kCaptured>
__global__ void __launch_bounds__(DEC_THREADS) decode_group_mma_kernel(DecParams p) {
  extern __shared__ float dsm[];
  pdl_launch_dependents();                         // the next step's feature-map kernel may come up while this one runs
  const int Ns = p.Np + 4;
  float* s_sc = dsm;                               // [G][Np + 4] scores, then e^{s - m_g}
  float* s_red = s_sc + G * Ns;                    // [G][kMmaRed][128] partial numerators: one row per warp, one for the new pair
  __shared__ float s_small[DEC_THREADS / 32];
  __shared__ unsigned long long s_key[DEC_THREADS / 32];
  __shared__ int s_vic;
  __shared__ float s_inv[G];

  const int tid = threadIdx.x;
  const size_t inst = decode_instance(p);
  const int l16 = tid & 15, rg = tid >> 4;
  const int N = p.N;
  const int t_now = kCaptured ? __ldcg(p.a.tpos) : p.t;
  int n = p.a.count[inst];
  if (n < 0 || n > N) {
    if (tid == 0) set_status(p.a.status, kStatusBounds, 1);
    step_done<kCaptured>(p);
    return;
  }
  const bool use_state = !(p.flags & LESS_NO_STATE);
  const float scale = 0.08838834764831845f;        // 1 / sqrt(128)

  const __half* Kb = p.a.kslots + inst * (size_t)N * kHeadDim;
  const __half* Vb = p.a.vslots + inst * (size_t)N * kHeadDim;

  const int warp = tid >> 5, lane = tid & 31;
  const int fg = lane >> 2, ft = lane & 3;         // fragment coordinates of mma.m16n8k16: row group, thread in group
  constexpr int Ng = G;
  // ---- scores: S[16 slots x 8 heads] += K[16 slots x 16 dims] Q^T[16 dims x 8 heads], 8 k-steps per tile ----
  // The contraction does not care which dims a k-slot stands for, as long as both operands agree:
  // thread ft takes the 16-byte chunks ft, ft + 4, ft + 8, ft + 12 of a row, so every load is a
  // whole chunk and a warp reads its 16 rows (4 KB) exactly once.
  uint4 qfrag[4];                                  // B fragments: head fg, this thread's chunks
#pragma unroll
  for (int c = 0; c < 4; ++c)
    qfrag[c] = fg < Ng ? *reinterpret_cast<const uint4*>(p.q + (inst * G + fg) * kHeadDim + (ft + 4 * c) * 8)
                       : make_uint4(0, 0, 0, 0);
  const int ntile16 = (n + 15) >> 4;
  for (int tl = warp; tl < ntile16; tl += DEC_THREADS / 32) {
    const int r0 = tl * 16 + fg, r1 = r0 + 8;
    const int c0 = min(r0, n - 1), c1 = min(r1, n - 1);        // rows past the live slots repeat the last one; their scores are dropped
    uint4 ka[4], kb[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      ka[c] = ldg_stream(Kb + (size_t)c0 * kHeadDim + (ft + 4 * c) * 8);
      kb[c] = ldg_stream(Kb + (size_t)c1 * kHeadDim + (ft + 4 * c) * 8);
    }
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      mma_m16n8k16(acc, ka[c].x, kb[c].x, ka[c].y, kb[c].y, qfrag[c].x, qfrag[c].y);
      mma_m16n8k16(acc, ka[c].z, kb[c].z, ka[c].w, kb[c].w, qfrag[c].z, qfrag[c].w);
    }
    // acc: (slot r0, head 2 ft), (r0, 2 ft + 1), (r1, 2 ft), (r1, 2 ft + 1)
    if (2 * ft < Ng) {
      if (r0 < n) s_sc[(2 * ft) * Ns + r0] = acc[0] * scale;
      if (r1 < n) s_sc[(2 * ft) * Ns + r1] = acc[2] * scale;
    }
    if (2 * ft + 1 < Ng) {
      if (r0 < n) s_sc[(2 * ft + 1) * Ns + r0] = acc[1] * scale;
      if (r1 < n) s_sc[(2 * ft + 1) * Ns + r1] = acc[3] * scale;
    }
  }
  const uint4 knew = *reinterpret_cast<const uint4*>(p.k + inst * kHeadDim + l16 * 8);
  const uint4 vnew = *reinterpret_cast<const uint4*>(p.v + inst * kHeadDim + l16 * 8);
  if (tid < 32) {
    float kf[8];
    half8_to_float(knew, kf);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float qf[8];
      half8_to_float(*reinterpret_cast<const uint4*>(p.q + (inst * G + g) * kHeadDim + l16 * 8), qf);
      float dot = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) dot = fmaf(qf[c], kf[c], dot);
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      if (tid == 0) s_sc[g * Ns + n] = dot * scale;
    }
  }
  __syncthreads();

  // ---- per head: m_g, e_i = exp(s_i - m_g), l_g ----
  __shared__ float s_ml[2][G];
  if (G >= DEC_THREADS / 32) {                      // a warp takes whole heads: no block barrier per head
    for (int g = warp; g < G; g += DEC_THREADS / 32) {
      float* sc = s_sc + g * Ns;
      float m = -INFINITY;
      for (int i = lane; i <= n; i += 32) m = fmaxf(m, sc[i]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      m = fmaxf(m, -80.f);
      float lsum = 0.f;
      for (int i = lane; i <= n; i += 32) {
        const float e = __expf(sc[i] - m);
        sc[i] = e;
        lsum += e;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);   // fixed order
      if (lane == 0) { s_ml[0][g] = m; s_ml[1][g] = lsum; }
    }
    __syncthreads();
  } else {                                          // fewer heads than warps: the whole CTA works on each
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float* sc = s_sc + g * Ns;
      float m = -INFINITY;
      for (int i = tid; i <= n; i += DEC_THREADS) m = fmaxf(m, sc[i]);
      m = block_max(m, s_small);
      m = fmaxf(m, -80.f);
      float lsum = 0.f;
      for (int i = tid; i <= n; i += DEC_THREADS) {
        const float e = __expf(sc[i] - m);
        sc[i] = e;
        lsum += e;
      }
      lsum = block_sum(lsum, s_small);
      if (tid == 0) { s_ml[0][g] = m; s_ml[1][g] = lsum; }
    }
  }

  // ---- O^T[16 dims x 8 heads] += V^T[16 dims x 16 slots] P^T[16 slots x 8 heads], 8 tiles of dims per 16 slots ----
  // A fragment row fg of tile m stands for dim 8 fg + m, row fg + 8 for dim 8 (fg + 8) + m: a thread
  // loads the chunks fg and fg + 8 of its four slots (k-slots 2 ft, 2 ft + 1, 2 ft + 8, 2 ft + 9)
  // and pairs the halves of two slots with a byte permute; again every byte is loaded once.
  float oacc[8][4];
#pragma unroll
  for (int m = 0; m < 8; ++m)
#pragma unroll
    for (int x = 0; x < 4; ++x) oacc[m][x] = 0.f;
  for (int tl = warp; tl < ntile16; tl += DEC_THREADS / 32) {
    const int base = tl * 16 + 2 * ft;
    const int rr[4] = {base, base + 1, base + 8, base + 9};
    uint4 va[4], vb[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const int row = min(rr[x], n - 1);
      va[x] = ldg_stream(Vb + (size_t)row * kHeadDim + fg * 8);
      vb[x] = ldg_stream(Vb + (size_t)row * kHeadDim + (fg + 8) * 8);
    }
    uint32_t b0 = 0u, b1 = 0u;                     // B fragment: head fg, this thread's four slots (zero past the live ones)
    if (fg < Ng) {
      const float* sc = s_sc + fg * Ns;
      const __half2 h0 = __floats2half2_rn(rr[0] < n ? sc[rr[0]] : 0.f, rr[1] < n ? sc[rr[1]] : 0.f);
      const __half2 h1 = __floats2half2_rn(rr[2] < n ? sc[rr[2]] : 0.f, rr[3] < n ? sc[rr[3]] : 0.f);
      b0 = *reinterpret_cast<const uint32_t*>(&h0);
      b1 = *reinterpret_cast<const uint32_t*>(&h1);
    }
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      const int w = m >> 1;
      const uint32_t sel = (m & 1) ? 0x7632u : 0x5410u;      // the high or the low halves of two words
      mma_m16n8k16(oacc[m], __byte_perm(word_of(va[0], w), word_of(va[1], w), sel),
                   __byte_perm(word_of(vb[0], w), word_of(vb[1], w), sel),
                   __byte_perm(word_of(va[2], w), word_of(va[3], w), sel),
                   __byte_perm(word_of(vb[2], w), word_of(vb[3], w), sel), b0, b1);
    }
  }
  // oacc[m]: (dim 8 fg + m, head 2 ft), (same, 2 ft + 1), (dim 8 (fg + 8) + m, head 2 ft), (same, 2 ft + 1)
  // partial numerators: rows 0..3 of s_red per head are the warps', row 4 the new pair's
#pragma unroll
  for (int m = 0; m < 8; ++m) {
    const int d0 = 8 * fg + m, d1 = 8 * (fg + 8) + m;
    if (2 * ft < Ng) {
      s_red[((2 * ft) * kMmaRed + warp) * kHeadDim + d0] = oacc[m][0];
      s_red[((2 * ft) * kMmaRed + warp) * kHeadDim + d1] = oacc[m][2];
    }
    if (2 * ft + 1 < Ng) {
      s_red[((2 * ft + 1) * kMmaRed + warp) * kHeadDim + d0] = oacc[m][1];
      s_red[((2 * ft + 1) * kMmaRed + warp) * kHeadDim + d1] = oacc[m][3];
    }
  }
  {
    const float vn = __half2float(p.v[inst * kHeadDim + tid]);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      s_red[(g * kMmaRed + 4) * kHeadDim + tid] = s_sc[g * Ns + n] * vn;
    }
  }
  __syncthreads();

  group_eq3_and_tail<R, G, kCaptured, kMmaRed>(p, inst, n, t_now, s_sc, Ns, s_red, s_ml[0], s_ml[1], knew, vnew, s_inv, s_key, &s_vic);
}

// --------------------------------------------------------------------------- //
// The same step for shapes the kernels above do not take: head dimension 64 or 128 and any number
// of query heads per KV head (the multi-query model the paper evaluates has 71 query heads over
// one KV head of dimension 64).  CUDA cores; one 128-thread CTA per KV head.  The query heads are
// taken eight at a time: every pass scores its heads against all live slots (the K and V rows of the
// later passes come from L1 / L2), runs their softmaxes (a warp per head) and their Eq. 3, and
// adds its heads' probabilities into one sum per entry; the tail then works on that sum as if it were
// a single head's probability.
// --------------------------------------------------------------------------- //
constexpr int kLoopHeads = 8;     // query heads per pass

template <int R, int D, bool kCaptured>
__global__ void __launch_bounds__(DEC_THREADS) decode_group_loop_kernel(DecParams p, int G) {
  constexpr int LPR = D / 8;                       // lanes per slot row
  constexpr int RGN = DEC_THREADS / LPR;           // row groups
  constexpr int GC = kLoopHeads;
  extern __shared__ float dsm[];
  pdl_launch_dependents();
  const int Ns = p.Np + 4;
  float* s_e = dsm;                                // [GC][Ns] scores of this pass's heads, then e^{s - m_g}
  float* s_ps = s_e + GC * Ns;                     // [Ns] sum over all heads of their probabilities
  float* s_red = s_ps + Ns;                        // [GC][RGN][D] partial numerators
  __shared__ float s_ml[2][GC];
  __shared__ float s_inv[GC];
  __shared__ unsigned long long s_key[DEC_THREADS / 32];
  __shared__ int s_vic;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int lp = tid % LPR, rg = tid / LPR, d = tid;
  const bool own = D == DEC_THREADS || d < D;
  const size_t inst = decode_instance(p);
  const int N = p.N;
  const int t_now = kCaptured ? __ldcg(p.a.tpos) : p.t;
  int n = p.a.count[inst];
  if (n < 0 || n > N) {
    if (tid == 0) set_status(p.a.status, kStatusBounds, 1);
    step_done<kCaptured>(p);
    return;
  }
  const bool use_state = !(p.flags & LESS_NO_STATE);
  const float scale = D == 64 ? 0.125f : 0.08838834764831845f;   // 1 / sqrt(D)
  const __half* Kb = p.a.kslots + inst * (size_t)N * D;
  const __half* Vb = p.a.vslots + inst * (size_t)N * D;
  const uint4 knew = *reinterpret_cast<const uint4*>(p.k + inst * D + lp * 8);
  const uint4 vnew = *reinterpret_cast<const uint4*>(p.v + inst * D + lp * 8);
  for (int i = tid; i <= n; i += DEC_THREADS) s_ps[i] = 0.f;
  float hcol[R], zr[R];
#pragma unroll
  for (int r = 0; r < R; ++r) hcol[r] = zr[r] = 0.f;

  for (int g0 = 0; g0 < G; g0 += GC) {
    const int gc = min(GC, G - g0);
    float qf[GC][8];
#pragma unroll
    for (int g = 0; g < GC; ++g) {
      if (g < gc) half8_to_float(*reinterpret_cast<const uint4*>(p.q + (inst * G + g0 + g) * D + lp * 8), qf[g]);
      else
#pragma unroll
        for (int c = 0; c < 8; ++c) qf[g][c] = 0.f;
    }
    // ---- scores of this pass's heads against every live slot and the new pair ----
    for (int r0 = 0; r0 <= n; r0 += RGN) {          // r0 is block-uniform: shuffles stay converged; row n = the new pair
      const int r = r0 + rg;
      float dot[GC];
#pragma unroll
      for (int g = 0; g < GC; ++g) dot[g] = 0.f;
      if (r <= n) {
        float kf[8];
        half8_to_float(r < n ? *reinterpret_cast<const uint4*>(Kb + (size_t)r * D + lp * 8) : knew, kf);
#pragma unroll
        for (int g = 0; g < GC; ++g)
#pragma unroll
          for (int c = 0; c < 8; ++c) dot[g] = fmaf(qf[g][c], kf[c], dot[g]);
      }
#pragma unroll
      for (int g = 0; g < GC; ++g) {
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) dot[g] += __shfl_xor_sync(0xffffffffu, dot[g], o);
        if (lp == 0 && r <= n) s_e[g * Ns + r] = dot[g] * scale;
      }
    }
    __syncthreads();
    // ---- per head: m_g, e_i = exp(s_i - m_g), l_g (a warp takes whole heads) ----
    for (int g = warp; g < gc; g += DEC_THREADS / 32) {
      float* sc = s_e + g * Ns;
      float m = -INFINITY;
      for (int i = lane; i <= n; i += 32) m = fmaxf(m, sc[i]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      m = fmaxf(m, -80.f);
      float lsum = 0.f;
      for (int i = lane; i <= n; i += 32) {
        const float e = __expf(sc[i] - m);
        sc[i] = e;
        lsum += e;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);   // fixed order
      if (lane == 0) { s_ml[0][g] = m; s_ml[1][g] = lsum; }
    }
    __syncthreads();
    // ---- u_g = sum e_{g,i} v_i over the live slots and the new pair ----
    float u[GC][8];
#pragma unroll
    for (int g = 0; g < GC; ++g)
#pragma unroll
      for (int c = 0; c < 8; ++c) u[g][c] = 0.f;
    for (int r = rg; r <= n; r += RGN) {
      float vf[8];
      half8_to_float(r < n ? *reinterpret_cast<const uint4*>(Vb + (size_t)r * D + lp * 8) : vnew, vf);
#pragma unroll
      for (int g = 0; g < GC; ++g) {
        const float e = g < gc ? s_e[g * Ns + r] : 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) u[g][c] = fmaf(e, vf[c], u[g][c]);
      }
    }
#pragma unroll
    for (int g = 0; g < GC; ++g)
#pragma unroll
      for (int c = 0; c < 8; ++c) s_red[(g * RGN + rg) * D + lp * 8 + c] = u[g][c];
    __syncthreads();
    // ---- Eq. 3 of each head over the KV head's shared H, z ----
    if (g0 == 0 && use_state) {
      wait_feature_maps<1>(p, 0);                    // general shapes never run with per-head counters: waits for the whole feature-map grid
      if (own) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
          hcol[r] = p.a.H[(inst * R + r) * D + d];
          zr[r] = p.a.z[inst * R + r];
        }
      }
    }
    if (own) {
      for (int g = 0; g < gc; ++g) {
        float num = 0.f;
#pragma unroll
        for (int j = 0; j < RGN; ++j) num += s_red[(g * RGN + j) * D + d];
        const float lg = s_ml[1][g];
        float den = lg;
        if (use_state) {
          const float em = __expf(-s_ml[0][g]);
          const float* ph = p.a.phi_q + (inst * G + g0 + g) * R;
          float lr = 0.f, lz = 0.f;
#pragma unroll
          for (int r = 0; r < R; ++r) {
            const float f = __ldcg(ph + r);
            lr = fmaf(f, hcol[r], lr);
            lz = fmaf(f, zr[r], lz);
          }
          num = fmaf(em, lr, num);
          den = fmaf(em, lz, den);
        }
        store_out(p, (inst * G + g0 + g) * D + d, num / den);
        if (d == 0) s_inv[g] = 1.0f / ((p.flags & LESS_SCORE_NORM_SPARSE) ? lg : den);
      }
    }
    __syncthreads();
    // ---- this pass's share of the aggregated probabilities ----
    for (int i = tid; i <= n; i += DEC_THREADS) {
      float ps = s_ps[i];
      for (int g = 0; g < gc; ++g) ps = fmaf(s_e[g * Ns + i], s_inv[g], ps);
      s_ps[i] = ps;
    }
    __syncthreads();                                 // before the next pass rewrites s_e, s_ml, s_inv
  }
  const float one[1] = {1.0f};
  decode_tail<R, 1, kCaptured, D>(p, inst, n, t_now, s_ps, Ns, one, hcol, knew, vnew, s_key, &s_vic);
}

template <int R, int D>
static void* decode_loop_entry(bool captured) {
  return captured ? (void*)decode_group_loop_kernel<R, D, true> : (void*)decode_group_loop_kernel<R, D, false>;
}

size_t decode_loop_smem_bytes(int Np, int D) {
  return ((size_t)(kLoopHeads + 1) * (Np + 4) + (size_t)kLoopHeads * (DEC_THREADS / (D / 8)) * D) * 4;
}

size_t decode_smem_bytes(const Dims& d) {
  return (size_t)d.G * (d.Np + 4 + DEC_RG * kHeadDim) * 4;
}

// which: 2 the CUDA-core version, 3 (default) the one with the contractions on the tensor cores
template <int R, int G>
static void* decode_group_entry(bool captured, int which) {
  if (which == 2)
    return captured ? (void*)decode_group_rows_kernel<R, G, true> : (void*)decode_group_rows_kernel<R, G, false>;
  return captured ? (void*)decode_group_mma_kernel<R, G, true> : (void*)decode_group_mma_kernel<R, G, false>;
}

int launch_decode(less_ctx* c, const void* q, const void* k, const void* v, void* out,
                  int32_t* evicted_pos, cudaStream_t s) {
  const Dims& d = c->d;
  DecParams p;
  p.q = (const __half*)q; p.k = (const __half*)k; p.v = (const __half*)v;
  p.out = out;
  p.evicted_pos = evicted_pos;
  p.a = c->a;
  p.N = d.N; p.Np = d.Np; p.heavy = d.heavy; p.recent = d.recent;
  p.t = (int)c->t;
  p.B = d.B; p.LH = d.L * d.Hd;
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  cudaStreamIsCapturing(s, &capturing);
  const bool captured = capturing == cudaStreamCaptureStatusActive;   // then the position is read from, and advanced in, device memory
  p.flags = d.flags;
  // this step's feature-map launch published per-head counters: wait for the instance's own only
  p.feat_flag = c->flags_this_step ? c->a.feat_flag : nullptr;
  p.flag_stride = d.L * d.Hd * d.G;
  p.flag_target[0] = c->flag_target[0];
  p.flag_target[1] = c->flag_target[1];
  const bool segment = c->seg_nl != d.L;            // a layer range: CTAs are numbered inside it, head-major
  p.lh0 = c->seg_l0 * d.Hd;
  p.head_major = (p.feat_flag != nullptr && d.B > 1) || segment;
  size_t smem = decode_smem_bytes(d);
  int which = c->group_path == 2 ? 2 : 3;
  char name[64];
  if (d.G == 1) snprintf(name, sizeof name, "decode_kernel<%d, %d>", d.R, (int)captured);
  else snprintf(name, sizeof name, "decode_group_%s_kernel<%d, %d, %d>", which == 2 ? "rows" : "mma", d.R, d.G, (int)captured);
  LaunchScope scope(c, LESS_KERNEL_DECODE, s, name);
  void* kern = d.R == 8 ? (captured ? (void*)decode_kernel<8, true> : (void*)decode_kernel<8, false>)
                        : (captured ? (void*)decode_kernel<16, true> : (void*)decode_kernel<16, false>);
  if (d.G > 1 && which == 3) smem = (size_t)d.G * (d.Np + 4 + kMmaRed * kHeadDim) * 4;
  int G_arg = d.G;
  if (d.general) {
    smem = decode_loop_smem_bytes(d.Np, d.D);
    kern = d.D == 64 ? (d.R == 8 ? decode_loop_entry<8, 64>(captured) : decode_loop_entry<16, 64>(captured))
                     : (d.R == 8 ? decode_loop_entry<8, 128>(captured) : decode_loop_entry<16, 128>(captured));
    snprintf(c->variant[LESS_KERNEL_DECODE], sizeof c->variant[0], "decode_group_loop_kernel<%d, %d, %d>", d.R, d.D, (int)captured);
  }
  if (!d.general && d.G == 2) kern = d.R == 8 ? decode_group_entry<8, 2>(captured, which) : decode_group_entry<16, 2>(captured, which);
  if (!d.general && d.G == 4) kern = d.R == 8 ? decode_group_entry<8, 4>(captured, which) : decode_group_entry<16, 4>(captured, which);
  if (!d.general && d.G == 8) kern = d.R == 8 ? decode_group_entry<8, 8>(captured, which) : decode_group_entry<16, 8>(captured, which);
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return fail_cuda("shared memory opt-in of decode_kernel");
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(segment ? d.B * c->seg_nl * d.Hd : d.I);
  p.done_ctas = (int)cfg.gridDim.x;
  cfg.blockDim = dim3(DEC_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  // Directly behind this step's feature-map kernel the decode kernel may start early and overlap
  // its K / V reads with the weight stream (it waits for the feature maps on the device).  With
  // per-kernel timing on, or without feature maps, it is an ordinary launch.
  const bool overlap = overlap_decode(c);
  cfg.attrs = attr;
  cfg.numAttrs = overlap ? 1 : 0;
  void* args[] = {&p, &G_arg};                         // the second argument is the general kernel's only
  if (cudaLaunchKernelExC(&cfg, kern, args) != cudaSuccess) return fail_cuda("launch of decode_kernel");
  return check_launch("decode_kernel");
}

// Whether a step of this context runs as the single small_step_kernel launch: the shapes the kernel
// takes, and (unless forced) no more CTAs than two per multiprocessor - up to there a step is bound by
// launches and latency (measured, batch 1: 8 heads 6.7 against 8.7 us per step replayed from a graph, 7.7
// against 11.3 us by direct calls; 32 heads 7.6 against 9.0 and 7.7 against 11.2; 64 heads 11.8 against
// 9.5 and 11.6 against 11.8), past it by the weight stream, which the tensor-core feature kernel moves faster.
bool small_step_path(const less_ctx* c) {
  const Dims& d = c->d;
  if (c->small_step == 0 || d.general || d.G != 1 || d.D != kHeadDim || (d.flags & LESS_NO_STATE)) return false;
  if (d.B > SS_MAXB || (d.Rp != 128 && d.Rp != 256 && d.Rp != 512) || c->seg_nl != d.L) return false;
  if (c->feature_path != 2) return false;             // a feature-map kernel was asked for by name
  return c->small_step == 1 || d.L * d.Hd * (d.B + SS_FEAT) <= 2 * c->sms;
}

int launch_small_step(less_ctx* c, const void* q, const void* k, const void* v, void* out, int32_t* evicted_pos,
                      cudaStream_t s) {
  const Dims& d = c->d;
  DecParams p;
  p.q = (const __half*)q; p.k = (const __half*)k; p.v = (const __half*)v;
  p.out = out;
  p.evicted_pos = evicted_pos;
  p.a = c->a;
  p.N = d.N; p.Np = d.Np; p.heavy = d.heavy; p.recent = d.recent;
  p.t = (int)c->t;
  p.B = d.B; p.LH = d.L * d.Hd;
  p.flags = d.flags;
  p.feat_flag = nullptr; p.flag_stride = 0; p.flag_target[0] = p.flag_target[1] = 0;
  p.head_major = 0; p.lh0 = 0;
  p.done_ctas = d.I;
  SsMaps mp;
  mp.w1[0] = (const __half*)c->w.w_phi1; mp.w1[1] = (const __half*)c->w.w_psi1;
  mp.w2[0] = (const __half*)c->w.w_phi2; mp.w2[1] = (const __half*)c->w.w_psi2;
  mp.w3 = (const __half*)c->w.w_psi3;
  mp.psi_scale = c->w.psi_scale;
  mp.Rp = d.Rp;
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  cudaStreamIsCapturing(s, &capturing);
  const bool captured = capturing == cudaStreamCaptureStatusActive;
  // the partial sums, then the larger of the two roles' shared memory
  size_t dec_bytes = (size_t)(d.Np + 4 + (SS_THREADS / 16) * kHeadDim) * 4 + (size_t)(3 * d.R + 4) * 4 + (size_t)d.R * d.R * 2;
  if (d.N <= SS_STAGE_SLOTS) dec_bytes += (size_t)2 * d.N * kHeadDim * 2 + (size_t)2 * d.Np * 4 + (size_t)d.N * d.R * 4;
  const size_t feat_bytes = (size_t)2 * kHeadDim * (SS_MAXJ + 8) * 2 + (size_t)2 * SS_MAXB * kHeadDim * 2 +
                            (size_t)2 * SS_MAXJ * d.R * 2 + (size_t)2 * SS_MAXB * SS_MAXJ * 4;
  const size_t smem = 1024 + (dec_bytes > feat_bytes ? dec_bytes : feat_bytes);
  // a step this small is bound by the host's work per launch as well: names and attributes are set once
  LaunchScope scope(c, LESS_KERNEL_DECODE, s);
  void* kern = d.R == 8 ? (captured ? (void*)small_step_kernel<8, true> : (void*)small_step_kernel<8, false>)
                        : (captured ? (void*)small_step_kernel<16, true> : (void*)small_step_kernel<16, false>);
  if (!c->small_step_ready[captured]) {
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return fail_cuda("shared memory opt-in of small_step_kernel");
    c->small_step_ready[captured] = true;
  }
  if (c->small_step_named != (int)captured) {
    snprintf(c->variant[LESS_KERNEL_DECODE], sizeof c->variant[0], "small_step_kernel<%d, %d>", d.R, (int)captured);
    c->variant[LESS_KERNEL_FEATURE_MAP][0] = 0;         // no feature-map kernel of its own
    c->small_step_named = (int)captured;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(d.L * d.Hd * (d.B + SS_FEAT));
  cfg.blockDim = dim3(SS_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = d.B + SS_FEAT;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (c->pdl && !c->profile) ? 2 : 1;       // with per-kernel timing on, an ordinary launch
  // W1 of phi / psi as tensor maps (boxes of 128 rows x 64 columns, 128-byte-swizzled), kept in the context
  // like the feature kernels' (the same two maps)
  static_assert(sizeof(CUtensorMap) <= 128, "tensor map cache slot");
  CUtensorMap* tmc = reinterpret_cast<CUtensorMap*>(c->tm_cache);
  if (!c->tm_w_ok) {
    const uint64_t lh = (uint64_t)d.L * d.Hd;
    if (!make_tmap_f16_2d(&tmc[2], c->w.w_phi1, lh * kHeadDim, d.Rp, (uint64_t)d.Rp * 2, kHeadDim) ||
        !make_tmap_f16_2d(&tmc[3], c->w.w_psi1, lh * kHeadDim, d.Rp, (uint64_t)d.Rp * 2, kHeadDim))
      return fail_cuda("tensor map of W1");
    c->tm_w_ok = true;
  }
  void* args[] = {&tmc[2], &tmc[3], &p, &mp};
  if (cudaLaunchKernelExC(&cfg, kern, args) != cudaSuccess) return fail_cuda("launch of small_step_kernel");
  return check_launch("small_step_kernel");
}

}  // namespace less
