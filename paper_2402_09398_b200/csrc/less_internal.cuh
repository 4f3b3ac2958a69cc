// Internal definitions shared by the translation units of the LESS library:
// the context, the arena layout and small device helpers.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include <vector>

#include "less.h"

namespace less {

constexpr int kHeadDim = 128;       // D
constexpr int kMaxSplit = 32;       // token splits of the prompt state build
constexpr int kSplitTokens = 256;   // tokens per split (lower bound)

// Device views of the arena.  All arrays are instance-major.
struct Arena {
  __half* kslots;    // [I][N][D]
  __half* vslots;    // [I][N][D]
  int32_t* pos;      // [I][Np]     absolute position of the token in a slot
  float* acc;        // [I][Np]     H2O accumulated attention probability
  float* psic;       // [I][N][R]   psi(k) of the token in a slot (evaluated at insertion)
  float* H;          // [I][R][D]   Eq. 4
  float* z;          // [I][R]      Eq. 5
  int32_t* count;    // [I]         live slots
  float* phi_q;      // [I*G][R]    phi(q_t) of the current step, per query head
  float* psi_k;      // [I][R]      psi(k_t) of the current step
  int32_t* status;   // [4]         device status word(s)
  int32_t* tpos;     // [4]         [0] tokens seen = position of the next decode token, [1] decode CTAs finished this step
  uint32_t* feat_flag; // [L*Hd*G + L*Hd]  per (layer, head): writer warps of the feature-map kernel that have published
                     //             phi(q_t) (first L*Hd*G entries, per query head) / psi(k_t) so far, over all steps
  __half* stage_q;   // [I*G][D]    staging of host inputs (less_decode_step_host)
  __half* stage_k;   // [I][D]
  __half* stage_v;   // [I][D]
  float* stage_out;  // [I*G][D]
  // prompt-phase workspace, for Iw = B * H * max_prefill_layers instances
  float* ws_m;       // [Iw*G][Sp]  row max of causal scores, per query head
  float* ws_invl;    // [Iw*G][Sp]  1 / row sum
  float* ws_acc;     // [Iw][Sp]    column sums
  int32_t* ws_slot;  // [Iw][Sp]    slot of a prompt token, -1 = evicted
  float* ws_hpart;   // [Iw][kMaxSplit][R*D + R]  partial H, z per token split
  float* ws_psi;     // [Iw][Sp][R]  psi(k_j) of every prompt token
  int32_t* ws_pmax;  // [Iw]        bit pattern of max psi over the instance's prompt tokens (scales the state build's fp16 operand)
  // parallel form only (LESS_WITH_PARALLEL_FORM); St = 128-row tiles of max_prompt
  float* ws_phi;     // [Iw * G][Sp][R]  phi(q_i) of every row of every query head
  unsigned char* ws_phiop;  // [Iw * G][St][8 KB]  phi as fp16 hi / lo operand tiles
  unsigned char* ws_psiop;  // [Iw][St][8 KB]  psi likewise
  float* ws_g;       // [Iw * G][St*128]  per row: log2 of (kernel value / value of the scaled operands)
  int32_t* ws_eu;    // [Iw][St*128]  exact_until, padded with zeros
  float* ws_ht;      // [Iw][St][R*D + R]  H, z of every key tile
  float* ws_hsum;    // [Iw][St][R*D + R]  per Q tile: H, z summed over the key tiles dead for it
  int32_t* ws_bucket; // [Iw][St]  first Q tile a key tile is dead for
  uint4* ws_bx;      // [Iw*G][Sbx]  per prompt row: -(m_i sqrt(D) - log2(1/l_i) / c) as three fp16 parts (column sums)
};

struct Dims {
  int32_t B, L, Hd, D, R, Rp;   // batch, layers, heads, head_dim, rank, hidden
  int32_t heavy, recent, N, Np; // slots; Np = N rounded up to a multiple of 4
  int32_t I;                    // instances (one per KV head)
  int32_t G;                    // query heads per KV head
  int32_t general;              // head_dim 64 or a group size other than 1, 2, 4, 8: the general CUDA-core decode path
  int32_t Sp;                   // max_prompt rounded up to a multiple of 4
  int32_t Sbx;                  // max_prompt rounded up to a multiple of 256 (+256)
  int32_t St;                   // 128-row tiles of max_prompt
  int32_t Lw;                   // max_prefill_layers
  uint32_t flags;
};

}  // namespace less

struct less_ctx {
  less_config cfg;
  less_weights w;
  less::Dims d;
  less::Arena a;
  void* arena_base;
  size_t arena_bytes;
  int64_t t;           // tokens seen
  int64_t launches;    // kernels launched
  int device;
  int sms;             // multiprocessors of the device
  bool pdl;            // decode kernel overlaps the feature-map kernel (off with LESS_NO_OVERLAP)
  int feature_stages;  // cap on the feature kernels' ring stages (LESS_FEATURE_STAGES), 0 = default
  int score_path;      // prompt scoring: 1 tensor cores, 0 CUDA cores (LESS_SCORE_KERNEL=plain)
  int feature_path;    // feature-map kernel: 2 tensor cores, 1 streaming GEMV, 0 plain (LESS_FEATURE_KERNEL)
  int small_step;      // the single-launch step for workloads of a few heads: -1 by size (default), 0 never, 1 whenever
                       // the shape allows (LESS_SMALL_STEP)
  bool small_step_ready[2];   // shared-memory opt-in of the small-step kernel done (direct / captured variant)
  int small_step_named;       // which variant's name is in `variant`, -1 = neither
  int group_path;      // grouped decode kernel: 2 on CUDA cores (LESS_GROUP_KERNEL=rows), else with warp-level mma
  int seg_l0, seg_nl;  // layers [seg_l0, seg_l0 + seg_nl) of the step being launched (the host entry launches a
                       // large step in layer segments so that its input copies overlap the kernels); default all
  cudaStream_t copy_stream;            // host entry: input copies of the later segments (created on first use)
  cudaEvent_t seg_event[8];            // host entry: "segment's inputs are in device memory"
  bool x_plain;        // set by the host entry around a step whose q, k are read in place from pinned host memory
  bool head_counters;  // decode CTAs follow the large-batch feature kernel head by head (LESS_HEAD_COUNTERS=1; off by default)
  int feature_ctas;    // cap on the feature kernels' persistent CTAs (LESS_FEATURE_CTAS), 0 = one per multiprocessor
  bool flags_this_step;     // the step's feature-map launch publishes per-head counters (set by its launcher)
  uint32_t flag_target[2];  // counter value of a head once this step's phi / psi are written
  int status_where;         // where-code of the last status word read by less_poll_status
  char variant[LESS_KERNEL_COUNT][64];   // name of the kernel variant last launched under each kernel id
  // tensor maps of the feature-map kernels, kept between steps (encoding four of them costs more host
  // time than a small step's launches): W1 of phi / psi (fixed), q / k rows (re-encoded when the
  // caller's pointers change)
  alignas(64) unsigned char tm_cache[4][128];
  const void* tm_q; const void* tm_k;
  int tm_box;          // rows per box of the cached q / k maps, 0 = none cached
  bool tm_w_ok;
  bool profile;                         // record an event pair around every launch
  std::vector<cudaEvent_t> prof_events; // start, stop, start, stop, ...
  std::vector<int> prof_kernel;         // kernel id of each pair
  std::vector<cudaEvent_t> prof_pool;   // events ready for reuse
};

namespace less {

// status word values written by kernels (first writer wins)
constexpr int kStatusOk = 0;
constexpr int kStatusTimeout = 1;
constexpr int kStatusBounds = 2;

__device__ __forceinline__ void set_status(int32_t* status, int code, int where) {
  if (atomicCAS(status, 0, code) == 0) status[1] = where;
}

// Programmatic dependent launch: the feature-map kernel lets the decode kernel of the same step
// start while it is still streaming weights; the decode kernel waits for the feature maps only
// where it first needs them.  Both are no-ops for a kernel launched without the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_primary() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Exact-form GELU, x * Phi(x), in about 11 instructions, without branches or selects:
//     Phi(-u) = E(u) / 2,  Phi(u) = 1 - E(u) / 2,  E(u) = erfc(u / sqrt(2)) = 2^(-u g(u))   (u = |x|)
//     =>  gelu(x) = max(x, 0) - u E(u) / 2          for both signs
// with g a degree-5 polynomial (coefficients and error from gelu_fit.py: the fp32 result is
// within 2.9e-7 of the exact value on [-12, 12], 2.1e-7 on [-3, 3], i.e. at its rounding error;
// both tails come straight out of the exponential).  The feature maps spend most of their
// arithmetic here: 512 + R evaluations per token and map.
__device__ __forceinline__ float gelu_erf(float x) {
  const float u = fminf(fabsf(x), 8.0f);
  float g = -3.155045488e-05f;
  g = fmaf(g, u, 7.533458411e-04f);
  g = fmaf(g, u, -8.018460125e-03f);
  g = fmaf(g, u, 5.329473317e-02f);
  g = fmaf(g, u, 4.588809609e-01f);
  g = fmaf(g, u, 1.151154518e+00f);
  float e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-g * u));   // 2 ulp; results below 2^-126 flush to 0
  return fmaf(-0.5f, u * e, fmaxf(x, 0.f));
}

// The same function for two values at once with Blackwell's packed fp32 arithmetic (fma / mul
// .f32x2: two results per issued instruction; bit-identical to gelu_erf, one rounding per
// operation either way).  The MLP epilogues are bound by instruction issue, not by the FMA lanes.
__device__ __forceinline__ uint64_t f32x2_pack(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void f32x2_unpack(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t f32x2_fma(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t f32x2_mul(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ void gelu_erf2(float x0, float x1, float& r0, float& r1) {
  const uint64_t u = f32x2_pack(fminf(fabsf(x0), 8.0f), fminf(fabsf(x1), 8.0f));
  uint64_t g = f32x2_pack(-3.155045488e-05f, -3.155045488e-05f);
  g = f32x2_fma(g, u, f32x2_pack(7.533458411e-04f, 7.533458411e-04f));
  g = f32x2_fma(g, u, f32x2_pack(-8.018460125e-03f, -8.018460125e-03f));
  g = f32x2_fma(g, u, f32x2_pack(5.329473317e-02f, 5.329473317e-02f));
  g = f32x2_fma(g, u, f32x2_pack(4.588809609e-01f, 4.588809609e-01f));
  g = f32x2_fma(g, u, f32x2_pack(1.151154518e+00f, 1.151154518e+00f));
  float t0, t1, e0, e1;
  f32x2_unpack(f32x2_mul(g, u), t0, t1);
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(-t0));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(-t1));
  f32x2_unpack(f32x2_fma(f32x2_pack(-0.5f, -0.5f), f32x2_mul(u, f32x2_pack(e0, e1)),
                         f32x2_pack(fmaxf(x0, 0.f), fmaxf(x1, 0.f))), r0, r1);
}

__device__ __forceinline__ void half8_to_float(const uint4& u, float* f) {
  const __half2* h = reinterpret_cast<const __half2*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 p = __half22float2(h[i]);
    f[2 * i] = p.x;
    f[2 * i + 1] = p.y;
  }
}

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  // 128-bit streaming load: K/V slots are read once per step
  return __ldcs(reinterpret_cast<const uint4*>(p));
}

__device__ __forceinline__ uint4 ldg_readonly(const void* p) {
  // 128-bit load through the read-only path (weights: never written by a kernel)
  return __ldg(reinterpret_cast<const uint4*>(p));
}

// Brackets one kernel launch with an event pair when profiling is on, and counts it.
struct LaunchScope {
  less_ctx* c;
  cudaStream_t s;
  bool on;
  LaunchScope(less_ctx* ctx, int kernel_id, cudaStream_t stream, const char* variant = nullptr)
      : c(ctx), s(stream), on(ctx->profile) {
    c->launches += 1;
    if (variant) snprintf(c->variant[kernel_id], sizeof c->variant[kernel_id], "%s", variant);
    if (!on) return;
    cudaEvent_t a = take(), b = take();
    c->prof_events.push_back(a);
    c->prof_events.push_back(b);
    c->prof_kernel.push_back(kernel_id);
    cudaEventRecord(a, s);
  }
  ~LaunchScope() {
    if (on) cudaEventRecord(c->prof_events.back(), s);
  }
  cudaEvent_t take() {
    cudaEvent_t e;
    if (!c->prof_pool.empty()) {
      e = c->prof_pool.back();
      c->prof_pool.pop_back();
    } else {
      cudaEventCreate(&e);
    }
    return e;
  }
};

// Host-side failure report: with LESS_LOG set in the environment, says on stderr which call
// failed and why; always returns LESS_ERR_CUDA.
int fail_cuda(const char* what, cudaError_t e = cudaSuccess);
// after a kernel launch: LESS_OK, or the report above for the launch error
inline int check_launch(const char* kernel) {
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? LESS_OK : fail_cuda(kernel, e);
}

// Whether the decode kernel is launched as a programmatic dependent of the feature-map kernel.
// When it waits for the feature kernel's whole grid this pays only while every decode CTA can be
// resident beside the feature-map CTAs: with more instances than that, the early CTAs sit on
// their SMs waiting and only take bandwidth and room from the weight stream (measured: 64 x 1024
// instances 1.54 -> 1.71 ms per step).  With per-head counters a decode CTA waits for its own
// head's feature maps only, and any number of instances can follow the feature kernel.
inline bool overlap_decode(const less_ctx* c) {
  return c->pdl && !c->profile && !(c->d.flags & LESS_NO_STATE) && (c->flags_this_step || c->d.I <= 8 * c->sms);
}

// launchers (host), defined in the kernel translation units
int launch_feature_maps(less_ctx* c, const void* q, const void* k, cudaStream_t s);
// whether a decode step of this context runs a tensor-core feature kernel, and the small-batch one (feature_tc.cu)
bool feature_tc_path(const less_ctx* c);
bool feature_small_tc_path(const less_ctx* c);
int launch_decode(less_ctx* c, const void* q, const void* k, const void* v, void* out,
                  int32_t* evicted_pos, cudaStream_t s);
// feature maps and decode step of a workload of a few heads in one launch (decode_kernels.cu)
bool small_step_path(const less_ctx* c);
int launch_small_step(less_ctx* c, const void* q, const void* k, const void* v, void* out, int32_t* evicted_pos,
                      cudaStream_t s);
int launch_prefill_group(less_ctx* c, int layer0, int nlayers, int lj0, int layer_count, int S,
                         const void* Q, const void* K, const void* V, void* attn_out,
                         cudaStream_t s);
// n state records between the arena and a device staging buffer (state_io.cu)
int launch_state_io(less_ctx* c, const int32_t* inst_dev, int n, void* records_dev, size_t rec_bytes, bool to_records,
                    cudaStream_t s);
// the parallel form of one layer group (masked_tc.cu)
int launch_masked_form(less_ctx* c, int layer0, int nlayers, int lj0, int layer_count, int S, const void* Q,
                       const void* K, const void* V, const int32_t* exact_until, void* out, cudaStream_t s);

}  // namespace less
