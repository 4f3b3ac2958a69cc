// Host side of the C ABI: config validation, arena carving, state export /
// import, status polling.  No device memory is allocated here.
#include <algorithm>
#include <new>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "less_internal.cuh"

using namespace less;

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// head dimension 64, or a number of query heads per KV head other than 1, 2, 4, 8: the general path
bool general_shape(const less_config* c) {
  const int g = c->group > 1 ? c->group : 1;
  return c->head_dim != kHeadDim || !(g == 1 || g == 2 || g == 4 || g == 8);
}

bool valid_config(const less_config* c) {
  if (!c) return false;
  if (c->batch < 1 || c->layers < 1 || c->heads < 1) return false;
  if (c->head_dim != kHeadDim && c->head_dim != 64) return false;
  if (c->rank != 8 && c->rank != 16) return false;
  if (c->hidden < 64 || c->hidden > 1024 || (c->hidden & (c->hidden - 1))) return false;
  if (c->heavy < 0 || c->recent < 1) return false;
  if ((int64_t)c->heavy + c->recent > LESS_MAX_SLOTS) return false;   // the decode kernel keeps one score per slot in shared memory
  if (c->max_prompt < 0 || c->max_prompt > (1 << 20)) return false;
  if (c->max_prefill_layers < 1 || c->max_prefill_layers > c->layers) return false;
  if ((int64_t)c->batch * c->heads * c->max_prefill_layers * (c->group > 1 ? c->group : 1) > 65535)
    return false;                                                                   // grid.y of the prompt kernels
  if (c->flags & ~(uint32_t)(LESS_SCORE_NORM_SPARSE | LESS_NO_STATE | LESS_POLICY_LAMBDA | LESS_POLICY_TOVA | LESS_WITH_PARALLEL_FORM | LESS_OUT_F16)) return false;
  if ((c->flags & LESS_POLICY_LAMBDA) && (c->flags & LESS_POLICY_TOVA)) return false;
  if (c->group < 0 || c->group > 128) return false;
  if (c->group > 1 && (c->flags & LESS_POLICY_TOVA)) return false;                         // TOVA stays per head
  if (general_shape(c)) {
    // decode only, on CUDA cores: eight heads' scores plus the aggregated ones per slot in shared memory
    if (c->flags & LESS_WITH_PARALLEL_FORM) return false;
    if ((int64_t)9 * ((((int64_t)c->heavy + c->recent + 3) & ~3) + 4 + 1024) * 4 > 227 * 1024) return false;
  } else {
    // the decode kernel keeps one score per slot and query head in shared memory (227 KB per CTA)
    if (c->group > 1 && (int64_t)c->group * ((((int64_t)c->heavy + c->recent + 3) & ~3) + 4 + 1024) * 4 > 227 * 1024)
      return false;
    if (c->group > 1 && c->hidden != 128 && c->hidden != 256 && c->hidden != 512) return false;   // tensor-core feature maps only
  }
  int64_t inst = (int64_t)c->batch * c->layers * c->heads;
  if (inst > (1 << 24)) return false;
  return true;
}

Dims make_dims(const less_config* c) {
  Dims d;
  d.B = c->batch;
  d.L = c->layers;
  d.Hd = c->heads;
  d.D = c->head_dim;
  d.R = c->rank;
  d.Rp = c->hidden;
  d.heavy = c->heavy;
  d.recent = c->recent;
  d.N = c->heavy + c->recent;
  d.Np = (d.N + 3) & ~3;
  d.I = c->batch * c->layers * c->heads;
  d.G = c->group > 1 ? c->group : 1;
  d.general = general_shape(c) ? 1 : 0;
  d.Sp = (c->max_prompt + 3) & ~3;
  d.Sbx = ((c->max_prompt + 255) & ~255) + 256;
  d.St = (c->max_prompt + 127) / 128;
  d.Lw = c->max_prefill_layers;
  d.flags = c->flags;
  return d;
}

// Walks the arena layout; with base == nullptr only the total size is computed.
size_t carve(const Dims& d, char* base, Arena* a) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    char* p = base ? base + off : nullptr;
    off = align_up(off + bytes, 256);
    return p;
  };
  const size_t I = d.I, N = d.N, Np = d.Np, D = d.D, R = d.R;
  const size_t Iw = (size_t)d.B * d.Hd * d.Lw, Sp = d.Sp, G = d.G;
  Arena t;
  t.kslots = (__half*)take(I * N * D * sizeof(__half));
  t.vslots = (__half*)take(I * N * D * sizeof(__half));
  t.pos = (int32_t*)take(I * Np * 4);
  t.acc = (float*)take(I * Np * 4);
  t.psic = (float*)take(I * N * R * 4);
  t.H = (float*)take(I * R * D * 4);
  t.z = (float*)take(I * R * 4);
  t.count = (int32_t*)take(I * 4);
  t.phi_q = (float*)take(I * G * R * 4);
  t.psi_k = (float*)take(I * R * 4);
  t.status = (int32_t*)take(4 * 4);
  t.tpos = (int32_t*)take(4 * 4);
  t.feat_flag = (uint32_t*)take((size_t)d.L * d.Hd * (G + 1) * 4);
  t.stage_q = (__half*)take(I * G * D * 2);
  t.stage_k = (__half*)take(I * D * 2);
  t.stage_v = (__half*)take(I * D * 2);
  t.stage_out = (float*)take(I * G * D * 4);
  t.ws_m = (float*)take(Iw * G * Sp * 4);
  t.ws_invl = (float*)take(Iw * G * Sp * 4);
  t.ws_acc = (float*)take(Iw * Sp * 4);
  t.ws_slot = (int32_t*)take(Iw * Sp * 4);
  t.ws_hpart = (float*)take(Iw * kMaxSplit * (R * D + R) * 4);
  t.ws_psi = (float*)take(Iw * Sp * R * 4);
  t.ws_bx = (uint4*)take(Iw * G * (size_t)d.Sbx * 16);
  t.ws_pmax = (int32_t*)take(Iw * 4);
  const size_t St = (d.flags & LESS_WITH_PARALLEL_FORM) ? d.St : 0;
  t.ws_phi = (float*)take(St ? Iw * G * Sp * R * 4 : 0);      // the query side of the parallel form: per query head
  t.ws_phiop = (unsigned char*)take(Iw * G * St * 8192);
  t.ws_psiop = (unsigned char*)take(Iw * St * 8192);
  t.ws_g = (float*)take(Iw * G * St * 128 * 4);
  t.ws_eu = (int32_t*)take(Iw * St * 128 * 4);
  t.ws_ht = (float*)take(Iw * St * (R * D + R) * 4);
  t.ws_hsum = (float*)take(Iw * St * (R * D + R) * 4);
  t.ws_bucket = (int32_t*)take(Iw * St * 4);
  if (a) *a = t;
  return off;
}

inline bool misaligned(const void* p) { return ((uintptr_t)p & 15) != 0; }

struct RecordLayout {
  size_t pos, acc, K, V, psi, H, z, total;
};

RecordLayout record_layout(const Dims& d) {
  RecordLayout r;
  size_t off = 16;
  r.pos = off; off += (size_t)d.N * 4;
  r.acc = off; off += (size_t)d.N * 4;
  r.K = off; off += (size_t)d.N * d.D * 2;
  r.V = off; off += (size_t)d.N * d.D * 2;
  r.psi = off; off += (size_t)d.N * d.R * 4;
  r.H = off; off += (size_t)d.R * d.D * 4;
  r.z = off; off += (size_t)d.R * 4;
  r.total = off;
  return r;
}

}  // namespace

namespace less {
int fail_cuda(const char* what, cudaError_t e) {
  if (getenv("LESS_LOG")) {
    if (e == cudaSuccess) e = cudaPeekAtLastError();
    fprintf(stderr, "[less] %s failed: %s\n", what, e == cudaSuccess ? "(no CUDA error recorded)" : cudaGetErrorString(e));
  }
  return LESS_ERR_CUDA;
}
}  // namespace less

extern "C" {

size_t less_arena_bytes(const less_config* cfg) {
  if (!valid_config(cfg)) return 0;
  Dims d = make_dims(cfg);
  return carve(d, nullptr, nullptr);
}

size_t less_state_record_bytes(const less_config* cfg) {
  if (!valid_config(cfg)) return 0;
  return record_layout(make_dims(cfg)).total;
}

int less_create(const less_config* cfg, const less_weights* w, void* arena, size_t arena_bytes,
                less_ctx** out) {
  if (!cfg || !w || !arena || !out) return LESS_ERR_NULL_POINTER;
  if (!valid_config(cfg)) return LESS_ERR_INVALID_CONFIG;
  if (!w->w_phi1 || !w->w_phi2 || !w->w_psi1 || !w->w_psi2 || !w->w_psi3)
    return LESS_ERR_NULL_POINTER;
  if (misaligned(w->w_phi1) || misaligned(w->w_phi2) || misaligned(w->w_psi1) ||
      misaligned(w->w_psi2) || misaligned(w->w_psi3) || ((uintptr_t)arena & 255))
    return LESS_ERR_MISALIGNED;
  Dims d = make_dims(cfg);
  size_t need = carve(d, nullptr, nullptr);
  if (arena_bytes < need) return LESS_ERR_ARENA_TOO_SMALL;
  less_ctx* c = new (std::nothrow) less_ctx;
  if (!c) return LESS_ERR_CUDA;
  c->cfg = *cfg;
  c->w = *w;
  c->d = d;
  carve(d, (char*)arena, &c->a);
  c->arena_base = arena;
  c->arena_bytes = need;
  c->t = 0;
  c->launches = 0;
  c->flags_this_step = false;
  c->flag_target[0] = c->flag_target[1] = 0;
  c->status_where = 0;
  c->tm_q = c->tm_k = nullptr;
  c->tm_box = 0;
  c->tm_w_ok = false;
  memset(c->variant, 0, sizeof c->variant);
  c->feature_ctas = 0;
  c->head_counters = getenv("LESS_HEAD_COUNTERS") != nullptr;
  c->x_plain = false;
  c->seg_l0 = 0; c->seg_nl = d.L;
  c->copy_stream = nullptr;
  for (cudaEvent_t& ev : c->seg_event) ev = nullptr;
  if (const char* e = getenv("LESS_FEATURE_CTAS")) c->feature_ctas = atoi(e);
  c->profile = false;
  c->feature_path = 2;
  c->pdl = getenv("LESS_NO_OVERLAP") == nullptr;
  c->score_path = 1;
  if (const char* e = getenv("LESS_SCORE_KERNEL"))
    if (!strcmp(e, "plain")) c->score_path = 0;
  c->feature_stages = 0;
  if (const char* e = getenv("LESS_FEATURE_STAGES")) c->feature_stages = atoi(e);
  if (const char* e = getenv("LESS_FEATURE_KERNEL")) {
    if (!strcmp(e, "gemv")) c->feature_path = 1;
    else if (!strcmp(e, "plain")) c->feature_path = 0;
  }
  if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; return LESS_ERR_CUDA; }
  c->small_step = -1;
  c->small_step_ready[0] = c->small_step_ready[1] = false;
  c->small_step_named = -1;
  if (const char* e = getenv("LESS_SMALL_STEP")) c->small_step = !strcmp(e, "0") ? 0 : (!strcmp(e, "1") ? 1 : -1);
  c->group_path = 3;
  if (const char* e = getenv("LESS_GROUP_KERNEL"))
    if (!strcmp(e, "rows")) c->group_path = 2;
  c->sms = 148;
  cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, c->device);
  int cluster_launch = 0;                               // e.g. off under some partitioning modes: then the step stays two kernels
  if (cudaDeviceGetAttribute(&cluster_launch, cudaDevAttrClusterLaunch, c->device) != cudaSuccess || !cluster_launch)
    c->small_step = 0;
  // H_0 = 0, z_0 = 0, no live slots, clean status
  cudaError_t e = cudaMemset(c->a.H, 0, (size_t)d.I * d.R * d.D * 4);
  if (e == cudaSuccess) e = cudaMemset(c->a.z, 0, (size_t)d.I * d.R * 4);
  if (e == cudaSuccess) e = cudaMemset(c->a.count, 0, (size_t)d.I * 4);
  if (e == cudaSuccess) e = cudaMemset(c->a.status, 0, 16);
  if (e == cudaSuccess) e = cudaMemset(c->a.tpos, 0, 16);
  if (e == cudaSuccess) e = cudaMemset(c->a.feat_flag, 0, (size_t)d.L * d.Hd * (d.G + 1) * 4);
  if (e == cudaSuccess) e = cudaMemset(c->a.phi_q, 0, (size_t)d.I * d.G * d.R * 4);
  if (e == cudaSuccess) e = cudaMemset(c->a.psi_k, 0, (size_t)d.I * d.R * 4);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { delete c; return LESS_ERR_CUDA; }
  *out = c;
  return LESS_OK;
}

int less_destroy(less_ctx* ctx) {
  if (!ctx) return LESS_ERR_NULL_POINTER;
  for (cudaEvent_t e : ctx->prof_events) cudaEventDestroy(e);
  for (cudaEvent_t e : ctx->prof_pool) cudaEventDestroy(e);
  for (cudaEvent_t e : ctx->seg_event) if (e) cudaEventDestroy(e);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  delete ctx;
  return LESS_OK;
}

int64_t less_position(const less_ctx* ctx) { return ctx ? ctx->t : -1; }
const char* less_kernel_variant(const less_ctx* ctx, int kernel_id) {
  if (!ctx || kernel_id < 0 || kernel_id >= LESS_KERNEL_COUNT) return "";
  return ctx->variant[kernel_id];
}
int less_last_status_where(const less_ctx* ctx) { return ctx ? ctx->status_where : 0; }
int64_t less_launch_count(const less_ctx* ctx) { return ctx ? ctx->launches : -1; }

int less_prefill(less_ctx* c, int32_t layer_begin, int32_t layer_count, int32_t prompt_len,
                 const void* Q, const void* K, const void* V, void* attn_out, void* stream) {
  if (!c) return LESS_ERR_NULL_POINTER;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > c->d.L)
    return LESS_ERR_BAD_LAYER_RANGE;
  if (prompt_len < 0) return LESS_ERR_INVALID_CONFIG;
  if (prompt_len > c->cfg.max_prompt) return LESS_ERR_PROMPT_TOO_LONG;
  if (prompt_len > 0) {
    // the tiled loads address prompt rows with 32-bit coordinates
    if ((int64_t)c->d.B * layer_count * c->d.Hd * c->d.G * prompt_len > 0x7fffffffLL) return LESS_ERR_PROMPT_TOO_LONG;
    if (!Q || !K || !V) return LESS_ERR_NULL_POINTER;
    if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(attn_out))
      return LESS_ERR_MISALIGNED;
  }
  cudaStream_t s = (cudaStream_t)stream;
  for (int lj0 = 0; lj0 < layer_count; lj0 += c->d.Lw) {
    int nl = layer_count - lj0 < c->d.Lw ? layer_count - lj0 : c->d.Lw;
    int rc = launch_prefill_group(c, layer_begin + lj0, nl, lj0, layer_count, prompt_len, Q, K, V,
                                  attn_out, s);
    if (rc != LESS_OK) return rc;
  }
  c->t = prompt_len;
  return LESS_OK;
}

int less_masked_attention(less_ctx* c, int32_t layer_begin, int32_t layer_count, int32_t seq_len,
                          const void* Q, const void* K, const void* V, const int32_t* exact_until,
                          void* out, void* stream) {
  if (!c) return LESS_ERR_NULL_POINTER;
  if (!(c->d.flags & LESS_WITH_PARALLEL_FORM) || c->d.general) return LESS_ERR_INVALID_CONFIG;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > c->d.L)
    return LESS_ERR_BAD_LAYER_RANGE;
  if (seq_len < 0) return LESS_ERR_INVALID_CONFIG;
  if (seq_len > c->cfg.max_prompt) return LESS_ERR_PROMPT_TOO_LONG;
  if (seq_len == 0) return LESS_OK;
  if ((int64_t)c->d.B * layer_count * c->d.Hd * c->d.G * seq_len > 0x7fffffffLL) return LESS_ERR_PROMPT_TOO_LONG;
  if (!Q || !K || !V || !exact_until || !out) return LESS_ERR_NULL_POINTER;
  if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(out) || ((uintptr_t)exact_until & 3))
    return LESS_ERR_MISALIGNED;
  cudaStream_t s = (cudaStream_t)stream;
  for (int lj0 = 0; lj0 < layer_count; lj0 += c->d.Lw) {
    int nl = layer_count - lj0 < c->d.Lw ? layer_count - lj0 : c->d.Lw;
    int rc = launch_masked_form(c, layer_begin + lj0, nl, lj0, layer_count, seq_len, Q, K, V, exact_until, out, s);
    if (rc != LESS_OK) return rc;
  }
  return LESS_OK;
}

int less_decode_step(less_ctx* c, const void* q, const void* k, const void* v, void* out,
                     int32_t* evicted_pos, void* stream) {
  if (!c || !q || !k || !v || !out) return LESS_ERR_NULL_POINTER;
  if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(out))
    return LESS_ERR_MISALIGNED;
  if (c->t >= 0x7fffff00) return LESS_ERR_BAD_STATE;
  cudaStream_t s = (cudaStream_t)stream;
  if (small_step_path(c)) {
    const int rc1 = launch_small_step(c, q, k, v, out, evicted_pos, s);
    if (rc1 == LESS_OK) c->t += 1;
    return rc1;
  }
  int rc = launch_feature_maps(c, q, k, s);
  if (rc != LESS_OK) return rc;
  rc = launch_decode(c, q, k, v, out, evicted_pos, s);
  if (rc != LESS_OK) return rc;
  c->t += 1;
  return LESS_OK;
}

// The host entry's large steps: the layers in kSegments ranges, each range's q, k copied on a stream
// of its own and its two kernels launched behind the copy, so that all copies but the first run
// under the kernels of the range before.
static constexpr int kSegments = 4;

static int staged_step_in_segments(less_ctx* c, const void* qh, const void* kh, const void* v_dev, void* out_dev,
                                   cudaStream_t s) {
  const Dims& d = c->d;
  if (!c->copy_stream) {
    if (cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return fail_cuda("copy stream");
    for (int i = 0; i < 2 * kSegments; ++i)
      if (cudaEventCreateWithFlags(&c->seg_event[i], cudaEventDisableTiming) != cudaSuccess) return fail_cuda("segment events");
  }
  // the copies may start once the caller's stream has reached this call
  if (cudaEventRecord(c->seg_event[kSegments], s) != cudaSuccess ||
      cudaStreamWaitEvent(c->copy_stream, c->seg_event[kSegments], 0) != cudaSuccess)
    return fail_cuda("segment ordering");
  const size_t rowq = (size_t)d.Hd * d.G * d.D * 2, rowk = (size_t)d.Hd * d.D * 2;   // bytes of one layer of one batch row
  int l0[kSegments + 1];
  for (int i = 0; i <= kSegments; ++i) l0[i] = (int)((long long)d.L * i / kSegments);
  for (int i = 0; i < kSegments; ++i) {
    const int nl = l0[i + 1] - l0[i];
    if (cudaMemcpy2DAsync((char*)c->a.stage_q + l0[i] * rowq, d.L * rowq, (const char*)qh + l0[i] * rowq, d.L * rowq,
                          nl * rowq, d.B, cudaMemcpyHostToDevice, c->copy_stream) != cudaSuccess ||
        cudaMemcpy2DAsync((char*)c->a.stage_k + l0[i] * rowk, d.L * rowk, (const char*)kh + l0[i] * rowk, d.L * rowk,
                          nl * rowk, d.B, cudaMemcpyHostToDevice, c->copy_stream) != cudaSuccess ||
        cudaEventRecord(c->seg_event[i], c->copy_stream) != cudaSuccess)
      return fail_cuda("segment copy");
  }
  int rc = LESS_OK;
  for (int i = 0; i < kSegments && rc == LESS_OK; ++i) {
    if (cudaStreamWaitEvent(s, c->seg_event[i], 0) != cudaSuccess) return fail_cuda("segment wait");
    c->seg_l0 = l0[i];
    c->seg_nl = l0[i + 1] - l0[i];
    rc = launch_feature_maps(c, c->a.stage_q, c->a.stage_k, s);
    if (rc == LESS_OK) rc = launch_decode(c, c->a.stage_q, c->a.stage_k, v_dev, out_dev, nullptr, s);
  }
  c->seg_l0 = 0;
  c->seg_nl = d.L;
  if (rc == LESS_OK) c->t += 1;
  return rc;
}

// Device-visible alias of a host buffer: pinned (page-locked, mapped) memory can be read and
// written by kernels directly over PCIe; pageable memory cannot (nullptr).
static void* device_alias(const void* host) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
    cudaGetLastError();                       // not a CUDA-known pointer: clear the error, use the staging path
    return nullptr;
  }
  return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

int less_decode_step_host(less_ctx* c, const void* qh, const void* kh, const void* vh, void* outh,
                          void* stream) {
  if (!c || !qh || !kh || !vh || !outh) return LESS_ERR_NULL_POINTER;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t osz = (c->d.flags & LESS_OUT_F16) ? 2 : 4;
  const size_t nin = (size_t)c->d.I * c->d.D * 2, nq = nin * c->d.G, nout = (size_t)c->d.I * c->d.G * c->d.D * osz;
  // v and the output are touched once per instance by the decode kernel: from pinned host memory
  // it reads / writes them in place.  q and k feed the feature-map kernel: with more than 8 batch rows
  // its TMA loads want them in device memory and they are staged in the arena (the two staging
  // buffers are neighbours, so a caller that keeps k directly behind q pays one copy, not two).
  const void* v_dev = device_alias(vh);
  void* out_dev = device_alias(outh);
  if (((uintptr_t)v_dev & 15) || ((uintptr_t)out_dev & 15)) { v_dev = nullptr; out_dev = nullptr; }
  cudaError_t e = cudaSuccess;
  // With a small batch the feature-map kernel can fetch its q, k rows with plain loads: from pinned
  // host memory they are then read in place too (by both kernels), and the step has no copy in front
  // of it - the rows cross PCIe while the weights stream.
  const void* q_dev = device_alias(qh);
  const void* k_dev = device_alias(kh);
  const bool qk_in_place = q_dev && k_dev && !((uintptr_t)q_dev & 15) && !((uintptr_t)k_dev & 15) &&
                           (feature_small_tc_path(c) || small_step_path(c) || (c->d.flags & LESS_NO_STATE));
  // a large staged step: its layers in segments, the copies under the kernels
  if (!qk_in_place && v_dev && out_dev && feature_tc_path(c) && !c->head_counters && c->d.L >= kSegments &&
      nq + nin >= ((size_t)4 << 20) && c->t < 0x7fffff00) {
    const int rc = staged_step_in_segments(c, qh, kh, v_dev, out_dev, s);
    if (rc != LESS_OK) return rc;
    return cudaStreamSynchronize(s) == cudaSuccess ? LESS_OK : LESS_ERR_CUDA;
  }
  if (!qk_in_place) {
    bool copied = false;
    if ((const char*)kh == (const char*)qh + nq && (char*)c->a.stage_k == (char*)c->a.stage_q + nq) {
      // k directly behind q.  If the two are separate host allocations that merely touch, the runtime
      // refuses the copy that spans them (nothing is enqueued): then they go one by one.
      copied = cudaMemcpyAsync(c->a.stage_q, qh, nq + nin, cudaMemcpyHostToDevice, s) == cudaSuccess;
      if (!copied) cudaGetLastError();
    }
    if (!copied) {
      e = cudaMemcpyAsync(c->a.stage_q, qh, nq, cudaMemcpyHostToDevice, s);
      if (e == cudaSuccess) e = cudaMemcpyAsync(c->a.stage_k, kh, nin, cudaMemcpyHostToDevice, s);
    }
  }
  if (e == cudaSuccess && !v_dev) e = cudaMemcpyAsync(c->a.stage_v, vh, nin, cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return LESS_ERR_CUDA;
  c->x_plain = qk_in_place;
  int rc = less_decode_step(c, qk_in_place ? q_dev : c->a.stage_q, qk_in_place ? k_dev : c->a.stage_k,
                            v_dev ? v_dev : c->a.stage_v, out_dev ? out_dev : c->a.stage_out, nullptr, s);
  c->x_plain = false;
  if (rc != LESS_OK) return rc;
  if (!out_dev) e = cudaMemcpyAsync(outh, c->a.stage_out, nout, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  return e == cudaSuccess ? LESS_OK : LESS_ERR_CUDA;
}

int less_profile(less_ctx* c, int enable) {
  if (!c) return LESS_ERR_NULL_POINTER;
  for (cudaEvent_t e : c->prof_events) c->prof_pool.push_back(e);
  c->prof_events.clear();
  c->prof_kernel.clear();
  c->profile = enable != 0;
  return LESS_OK;
}

int less_profile_read(less_ctx* c, float* ms_total, int64_t* launches) {
  if (!c || !ms_total || !launches) return LESS_ERR_NULL_POINTER;
  for (int i = 0; i < LESS_KERNEL_COUNT; ++i) { ms_total[i] = 0.f; launches[i] = 0; }
  for (size_t i = 0; i < c->prof_kernel.size(); ++i) {
    cudaEvent_t a = c->prof_events[2 * i], b = c->prof_events[2 * i + 1];
    if (cudaEventSynchronize(b) != cudaSuccess) return LESS_ERR_CUDA;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, a, b) != cudaSuccess) return LESS_ERR_CUDA;
    const int k = c->prof_kernel[i];
    if (k >= 0 && k < LESS_KERNEL_COUNT) { ms_total[k] += ms; launches[k] += 1; }
  }
  return LESS_OK;
}

static int copy_state(less_ctx* c, const int32_t* inst, int32_t n, void* host, size_t bytes,
                      cudaStream_t s, bool to_host) {
  if (!c || !inst || !host) return LESS_ERR_NULL_POINTER;
  if (n < 0) return LESS_ERR_INVALID_CONFIG;
  const Dims& d = c->d;
  RecordLayout r = record_layout(d);
  if (bytes < r.total * (size_t)n) return LESS_ERR_BUFFER_TOO_SMALL;
  cudaMemcpyKind kind = to_host ? cudaMemcpyDeviceToHost : cudaMemcpyHostToDevice;
  cudaError_t e = cudaSuccess;
  auto cp = [&](void* hostp, void* devp, size_t nbytes) {
    if (e != cudaSuccess || nbytes == 0) return;
    e = to_host ? cudaMemcpyAsync(hostp, devp, nbytes, kind, s)
                : cudaMemcpyAsync(devp, hostp, nbytes, kind, s);
  };
  for (int i = 0; i < n; ++i)
    if (inst[i] < 0 || inst[i] >= d.I) return LESS_ERR_INVALID_CONFIG;
  // Records are packed / unpacked on the device, a batch at a time, in the host entry's staging
  // buffers (free between calls): the instance list in stage_q, the records in stage_out; the host
  // then sees one copy per batch.  Contexts whose staging buffer is smaller than one record (a handful
  // of instances with many slots) copy field by field.
  const size_t stage_bytes = (size_t)d.I * d.G * d.D * 4, list_cap = (size_t)d.I * d.G * d.D * 2 / 4;
  const size_t per_batch = std::min(stage_bytes / r.total, list_cap);
  if (per_batch >= 1 && r.total % 4 == 0) {
    for (size_t i0 = 0; i0 < (size_t)n && e == cudaSuccess; i0 += per_batch) {
      const int nb = (int)std::min(per_batch, (size_t)n - i0);
      char* rec = (char*)host + r.total * i0;
      e = cudaMemcpyAsync(c->a.stage_q, inst + i0, (size_t)nb * 4, cudaMemcpyHostToDevice, s);
      if (e == cudaSuccess && !to_host) e = cudaMemcpyAsync(c->a.stage_out, rec, r.total * nb, cudaMemcpyHostToDevice, s);
      if (e == cudaSuccess && launch_state_io(c, (const int32_t*)c->a.stage_q, nb, c->a.stage_out, r.total, to_host, s) != LESS_OK)
        return LESS_ERR_CUDA;
      if (e == cudaSuccess && to_host) e = cudaMemcpyAsync(rec, c->a.stage_out, r.total * nb, cudaMemcpyDeviceToHost, s);
      // the staging buffers are reused by the next batch
      if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    }
  } else {
    for (int i = 0; i < n; ++i) {
      char* rec = (char*)host + r.total * (size_t)i;
      size_t I = inst[i];
      cp(rec, c->a.count + I, 4);
      cp(rec + r.pos, c->a.pos + I * d.Np, (size_t)d.N * 4);
      cp(rec + r.acc, c->a.acc + I * d.Np, (size_t)d.N * 4);
      cp(rec + r.K, c->a.kslots + I * d.N * d.D, (size_t)d.N * d.D * 2);
      cp(rec + r.V, c->a.vslots + I * d.N * d.D, (size_t)d.N * d.D * 2);
      cp(rec + r.psi, c->a.psic + I * d.N * d.R, (size_t)d.N * d.R * 4);
      cp(rec + r.H, c->a.H + I * d.R * d.D, (size_t)d.R * d.D * 4);
      cp(rec + r.z, c->a.z + I * d.R, (size_t)d.R * 4);
    }
  }
  // the position lives on the device (a captured step advances it without the host); the host
  // keeps a copy for less_position
  int32_t tdev = 0;
  if (to_host) {
    if (e == cudaSuccess) e = cudaMemcpyAsync(&tdev, c->a.tpos, 4, cudaMemcpyDeviceToHost, s);
  } else if (n > 0) {
    tdev = ((const int32_t*)host)[1];
    if (e == cudaSuccess) e = cudaMemcpyAsync(c->a.tpos, &tdev, 4, cudaMemcpyHostToDevice, s);
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return LESS_ERR_CUDA;
  if (to_host) {
    c->t = tdev;
    for (int i = 0; i < n; ++i) {
      int32_t* hdr = (int32_t*)((char*)host + r.total * (size_t)i);
      hdr[1] = tdev;
      hdr[2] = hdr[3] = 0;
    }
  } else if (n > 0) {
    c->t = tdev;
  }
  return LESS_OK;
}

int less_export_state(less_ctx* c, const int32_t* inst, int32_t n, void* host, size_t bytes,
                      void* stream) {
  return copy_state(c, inst, n, host, bytes, (cudaStream_t)stream, true);
}

int less_import_state(less_ctx* c, const int32_t* inst, int32_t n, const void* host, size_t bytes,
                      void* stream) {
  if (c && host) {
    // the count field must be sane before it reaches a kernel
    RecordLayout r = record_layout(c->d);
    if (bytes < r.total * (size_t)(n < 0 ? 0 : n)) return LESS_ERR_BUFFER_TOO_SMALL;
    for (int i = 0; i < n; ++i) {
      int32_t cnt = *(const int32_t*)((const char*)host + r.total * (size_t)i);
      if (cnt < 0 || cnt > c->d.N) return LESS_ERR_BAD_STATE;
    }
  }
  return copy_state(c, inst, n, const_cast<void*>(host), bytes, (cudaStream_t)stream, false);
}

int less_read_feature_maps(less_ctx* c, float* phi_host, float* psi_host, void* stream) {
  if (!c) return LESS_ERR_NULL_POINTER;
  cudaStream_t s = (cudaStream_t)stream;
  size_t bytes = (size_t)c->d.I * c->d.R * 4;
  cudaError_t e = cudaSuccess;
  if (phi_host) e = cudaMemcpyAsync(phi_host, c->a.phi_q, bytes * c->d.G, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess && psi_host)
    e = cudaMemcpyAsync(psi_host, c->a.psi_k, bytes, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  return e == cudaSuccess ? LESS_OK : LESS_ERR_CUDA;
}

int less_poll_status(less_ctx* c, void* stream) {
  if (!c) return LESS_ERR_NULL_POINTER;
  int32_t st[4] = {0, 0, 0, 0};
  cudaStream_t s = (cudaStream_t)stream;
  int32_t tdev = 0;
  cudaError_t e = cudaMemcpyAsync(st, c->a.status, 16, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(&tdev, c->a.tpos, 4, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return LESS_ERR_CUDA;
  c->t = tdev;                                   // replays of a captured step advance only the device's count
  c->status_where = st[1];
  if (st[0] == kStatusTimeout) return LESS_ERR_DEVICE_TIMEOUT;
  if (st[0] == kStatusBounds) return LESS_ERR_DEVICE_BOUNDS;
  return LESS_OK;
}

const char* less_strerror(int code) {
  switch (code) {
    case LESS_OK: return "ok";
    case LESS_ERR_INVALID_CONFIG: return "invalid configuration or argument";
    case LESS_ERR_NULL_POINTER: return "null pointer";
    case LESS_ERR_MISALIGNED: return "pointer not 16-byte aligned (arena: 256)";
    case LESS_ERR_ARENA_TOO_SMALL: return "arena too small";
    case LESS_ERR_PROMPT_TOO_LONG: return "prompt longer than max_prompt";
    case LESS_ERR_BAD_LAYER_RANGE: return "layer range outside the model";
    case LESS_ERR_DEVICE_TIMEOUT: return "a device-side wait ran out";
    case LESS_ERR_DEVICE_BOUNDS: return "a device-side index check failed";
    case LESS_ERR_CUDA: return "CUDA runtime error";
    case LESS_ERR_BAD_STATE: return "state record or context state not usable";
    case LESS_ERR_BUFFER_TOO_SMALL: return "host buffer too small";
    case LESS_ERR_NOALLOC_TOO_LARGE: return "more rows than the built-in scratch array holds";
    default: return "unknown error";
  }
}

}  // extern "C"
