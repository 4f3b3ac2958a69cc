/*
 * less.h -- C ABI of the B200 (sm_100a) LESS hot path.
 *
 * LESS ("Get More with LESS", arxiv 2402.09398) pairs an eviction-based sparse
 * KV cache (here H2O: heavy hitters + recent window) with a constant-size
 * low-rank state (H, z) that absorbs every evicted key/value pair, so that
 * evicted tokens still contribute to later attention outputs.
 *
 * One "instance" is one (batch, layer, head); instances are independent.
 * Flat instance index: inst = (b * layers + layer) * heads + head, the order of
 * every [B, L, H, ...] buffer below.
 *
 * Conventions
 *   - Every function returns 0 (LESS_OK) or a negative LESS_ERR_* code; nothing
 *     throws or aborts across this boundary.
 *   - Pointers named in a signature as "device" are CUDA device pointers of the
 *     current device, 16-byte aligned; "host" are ordinary host pointers.
 *   - The library allocates no device memory: the caller provides one arena
 *     (less_arena_bytes) that the context carves up and owns until destroy.
 *   - Weight buffers and the arena are BORROWED for the context's lifetime.
 *     The weights must not change while the context exists: a decode step may fetch them before the work
 *     enqueued ahead of it on its stream has finished (its kernels are programmatic dependent launches; everything
 *     else a step reads - its inputs, the arena - it reads only once that work is complete).
 *   - less_prefill / less_decode_step are asynchronous on the given stream;
 *     their inputs must stay valid until the stream reaches the call.
 *   - A context is not thread-safe.
 *   - 16-bit inputs are IEEE fp16; accumulation, scores, H, z and outputs fp32.
 *   - D below is less_config.head_dim.
 *   - Environment, read by less_create: LESS_LOG (explain host-side failures on
 *     stderr), LESS_FEATURE_KERNEL=gemv|plain (CUDA-core feature-map kernels),
 *     LESS_NO_OVERLAP (no programmatic dependent launches: neither the decode kernel behind its step's
 *     feature-map kernel nor a step's first kernel behind the kernel before it in the stream),
 *     LESS_SCORE_KERNEL=plain (CUDA-core prompt scoring),
 *     LESS_FEATURE_STAGES=n (cap on the feature kernels' weight ring),
 *     LESS_GROUP_KERNEL=rows (grouped query heads: the CUDA-core decode kernel instead of
 *     the one with its two contractions as warp-level tensor-core products),
 *     LESS_FEATURE_CTAS=n (cap on the persistent CTAs of the tensor-core feature kernels),
 *     LESS_HEAD_COUNTERS=1 (with more instances than fit the GPU at once and more than 8 batch rows:
 *     the decode kernel starts behind the feature-map kernel and each of its CTAs waits for its own
 *     head's feature maps through a per-head counter; measured neutral, off by default),
 *     LESS_SMALL_STEP=0|1 (a decode step as ONE launch - a thread-block cluster per head splits the
 *     two MLPs and runs the step of each batch row - never / whenever the shape allows: head_dim 128,
 *     group 1, at most 4 batch rows, hidden in {128, 256, 512}, the state in use; by default when
 *     layers x heads x (batch + 4) CTAs are at most two per multiprocessor).
 */
#ifndef LESS_B200_H
#define LESS_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct less_ctx less_ctx; /* opaque */

enum {
  LESS_OK = 0,
  LESS_ERR_INVALID_CONFIG = -1,
  LESS_ERR_NULL_POINTER = -2,
  LESS_ERR_MISALIGNED = -3,
  LESS_ERR_ARENA_TOO_SMALL = -4,
  LESS_ERR_PROMPT_TOO_LONG = -5,
  LESS_ERR_BAD_LAYER_RANGE = -6,
  LESS_ERR_DEVICE_TIMEOUT = -7,
  LESS_ERR_DEVICE_BOUNDS = -8,
  LESS_ERR_CUDA = -9,
  LESS_ERR_BAD_STATE = -10,
  LESS_ERR_BUFFER_TOO_SMALL = -11
};

/* flags */
enum {
  /* H2O accumulates e^{s_i} / (sparse-only denominator) instead of Eq. 3's
   * full denominator (Section 2.1 describes H2O as summing the attention
   * probabilities a token receives and does not say under which normaliser). */
  LESS_SCORE_NORM_SPARSE = 1u,
  /* Sparse policy alone (the paper's Baseline / Baseline+, Section 4):
   * evicted pairs are dropped, H and z stay zero. */
  LESS_NO_STATE = 2u,
  /* Lambda-masking as the sparse policy (Section 4: a fixed handful of first
   * positions plus the recent window are cached) instead of H2O: `heavy` counts the first
   * positions, which are never evicted, `recent` the sliding window; the prompt
   * keeps positions [0, heavy) and the last `recent`, a decode step evicts the
   * lowest position >= heavy.  Accumulated scores are not used (prompt scoring
   * is skipped unless attn_out is asked for); evicted pairs go to H, z as usual. */
  LESS_POLICY_LAMBDA = 4u,
  /* TOVA as the sparse policy (named in Section 4; the paper does not define
   * it, the rule is the cited work's, applied per head): when the slots
   * overflow, the entry with the lowest attention probability of the CURRENT
   * query is evicted, ties to the lowest position; the new pair competes too
   * (if it loses it is absorbed into H, z and never cached) and no window is
   * protected.  `heavy + recent` only sets the slot count.  The prompt is
   * ranked once, by its last query's attention row.  Not together with
   * LESS_POLICY_LAMBDA. */
  LESS_POLICY_TOVA = 8u,
  /* Reserve the workspace of less_masked_attention (the parallel form) in the arena. */
  LESS_WITH_PARALLEL_FORM = 16u,
  /* less_decode_step / less_decode_step_host write the attention output as fp16 (rounded once
   * from the fp32 result of Eq. 3) instead of fp32: half the output traffic of a step. */
  LESS_OUT_F16 = 32u
};

#define LESS_MAX_SLOTS 32768

typedef struct less_config {
  int32_t batch, layers, heads; /* heads = KV heads: one cache, one H, z and one eviction per (batch, layer, head) */
  int32_t head_dim;           /* D: 128, or 64 (general shapes, see `group`) */
  int32_t rank;               /* R: 8 or 16 (Section 4: R = 8 by default) */
  int32_t hidden;             /* R' = 512 (Section 3.2) */
  int32_t heavy, recent;      /* slots per instance: heavy >= 0, recent >= 1, heavy + recent <= LESS_MAX_SLOTS */
  int32_t max_prompt;         /* longest prompt less_prefill will be given (>= 0) */
  int32_t max_prefill_layers; /* layers scored together in less_prefill (>= 1): sizes the workspace */
  uint32_t flags;
  int32_t group;              /* query heads per KV head (Section 3.2, multi-query attention): 0 or 1 = one;
                               * 2, 4 or 8 with head_dim 128 need hidden in {128, 256, 512}, a policy other than
                               * LESS_POLICY_TOVA, the tensor-core prompt scoring, and
                               * group * (heavy + recent + 1028) * 4 bytes <= 227 KB (the decode kernel
                               * keeps one score per slot and query head in shared memory).
                               * General shapes - head_dim 64, or any other group up to 128 (Section 4's
                               * multi-query model has 71 query heads over one KV head of dimension 64) -
                               * run on CUDA-core kernels (prompt phase and decode); less_masked_attention
                               * is not available for them; 9 * (heavy + recent + 1028) * 4 bytes <= 227 KB,
                               * no LESS_POLICY_TOVA with group > 1.  Anything else is LESS_ERR_INVALID_CONFIG */
} less_config;

/* Per-head feature-map weights (Eq. 1, Eq. 2), device, fp16, row-major, no biases:
 *   phi(q) = | gelu( gelu(q W_phi1) W_phi2 ) |
 *   psi(k) = | c2 * gelu( c1 * gelu(k W_psi1) W_psi2 ) W_psi3 |                     */
typedef struct less_weights {
  const void* w_phi1;     /* [L, H * group, D, R']   (phi belongs to the query head) */
  const void* w_phi2;     /* [L, H * group, R', R] */
  const void* w_psi1;     /* [L, H, D, R'] */
  const void* w_psi2;     /* [L, H, R', R] */
  const void* w_psi3;     /* [L, H, R, R]  */
  const float* psi_scale; /* optional device [L, H, 2] = (c1, c2), the learnable
                             scalars of Section 3.2; NULL means 1 */
} less_weights;

/* Bytes of device memory a context of this shape needs (0 if the config is
 * invalid).  The arena must be 256-byte aligned. */
size_t less_arena_bytes(const less_config* cfg);

/* Validates the config, carves the arena, zeroes H, z (H_0 = 0, z_0 = 0,
 * Section 2.2) and the slot counts.  Synchronous; runs on the legacy default
 * stream.  *out is set only on success. */
int less_create(const less_config* cfg, const less_weights* weights, void* arena_device,
                size_t arena_bytes, less_ctx** out);

/* Prompt phase for layers [layer_begin, layer_begin + layer_count) (Section 3.1:
 * regular attention since H_0 = 0; the policy and the state act afterwards):
 *   1. causal softmax rows of Q K^T / sqrt(D);
 *   2. H2O accumulated scores acc_j = sum_{i >= j} P_ij (diagonal included);
 *   3. keep the `recent` last positions plus the `heavy` others with the
 *      largest (acc, position) keys; if prompt_len <= heavy + recent keep all;
 *   4. kept rows go to slots in ascending position; every other row is
 *      absorbed: H = sum psi(k_j)^T v_j, z = sum psi(k_j) (Eq. 4, Eq. 5 over D_1).
 * Q: device fp16 [B, layer_count, H * group, prompt_len, D]; K, V: device fp16
 * [B, layer_count, H, prompt_len, D]; all contiguous, fewer than
 * 2^31 rows (B * layer_count * H * prompt_len) per call, else LESS_ERR_PROMPT_TOO_LONG.
 * attn_out: device fp32, same shape as Q, or NULL when the caller does not need the
 * prompt's attention output.
 * Every call of one generation must pass the same prompt_len; the first decode
 * token then has absolute position prompt_len.  A layer that was never
 * prefilled starts empty and fills without eviction until its slots are full.
 * Calling it again for a layer resets that layer.  prompt_len == 0 only resets. */
int less_prefill(less_ctx* ctx, int32_t layer_begin, int32_t layer_count, int32_t prompt_len,
                 const void* Q, const void* K, const void* V, void* attn_out, void* cuda_stream);

/* The parallel form (Section 3.2, Inexpensive Training; Section 4.1): all rows of the
 * causal attention matrix of a sequence at once, for training-time / evaluation-time use of
 * the feature maps.  Entry (i, j), j <= i, is exp(q_i . k_j / sqrt(D)) while key j is in the
 * sparse cache when query i attends (i < exact_until[j]) and phi(q_i) psi(k_j)^T from then
 * on; every row is normalised once (Eq. 3):  out_i = sum_j A_ij v_j / sum_j A_ij.
 * exact_until: device int32 [B, layer_count, H, seq_len]: 1 + the step at whose end the
 * policy discarded key j (so exact_until[j] > j when a token attends to itself), INT32_MAX
 * for a key that is never discarded; the caller obtains it from the policy (e.g. the
 * evicted_pos record of less_decode_step).
 * Q, K, V as in less_prefill (seq_len <= max_prompt); out: device fp32, Q's shape
 * [B, layer_count, H * group, seq_len, D].  With group > 1 the query heads of a group read
 * the same K, V, psi(K) and exact_until (the cache belongs to the KV head); each has its own
 * phi and its own normalisation.  Reads the context's weights, touches no cache or state;
 * needs LESS_WITH_PARALLEL_FORM at creation, head_dim 128 with group in {1, 2, 4, 8} and the
 * tensor-core kernels (hidden in {64, 128, 256, 512}), else LESS_ERR_INVALID_CONFIG. */
int less_masked_attention(less_ctx* ctx, int32_t layer_begin, int32_t layer_count, int32_t seq_len,
                          const void* Q, const void* K, const void* V, const int32_t* exact_until,
                          void* out, void* cuda_stream);

/* One generation step for every instance (Algorithm 1), at position t = tokens seen:
 *   phi(q_t), psi(k_t) (Eq. 1, 2); scores over the live slots plus the new pair;
 *   out = (phi(q) H + sum e^{s_i} v_i) / (phi(q) z^T + sum e^{s_i})        (Eq. 3)
 *   acc_i += p_i, acc_new = p_new  with p = e^{s} / denominator            (H2O)
 *   if the slots overflow: victim = argmin (acc, position) over entries with
 *   position <= t - recent;  H += psi(k_vic)^T v_vic,  z += psi(k_vic)  (Eq. 4, 5);
 *   the new pair overwrites the victim's slot in place (Section 3.2), else
 *   it takes the next free slot.
 * q: device fp16 [B, L, H * group, D]; k, v: device fp16 [B, L, H, D]; out: device fp32
 * (fp16 with LESS_OUT_F16) [B, L, H * group, D] (query head h * group + g belongs to KV head h).  With group > 1
 * (Section 3.2: multi-query attention) every query head has its own phi and its own Eq. 3 over
 * the KV head's cache and state, and the H2O score of an entry grows by the sum of the query
 * heads' probabilities; policies: H2O and Lambda-masking.
 * evicted_pos: device int32 [B, L, H] or NULL; receives the evicted position
 * or -1.  Advances the context's position by one.  A step captured in a CUDA
 * graph (fixed q, k, v, out buffers; make one direct call first) reads the
 * position from device memory and advances it there, so every replay is the
 * next step; after replays, call less_poll_status (or less_export_state)
 * before the next direct call so that the host's copy of the position catches
 * up. */
int less_decode_step(less_ctx* ctx, const void* q, const void* k, const void* v, void* out,
                     int32_t* evicted_pos, void* cuda_stream);

/* The same step for callers whose tensors live in host memory (Algorithm 1's
 * inputs and return value): q host fp16 [B, L, H * group, D], k, v host fp16
 * [B, L, H, D], out host fp32 (fp16 with LESS_OUT_F16) [B, L, H * group, D].  From pinned
 * (page-locked, device-mapped) memory v and out are read / written in place by the decode kernel,
 * and with at most 8 batch rows q and k are read in place too (the feature-map kernel then fetches
 * its rows with plain loads while the weights stream: no copy in front of the step).  Otherwise q
 * and k are copied to staging buffers inside the arena: a large step goes in four layer segments
 * whose copies (on a stream the context creates at the first such call) run under the kernels of
 * the segment before; a small one in ONE copy when k_host starts exactly where q_host ends (one
 * host block [q | k]), else in two.  Pageable v / out are staged and copied as well.  Everything is
 * ordered behind the given stream, which is synchronised before returning. */
int less_decode_step_host(less_ctx* ctx, const void* q_host, const void* k_host, const void* v_host,
                          void* out_host, void* cuda_stream);

/* Per-kernel device timing.  less_profile(ctx, 1) makes every later kernel
 * launch of this context record a CUDA event pair on its stream;
 * less_profile(ctx, 0) stops and discards.  less_profile_read synchronises the
 * recorded events and adds up, per kernel id, the elapsed milliseconds and the
 * launch count since profiling was enabled (arrays of LESS_KERNEL_COUNT). */
enum {
  LESS_KERNEL_FEATURE_MAP = 0,
  LESS_KERNEL_DECODE = 1,
  LESS_KERNEL_ROWSTAT = 2,
  LESS_KERNEL_COLSUM = 3,
  LESS_KERNEL_ATTN_OUT = 4,
  LESS_KERNEL_SELECT = 5,
  LESS_KERNEL_BUILD = 6,
  LESS_KERNEL_FINALIZE = 7,
  LESS_KERNEL_PSI = 8,
  LESS_KERNEL_GATHER = 9,
  LESS_KERNEL_MASKED_PACK = 10,
  LESS_KERNEL_MASKED_OUT = 11,
  LESS_KERNEL_COUNT = 12
};
int less_profile(less_ctx* ctx, int enable);
int less_profile_read(less_ctx* ctx, float* ms_total_host, int64_t* launches_host);

/* Tokens seen so far (= absolute position of the next decode token), as the
 * host last knew it: direct calls keep it current; after graph replays
 * less_poll_status or less_export_state refresh it from the device. */
int64_t less_position(const less_ctx* ctx);

/* Bytes of one exported instance record:
 *   int32 count, int32 position, int32 reserved[2],
 *   int32 pos[N], float acc[N], fp16 K[N][D], fp16 V[N][D], float psi[N][R],
 *   float H[R][D], float z[R]        with N = heavy + recent.
 * Slots [count, N) are unspecified. */
size_t less_state_record_bytes(const less_config* cfg);

/* Copies the records of the listed instances (host int32 list) to / from a
 * host buffer of n * less_state_record_bytes bytes.  Synchronises the stream
 * before returning.  Algorithm 1's "save K, V, H, z"; also what teacher-forced
 * tests use.  Import sets the context's position from record 0. */
int less_export_state(less_ctx* ctx, const int32_t* inst_host, int32_t n, void* host_buf,
                      size_t bytes, void* cuda_stream);
int less_import_state(less_ctx* ctx, const int32_t* inst_host, int32_t n, const void* host_buf,
                      size_t bytes, void* cuda_stream);

/* phi(q_t) and psi(k_t) of the last decode step: host float [B*L*H*group, R]
 * and [B*L*H, R] (either may be NULL).  Synchronises the stream. */
int less_read_feature_maps(less_ctx* ctx, float* phi_host, float* psi_host, void* cuda_stream);

/* Reads the device status word (synchronises the stream): 0, or
 * LESS_ERR_DEVICE_TIMEOUT / LESS_ERR_DEVICE_BOUNDS if a kernel gave up on a
 * bounded wait or refused an out-of-range index. */
int less_poll_status(less_ctx* ctx, void* cuda_stream);

/* Kernels of this library launched through this context so far. */
int64_t less_launch_count(const less_ctx* ctx);

/* Name of the kernel variant last launched under a LESS_KERNEL_* id (template arguments
 * included), "" if none yet.  The string lives in the context. */
const char* less_kernel_variant(const less_ctx* ctx, int kernel_id);

/* The where-code that came with the status word at the last less_poll_status (which wait gave
 * up, which check refused), 0 if the status was clean. */
int less_last_status_where(const less_ctx* ctx);

/* Self-test of the bounded device-side waits (no counterpart in the paper).  Launches one small
 * CTA whose consumer waits, for at most `polls` polls (1 .. 2^20), on a barrier nothing ever
 * arrives at, through the same helper every pipeline of the library waits with.  The wait runs
 * out, the kernel returns, and the context's status word then reads LESS_ERR_DEVICE_TIMEOUT
 * (less_poll_status; less_last_status_where gives 90).  The status word is sticky: use a context
 * of its own for this call.  Asynchronous on the given stream. */
int less_selftest_wait_timeout(less_ctx* ctx, uint32_t polls, void* cuda_stream);

/* The paper has no counterpart for this entry point: it exists for callers
 * that may not allocate device memory (a process whose memory pool owns the
 * whole GPU, a plugin that is only handed buffers and a stream, code that must
 * not trigger the synchronisation an allocation implies).  It computes the H2O
 * prompt scores of less_prefill's step 2 on its own:
 *     acc_out[n][j] = sum_{i >= j} softmax_row_i( Q_n K_n^T / sqrt(D), causal )[j]
 * for n_inst independent heads, with the per-row scratch (row maximum and
 * reciprocal row sum) held in a fixed 512 KB array inside the library image,
 * which every GPU that loads the library keeps until the process exits.
 *   Q, K      device fp16 [n_inst, prompt_len, 128], 16-byte aligned
 *   acc_out   device fp32 [n_inst, prompt_len]
 * Limits and rules:
 *   - n_inst * prompt_len <= LESS_NOALLOC_MAX_ROWS, else LESS_ERR_NOALLOC_TOO_LARGE
 *     (nothing is launched);
 *   - it calls no cudaMalloc / cudaFree and no allocating library routine;
 *   - all calls on a device share the one array: calls ordered on a stream are
 *     safe, calls that can overlap on the GPU race with each other;
 *   - no part of the array needs clearing between calls (each call overwrites
 *     every row it reads);
 *   - the first call on each device looks up the array's device address: make
 *     that call with the device current and outside any stream capture; first
 *     calls from several host threads at once are safe (the lookup is idempotent
 *     and its result is published atomically).
 * Asynchronous on the given stream. */
#define LESS_NOALLOC_MAX_ROWS 65536
#define LESS_ERR_NOALLOC_TOO_LARGE (-12)
int less_prompt_scores_noalloc(const void* Q, const void* K, int32_t n_inst, int32_t prompt_len,
                               float* acc_out, void* cuda_stream);

const char* less_strerror(int code);

/* Releases the context; frees nothing the caller owns. */
int less_destroy(less_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* LESS_B200_H */
