// Prompt state build on the tensor cores (Eq. 4 / Eq. 5 summed over the
// discarded set D_1):   H^T[D x R] = V_ev^T psi(K_ev),   z = 1^T psi(K_ev).
//
// One CTA = one token split of one instance.  Per 128-token tile:
//   * TMA brings the V tile [128 tokens x 128] into shared memory (128-byte swizzle);
//     as the A operand it is "M-major": M = head dimension, K = tokens;
//   * four worker warps read psi of their token, zero it for kept / out-of-range
//     tokens, scale it by a per-instance power of two, split it into fp16 hi + lo (so the
//     fp16 tensor-core product keeps fp32 accuracy) and lay it out as the B operand [K = tokens, N = 2R];
//   * one thread issues tcgen05.mma: 8 k-steps into the H accumulator and 8 more
//     with an all-ones A operand into the z accumulator, both in tensor memory.
// After the last tile the workers read the accumulators back (tcgen05.ld), add
// hi + lo and store the split's partial H, z; finalize_kernel sums the splits in
// a fixed order.  Every wait is bounded (see pipeline.cuh).
#include "prefill.cuh"
#include "tc_common.cuh"

namespace less {

constexpr int ST_WORKERS = 128;
constexpr int ST_THREADS = ST_WORKERS + 64;      // + TMA warp + MMA warp
constexpr int ST_STAGES = 2;
constexpr int ST_TILE = 128;                     // tokens per tile
constexpr int ST_VBYTES = ST_TILE * kHeadDim * 2;

struct StShared {
  uint64_t full_v[ST_STAGES];
  uint64_t full_b[ST_STAGES];
  uint64_t empty[ST_STAGES];
  uint64_t done;
  uint32_t tmem_base;
  int abort;
};

__device__ __forceinline__ void st_wait(uint64_t* bar, uint32_t parity, volatile int* abort, int32_t* status,
                                        int where) {
  if (*abort) return;
  if (!mbar_wait(bar, parity)) {
    *abort = 1;
    set_status(status, kStatusTimeout, where);
  }
}

template <int R>
__global__ void __launch_bounds__(ST_THREADS) state_tc_kernel(const __grid_constant__ CUtensorMap tmap_v,
                                                              PfParams p) {
  constexpr int NB = 2 * R;                         // hi | lo columns
  constexpr int BBYTES = ST_TILE * NB * 2;          // B operand of one tile
  constexpr uint32_t B_SBO = 128;                   // between 8-column blocks
  constexpr uint32_t B_LBO = (NB / 8) * 128;        // between 8-token groups
  extern __shared__ __align__(1024) unsigned char st_smem[];
  if (smem_misaligned(st_smem, p.a.status, 19)) return;
  unsigned char* vbuf = st_smem;                                        // [stages][2 dblocks][128][128 B]
  unsigned char* bbuf = vbuf + ST_STAGES * ST_VBYTES;                   // [stages][BBYTES]
  __half* ones = reinterpret_cast<__half*>(bbuf + ST_STAGES * BBYTES);  // 4 KB of 1.0
  StShared* sh = reinterpret_cast<StShared*>(reinterpret_cast<unsigned char*>(ones) + 4096);

  const int tid = threadIdx.x, warp = tid >> 5;
  const int split = blockIdx.x, g = blockIdx.y;
  const InstMap im = map_instance(p, g);
  const int jbeg = split * p.split_tokens, jend = min(p.S, jbeg + p.split_tokens);
  const int ntiles = (jend - jbeg + ST_TILE - 1) / ST_TILE;

  if (tid == 0) {
    for (int s = 0; s < ST_STAGES; ++s) {
      mbar_init(&sh->full_v[s], 1);
      mbar_init(&sh->full_b[s], ST_WORKERS / 32);
      mbar_init(&sh->empty[s], 1);
    }
    mbar_init(&sh->done, 1);
    // a CTA that starts after another one has given up skips every wait: the grid drains at once
    sh->abort = *reinterpret_cast<volatile int32_t*>(p.a.status) != 0;
    mbar_fence_init();
  }
  for (int e = tid; e < 2048; e += ST_THREADS) ones[e] = __float2half(1.0f);
  if (warp == 5) tmem_alloc(&sh->tmem_base, 64);
  fence_proxy_async_smem();            // the ones tile is read by the MMA (async proxy)
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh->tmem_base;
  volatile int* abortp = &sh->abort;

  if (warp == 4) {
    // ---------------- TMA producer ----------------
    if (tid == ST_WORKERS) {
      const uint64_t stream_policy = l2_evict_first_policy();
      for (int i = 0; i < ntiles; ++i) {
        const int s = i % ST_STAGES;
        st_wait(&sh->empty[s], ((i / ST_STAGES) & 1) ^ 1, abortp, p.a.status, 20);
        if (*abortp) break;                      // issue nothing more once the CTA has given up
        mbar_expect_tx(&sh->full_v[s], ST_VBYTES);
        const int row = (int)(im.in_row0 + jbeg + (size_t)i * ST_TILE);
        tma_load_2d_hint(vbuf + s * ST_VBYTES, &tmap_v, 0, row, &sh->full_v[s], stream_policy);
        tma_load_2d_hint(vbuf + s * ST_VBYTES + ST_VBYTES / 2, &tmap_v, 64, row, &sh->full_v[s], stream_policy);
      }
    }
  } else if (warp == 5) {
    // ---------------- MMA issuer ----------------
    if (tid == ST_WORKERS + 32) {
      constexpr uint32_t idesc_h = idesc_f16(128, NB, 1, 1);   // A = V tile (M-major), B = psi (N-major)
      constexpr uint32_t idesc_z = idesc_f16(128, NB, 0, 1);   // A = ones (K-major)
      const uint32_t ones_addr = smem_u32(ones);
      for (int i = 0; i < ntiles; ++i) {
        const int s = i % ST_STAGES;
        const uint32_t par = (i / ST_STAGES) & 1;
        st_wait(&sh->full_v[s], par, abortp, p.a.status, 21);
        st_wait(&sh->full_b[s], par, abortp, p.a.status, 22);
        if (*abortp) break;
        tc_fence_after_sync();
        const uint32_t va = smem_u32(vbuf + s * ST_VBYTES), ba = smem_u32(bbuf + s * BBYTES);
#pragma unroll
        for (int ks = 0; ks < ST_TILE / 16; ++ks) {
          const uint64_t bd = smem_desc(ba + ks * 2 * B_LBO, B_LBO, B_SBO, kLayoutNone);
          const uint64_t ad = smem_desc(va + ks * 2048, ST_VBYTES / 2, 1024, kLayoutSw128);
          mma_f16_ss(tmem, ad, bd, idesc_h, (i | ks) ? 1u : 0u);
          const uint64_t od = smem_desc(ones_addr, 128, 256, kLayoutNone);
          mma_f16_ss(tmem + 32, od, bd, idesc_z, (i | ks) ? 1u : 0u);
        }
        mma_commit(&sh->empty[s]);
      }
      mma_commit(&sh->done);
    }
  } else {
    // ---------------- workers: B operand, then epilogue ----------------
    // psi is scaled by a power of two so that the instance's largest value lands near 8192: the hi
    // parts stay far from fp16's overflow and the lo parts as far from its underflow as they can be,
    // whatever the magnitude of the trained maps (the paper initialises psi's scalars to 1e-4)
    const float pmax = __int_as_float(p.a.ws_pmax[g]);
    float scale = 1.f;
    if (pmax > 0.f && pmax < INFINITY) scale = exp2f(fminf(fmaxf(floorf(log2f(8192.f / pmax)), -100.f), 100.f));
    const float* psi = p.a.ws_psi + (size_t)g * p.Sp * R;
    const int32_t* slot_of = p.a.ws_slot + (size_t)g * p.Sp;
    for (int i = 0; i < ntiles; ++i) {
      const int s = i % ST_STAGES;
      const int j = jbeg + i * ST_TILE + tid;
      float v[R];
      const bool use = j < jend && slot_of[j] < 0;           // discarded prompt token
      if (use) {
#pragma unroll
        for (int r4 = 0; r4 < R / 4; ++r4) {
          const float4 f = __ldg(reinterpret_cast<const float4*>(psi + (size_t)j * R) + r4);
          v[r4 * 4] = f.x; v[r4 * 4 + 1] = f.y; v[r4 * 4 + 2] = f.z; v[r4 * 4 + 3] = f.w;
        }
      } else {
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = 0.f;
      }
      __align__(16) __half hi[R], lo[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float x = v[r] * scale;
        hi[r] = __float2half_rn(x);
        lo[r] = __float2half_rn(x - __half2float(hi[r]));
      }
      st_wait(&sh->empty[s], ((i / ST_STAGES) & 1) ^ 1, abortp, p.a.status, 23);
      if (*abortp) break;
      unsigned char* brow = bbuf + s * BBYTES + (tid >> 3) * B_LBO + (tid & 7) * 16;
#pragma unroll
      for (int nb = 0; nb < R / 8; ++nb) {
        *reinterpret_cast<uint4*>(brow + nb * B_SBO) = *reinterpret_cast<const uint4*>(&hi[nb * 8]);
        *reinterpret_cast<uint4*>(brow + (R / 8 + nb) * B_SBO) = *reinterpret_cast<const uint4*>(&lo[nb * 8]);
      }
      fence_proxy_async_smem();
      mbar_arrive_warp(&sh->full_b[s]);
    }
    st_wait(&sh->done, 0, abortp, p.a.status, 24);
    tc_fence_after_sync();
    uint32_t acc[NB];
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
#pragma unroll
    for (int c = 0; c < NB / 8; ++c) tmem_ld8(lane_addr + c * 8, acc + c * 8);
    tmem_ld_wait();
    float* hp = p.a.ws_hpart + ((size_t)g * kMaxSplit + split) * (R * kHeadDim + R);
    const float inv = 1.0f / scale;                    // exact: a power of two
#pragma unroll
    for (int r = 0; r < R; ++r)
      hp[r * kHeadDim + tid] = (__uint_as_float(acc[r]) + __uint_as_float(acc[R + r])) * inv;
    if (warp == 0) {                                  // every row of the z accumulator holds z
#pragma unroll
      for (int c = 0; c < NB / 8; ++c) tmem_ld8(lane_addr + 32 + c * 8, acc + c * 8);
      tmem_ld_wait();
      if (tid == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r)
          hp[R * kHeadDim + r] = (__uint_as_float(acc[r]) + __uint_as_float(acc[R + r])) * inv;
      }
    }
  }
  drain_after_abort(abortp);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, 64);
}

int launch_state_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s) {
  const Dims& d = c->d;
  CUtensorMap tmap_v;
  const uint64_t rows = (uint64_t)d.B * p.layer_count * d.Hd * p.S;
  if (!make_tmap_f16_2d(&tmap_v, p.V, rows, kHeadDim, kHeadDim * 2, ST_TILE)) return fail_cuda("tensor map of V");
  const int NB = 2 * d.R;
  const size_t smem = (size_t)ST_STAGES * (ST_VBYTES + ST_TILE * NB * 2) + 4096 + sizeof(StShared) + 1024;
  LaunchScope scope(c, LESS_KERNEL_BUILD, s, "state_tc_kernel");
  if (d.R == 8) {
    cudaFuncSetAttribute(state_tc_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    state_tc_kernel<8><<<dim3(p.nsplit, G), ST_THREADS, smem, s>>>(tmap_v, p);
  } else {
    cudaFuncSetAttribute(state_tc_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    state_tc_kernel<16><<<dim3(p.nsplit, G), ST_THREADS, smem, s>>>(tmap_v, p);
  }
  return check_launch("state_tc_kernel");
}

}  // namespace less
