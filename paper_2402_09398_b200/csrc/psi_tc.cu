// psi(k_j) of every prompt token on the tensor cores (Eq. 2):
//     psi(k) = | c2 * gelu( c1 * gelu(k W1) W2 ) W3 |
//
// One CTA = one token split of one instance; W1 of the instance's head (128 KB)
// stays in shared memory for all of the split's tiles.  Per 128-token tile:
//   GEMM1  D1[128 x 64] = Ktile[128 x 128] * W1[:, chunk]       8 chunks of 64 hidden units,
//                                                               D1 double-buffered in tensor memory
//   epilogue warps: tcgen05.ld D1 -> gelu -> fp16 hi + lo -> shared memory (A operands of GEMM2;
//                   a single fp16 rounding of the hidden layer costs ~2e-3 on individual psi vectors)
//   GEMM2  G2[128 x 16] += (hidden_hi + hidden_lo)[128 x 64] * W2[chunk rows, :]
//   after 8 chunks: tcgen05.ld G2 -> c2 * gelu(c1 * .) -> W3 on CUDA cores -> abs -> psi[token][R]
// The same kernel evaluates phi(q) = | gelu( gelu(q W1) W2 ) | (Eq. 1) over a sequence of queries for
// the parallel form (PtMap::is_phi: no W3, no scalars, rows of Q).
// Roles: warps 0-15 epilogue (lane quadrant = warp & 3, token row = tensor-memory lane; the four
// warps of a quadrant split a chunk's 64 columns), warp 16 TMA producer, warp 17 issues GEMM1, warp 18
// GEMM2.  Operands come in by TMA tiled loads with the 128-byte swizzle (no multicast).  Every wait is bounded.
#include "prefill.cuh"
#include "tc_common.cuh"

namespace less {

constexpr int PT_WORKERS = 512;                    // 16 epilogue warps: four per tensor-memory lane quadrant (GELU issue and latency bound the kernel)
constexpr int PT_THREADS = PT_WORKERS + 96;         // + TMA producer, GEMM1 issuer, GEMM2 issuer
constexpr int PT_TILE = 128;                       // tokens per tile
constexpr int PT_CHUNK = 64;                       // hidden units per GEMM1 chunk
constexpr int PT_PARTS = PT_WORKERS / 128;         // warps per lane quadrant
constexpr int PT_COLS = PT_CHUNK / PT_PARTS;       // columns of a chunk per warp (16)
constexpr int PT_KBYTES = PT_TILE * kHeadDim * 2;  // one K tile
constexpr int PT_W2N = 16;                         // GEMM2 N (R padded to 16)

struct PtShared {
  uint64_t w1_full;
  uint64_t k_full, k_empty;
  uint64_t d1_full[2], d1_free[2];
  uint64_t hid_full, hid_free;
  uint64_t g2_full, g2_free;
  uint32_t tmem_base;
  int abort;
  float w3[16 * 16];
  float c1, c2;
};

__device__ __forceinline__ void pt_wait(uint64_t* bar, uint32_t parity, volatile int* abort, int32_t* status,
                                        int where) {
  if (*abort) return;
  if (!mbar_wait(bar, parity)) {
    *abort = 1;
    set_status(status, kStatusTimeout, where);
  }
}

// which map: its layer-2 (and layer-3) weights, where the result goes
struct PtMap {
  const __half* w2;     // [L, Hd, Rp, R]
  const __half* w3;     // [L, Hd, R, R], psi only
  float* out;           // [Iw][Sp][R]
  int32_t* pmax;        // [Iw] bit pattern of the largest value per instance, or null
  int is_phi;
};

template <int R>
__global__ void __launch_bounds__(PT_THREADS) psi_tc_kernel(const __grid_constant__ CUtensorMap tmap_k,
                                                            const __grid_constant__ CUtensorMap tmap_w1,
                                                            PfParams p, PtMap mp) {
  extern __shared__ __align__(1024) unsigned char pt_smem[];
  const int Rp = p.Rp;
  const int nchunk = Rp / PT_CHUNK;
  unsigned char* w1s = pt_smem;                                  // [nchunk][128 k][64 n]  (16 KB each)
  unsigned char* kbuf = w1s + (size_t)nchunk * 16384;            // [2 kblocks][128 tok][64]
  unsigned char* hid = kbuf + PT_KBYTES;                         // hi, lo: [128 tok][64 hidden] fp16, swizzled
  unsigned char* w2s = hid + 2 * 16384;                          // [Rp/8][2 nblocks][8 k][8 n] fp16
  PtShared* sh = reinterpret_cast<PtShared*>(w2s + (size_t)Rp * PT_W2N * 2);

  const int tid = threadIdx.x, warp = tid >> 5;
  const int split = blockIdx.x, g = blockIdx.y;
  const InstMap im = map_instance(p, g);
  const int jbeg = split * p.split_tokens, jend = min(p.S, jbeg + p.split_tokens);
  const int ntiles = (jend - jbeg + PT_TILE - 1) / PT_TILE;

  if (tid == 0) {
    mbar_init(&sh->w1_full, 1);
    mbar_init(&sh->k_full, 1);
    mbar_init(&sh->k_empty, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh->d1_full[s], 1);
      mbar_init(&sh->d1_free[s], PT_WORKERS / 32);
    }
    mbar_init(&sh->hid_full, PT_WORKERS / 32);
    mbar_init(&sh->hid_free, 1);
    mbar_init(&sh->g2_full, 1);
    mbar_init(&sh->g2_free, PT_WORKERS / 32);
    // a CTA that starts after another one has given up skips every wait: the grid drains at once
    sh->abort = *reinterpret_cast<volatile int32_t*>(p.a.status) != 0;
    sh->c1 = (p.psi_scale && !mp.is_phi) ? p.psi_scale[im.lh * 2] : 1.f;
    sh->c2 = (p.psi_scale && !mp.is_phi) ? p.psi_scale[im.lh * 2 + 1] : 1.f;
    mbar_fence_init();
  }
  // W2 as the GEMM2 B operand (N padded to 16 with zeros), W3 as fp32
  {
    const __half* w2 = mp.w2 + (size_t)im.lh * Rp * R;
    for (int e = tid; e < Rp * 2; e += PT_THREADS) {             // e = (k, nblock)
      const int k = e >> 1, nb = e & 1;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (nb * 8 < R) v = __ldg(reinterpret_cast<const uint4*>(w2 + (size_t)k * R + nb * 8));
      *reinterpret_cast<uint4*>(w2s + (k >> 3) * 256 + nb * 128 + (k & 7) * 16) = v;
    }
    if (!mp.is_phi) {
      const __half* w3 = mp.w3 + (size_t)im.lh * R * R;
      for (int e = tid; e < R * R; e += PT_THREADS) sh->w3[e] = __half2float(w3[e]);
    }
  }
  if (warp == PT_WORKERS / 32 + 1) tmem_alloc(&sh->tmem_base, 256);
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh->tmem_base;
  volatile int* abortp = &sh->abort;
  int32_t* status = p.a.status;

  if (warp == PT_WORKERS / 32) {
    // ---------------- TMA producer ----------------
    if (tid == PT_WORKERS) {
      const uint64_t stream_policy = l2_evict_first_policy();
      mbar_expect_tx(&sh->w1_full, (uint32_t)nchunk * 16384);
      for (int c = 0; c < nchunk; ++c)
        tma_load_2d(w1s + (size_t)c * 16384, &tmap_w1, c * 64, im.lh * kHeadDim, &sh->w1_full);
      for (int i = 0; i < ntiles; ++i) {
        pt_wait(&sh->k_empty, (i & 1) ^ 1, abortp, status, 30);
        if (*abortp) break;                      // issue nothing more once the CTA has given up
        mbar_expect_tx(&sh->k_full, PT_KBYTES);
        const int row = (int)(im.in_row0 + jbeg + (size_t)i * PT_TILE);
        tma_load_2d_hint(kbuf, &tmap_k, 0, row, &sh->k_full, stream_policy);
        tma_load_2d_hint(kbuf + PT_KBYTES / 2, &tmap_k, 64, row, &sh->k_full, stream_policy);
      }
    }
  } else if (warp == PT_WORKERS / 32 + 1) {
    // ---------------- MMA issuer of GEMM1 ----------------
    // One issuing thread per GEMM: a single thread gets an MMA out every ~84 cycles, and 128 of them per
    // token tile in one thread were on the critical path of every chunk; the two streams only meet at
    // the barriers they already had (d1_free / d1_full, hid_full / hid_free, g2_free / g2_full).
    if (tid == PT_WORKERS + 32) {
      constexpr uint32_t idesc1 = idesc_f16(128, PT_CHUNK, 0, 1);   // A = K tile (K-major), B = W1 (N-major)
      const uint32_t w1a = smem_u32(w1s);
      pt_wait(&sh->w1_full, 0, abortp, status, 31);
      uint32_t q = 0;                                               // chunk counter over all tiles
      for (int i = 0; i < ntiles && !*abortp; ++i) {
        pt_wait(&sh->k_full, i & 1, abortp, status, 33);
        const uint32_t ka = smem_u32(kbuf);
        for (int c = 0; c < nchunk && !*abortp; ++c, ++q) {
          const int b = q & 1;
          pt_wait(&sh->d1_free[b], ((q >> 1) & 1) ^ 1, abortp, status, 32);
          if (*abortp) break;
          tc_fence_after_sync();
#pragma unroll
          for (int ks = 0; ks < kHeadDim / 16; ++ks) {
            const uint64_t ad = smem_desc(ka + (ks >> 2) * (PT_KBYTES / 2) + (ks & 3) * 32, 16, 1024, kLayoutSw128);
            const uint64_t bd = smem_desc(w1a + c * 16384 + ks * 2048, 16384, 1024, kLayoutSw128);
            mma_f16_ss(tmem + b * PT_CHUNK, ad, bd, idesc1, ks ? 1u : 0u);
          }
          mma_commit(&sh->d1_full[b]);
        }
        mma_commit(&sh->k_empty);                                   // all GEMM1s of this tile are issued
      }
    }
  } else if (warp == PT_WORKERS / 32 + 2) {
    // ---------------- MMA issuer of GEMM2 ----------------
    if (tid == PT_WORKERS + 64) {
      constexpr uint32_t idesc2 = idesc_f16(128, PT_W2N, 0, 1);     // A = hidden (K-major), B = W2 (N-major)
      const uint32_t w2a = smem_u32(w2s), hida = smem_u32(hid);
      uint32_t q = 0;
      for (int i = 0; i < ntiles && !*abortp; ++i) {
        for (int c = 0; c < nchunk; ++c, ++q) {
          if (c == 0) pt_wait(&sh->g2_free, (i & 1) ^ 1, abortp, status, 34);
          pt_wait(&sh->hid_full, q & 1, abortp, status, 35);
          if (*abortp) break;
          tc_fence_after_sync();
#pragma unroll
          for (int ks = 0; ks < PT_CHUNK / 16; ++ks) {
            const uint64_t bd = smem_desc(w2a + (c * (PT_CHUNK / 8) + ks * 2) * 256, 256, 128, kLayoutNone);
            const uint64_t ah = smem_desc(hida + ks * 32, 16, 1024, kLayoutSw128);
            const uint64_t al = smem_desc(hida + 16384 + ks * 32, 16, 1024, kLayoutSw128);
            mma_f16_ss(tmem + 128, ah, bd, idesc2, (c | ks) ? 1u : 0u);
            mma_f16_ss(tmem + 128, al, bd, idesc2, 1u);
          }
          mma_commit(&sh->hid_free);
        }
        if (*abortp) break;
        mma_commit(&sh->g2_full);
      }
    }
  } else {
    // ---------------- epilogue workers ----------------
    const float c1 = sh->c1, c2 = sh->c2;
    const int quad = warp & 3, half = warp >> 2;       // half: which PT_COLS columns of a chunk
    const int row = quad * 32 + (tid & 31);                         // token row of the tile = tensor-memory lane
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    float* psi = mp.out + (size_t)g * p.Sp * R;
    unsigned char* hrow = hid + row * 128;
    uint32_t q = 0;
    float pmax = 0.f;                                               // largest psi this thread has produced
    for (int i = 0; i < ntiles && !*abortp; ++i) {
      for (int c = 0; c < nchunk && !*abortp; ++c, ++q) {
        const int b = q & 1;
        pt_wait(&sh->d1_full[b], (q >> 1) & 1, abortp, status, 36);
        tc_fence_after_sync();
        uint32_t acc[PT_COLS];                                       // this warp's 16 of the chunk's 64 columns
        static_assert(PT_COLS == 16, "one 16-column tensor-memory load per warp and chunk");
        tmem_ld16(lane_addr + b * PT_CHUNK + half * PT_COLS, acc);
        tmem_ld_wait();
        tc_fence_before_sync();
        mbar_arrive_warp(&sh->d1_free[b]);
        uint32_t phi_[PT_COLS / 2], plo_[PT_COLS / 2];
#pragma unroll
        for (int e = 0; e < PT_COLS / 2; ++e) {
          // c1 multiplies the layer-2 sums instead (same value): the fp16 hi + lo operand then never
          // depends on how small the learnable scalar is (the paper initialises it to 1e-4)
          const float h0 = gelu_erf(__uint_as_float(acc[2 * e]));
          const float h1 = gelu_erf(__uint_as_float(acc[2 * e + 1]));
          const __half2 hh = __floats2half2_rn(h0, h1);
          const float2 hf = __half22float2(hh);
          const __half2 ll = __floats2half2_rn(h0 - hf.x, h1 - hf.y);
          phi_[e] = *reinterpret_cast<const uint32_t*>(&hh);
          plo_[e] = *reinterpret_cast<const uint32_t*>(&ll);
        }
        pt_wait(&sh->hid_free, (q & 1) ^ 1, abortp, status, 37);
#pragma unroll
        for (int cq = 0; cq < PT_COLS / 8; ++cq) {     // 16-byte chunk half * 2 + cq of this row, 128-byte swizzle
          const int off = ((half * (PT_COLS / 8) + cq) ^ (row & 7)) << 4;
          *reinterpret_cast<uint4*>(hrow + off) =
              make_uint4(phi_[cq * 4], phi_[cq * 4 + 1], phi_[cq * 4 + 2], phi_[cq * 4 + 3]);
          *reinterpret_cast<uint4*>(hrow + 16384 + off) =
              make_uint4(plo_[cq * 4], plo_[cq * 4 + 1], plo_[cq * 4 + 2], plo_[cq * 4 + 3]);
        }
        fence_proxy_async_smem();
        mbar_arrive_warp(&sh->hid_full);
      }
      pt_wait(&sh->g2_full, i & 1, abortp, status, 38);
      tc_fence_after_sync();
      uint32_t g2[PT_W2N];
      if (half == 0) {                                 // warp-uniform: one warp per quadrant finishes the rows
        tmem_ld16(lane_addr + 128, g2);
        tmem_ld_wait();
      }
      tc_fence_before_sync();
      mbar_arrive_warp(&sh->g2_free);
      const int j = jbeg + i * PT_TILE + row;
      if (half == 0 && j < jend) {
        float gv[R], out[R];
#pragma unroll
        for (int r = 0; r < R; ++r) gv[r] = c2 * gelu_erf(c1 * __uint_as_float(g2[r]));
#pragma unroll
        for (int r = 0; r < R; ++r) {
          float s = gv[r];                               // phi stops after the second layer (Eq. 1)
          if (!mp.is_phi) {
            s = 0.f;
#pragma unroll
            for (int rr = 0; rr < R; ++rr) s = fmaf(gv[rr], sh->w3[rr * R + r], s);
          }
          out[r] = fabsf(s);
          pmax = fmaxf(pmax, out[r]);
        }
#pragma unroll
        for (int r4 = 0; r4 < R / 4; ++r4)
          reinterpret_cast<float4*>(psi + (size_t)j * R)[r4] =
              make_float4(out[r4 * 4], out[r4 * 4 + 1], out[r4 * 4 + 2], out[r4 * 4 + 3]);
      }
    }
    // maximum over the split, into the instance's cell: psi >= 0, so its bit pattern orders like an
    // integer, and a maximum does not depend on the order of the atomics
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) pmax = fmaxf(pmax, __shfl_xor_sync(0xffffffffu, pmax, o));
    if ((tid & 31) == 0 && mp.pmax && pmax > 0.f && pmax < INFINITY) atomicMax(mp.pmax + g, __float_as_int(pmax));
  }
  drain_after_abort(abortp);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == PT_WORKERS / 32 + 1) tmem_dealloc(tmem, 256);
}

bool psi_tc_supported(const Dims& d) { return d.Rp == 512 || d.Rp == 256 || d.Rp == 128 || d.Rp == 64; }

// x: the rows the map is applied to ([B, layer_count, Hd, S, D]); which = 0 phi (w_phi1, w_phi2 -> out), 1 psi
static int launch_map_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s, const __half* x, const void* w1,
                         const PtMap& mp) {
  const Dims& d = c->d;
  CUtensorMap tmap_k, tmap_w1;
  const uint64_t rows = (uint64_t)d.B * p.layer_count * d.Hd * p.S;
  if (!make_tmap_f16_2d(&tmap_k, x, rows, kHeadDim, kHeadDim * 2, PT_TILE)) return fail_cuda("tensor map of K");
  if (!make_tmap_f16_2d(&tmap_w1, w1, (uint64_t)d.L * d.Hd * kHeadDim, d.Rp, (uint64_t)d.Rp * 2, kHeadDim))
    return fail_cuda("tensor map or shared memory opt-in");
  const size_t smem = (size_t)(d.Rp / PT_CHUNK) * 16384 + PT_KBYTES + 2 * 16384 + (size_t)d.Rp * PT_W2N * 2 +
                      sizeof(PtShared) + 64;
  LaunchScope scope(c, LESS_KERNEL_PSI, s);
  if (d.R == 8) {
    if (cudaFuncSetAttribute(psi_tc_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return fail_cuda("tensor map or shared memory opt-in");
    psi_tc_kernel<8><<<dim3(p.nsplit, G), PT_THREADS, smem, s>>>(tmap_k, tmap_w1, p, mp);
  } else {
    if (cudaFuncSetAttribute(psi_tc_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return fail_cuda("tensor map or shared memory opt-in");
    psi_tc_kernel<16><<<dim3(p.nsplit, G), PT_THREADS, smem, s>>>(tmap_k, tmap_w1, p, mp);
  }
  return check_launch("psi_tc_kernel");
}

int launch_psi_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s) {
  PtMap mp;
  mp.w2 = p.w_psi2; mp.w3 = p.w_psi3; mp.out = p.a.ws_psi; mp.pmax = p.a.ws_pmax; mp.is_phi = 0;
  return launch_map_tc(c, p, G, s, p.K, p.w_psi1, mp);
}

// phi(q_i) of every row of Q into `out` [Iw][Sp][R] (one query head per KV head)
int launch_phi_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s, float* out) {
  PtMap mp;
  mp.w2 = (const __half*)c->w.w_phi2; mp.w3 = nullptr; mp.out = out; mp.pmax = nullptr; mp.is_phi = 1;
  return launch_map_tc(c, p, G, s, p.Q, c->w.w_phi1, mp);
}

}  // namespace less
