// Feature maps phi(q_t), psi(k_t) of one decode step (Eq. 1, Eq. 2) on the
// tensor cores, for every batch size:
//     phi(q) = | gelu( gelu(q W1) W2 ) |        psi(k) = | c2 gelu( c1 gelu(k W1) W2 ) W3 |
//
// The step is bound by reading each head's weights from HBM once, so the kernel
// is a weight stream: persistent CTAs (one per SM) walk a list of work items
// (layer-head, map, token tile); a producer thread streams the item's W1 in
// 32-KB chunks of 128 hidden units through a shared-memory ring with TMA.
//
// GEMM1 is computed transposed, hidden units on the accumulator's 128 lanes and
// tokens on its columns:
//     D1^T[128 hidden x n tokens] = W1[:, chunk]^T (A, M-major, as it lies in HBM)
//                                   * X^T           (B, K-major, n = tokens padded to 16..128)
// so the GELU work of the epilogue grows with the number of tokens, not with the
// 128-row tile, and a batch of one costs one GELU per thread and chunk.
// Epilogue warps (two per lane quadrant) read D1^T from tensor memory, apply
// c1 * gelu, split the result into fp16 hi + lo (one fp16 rounding of the hidden
// layer would cost ~2e-3 on psi) and store it, tokens contiguous, as the M-major
// A operand of
//     D2[tokens x 16] += H[tokens x 128 hidden] * W2[chunk rows, :]       (GEMM2)
// whose accumulator lives in tensor memory across the chunks.  After the last
// chunk: c2 * gelu, W3 (psi only) and the absolute value on CUDA cores.
// The hidden activations never leave the SM (the paper's "absorbed activation",
// Section 3.2, taken to the whole MLP).  No multicast; every wait is bounded.
#include "feature_gemv.cuh"
#include "tc_common.cuh"

namespace less {

constexpr int FT_EPI_WARPS = 8;
constexpr int FT_EPI_THREADS = FT_EPI_WARPS * 32;
constexpr int FT_THREADS = 64 + FT_EPI_THREADS;   // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue
constexpr int FT_CHUNK = 128;                     // hidden units per GEMM1
constexpr int FT_STAGE_BYTES = FT_CHUNK * kHeadDim * 2;
constexpr int FT_MAX_STAGES = 6;
constexpr int FT_SMEM_LIMIT = 232448;             // 227 KB per CTA

struct FtShared {
  uint64_t full[FT_MAX_STAGES], empty[FT_MAX_STAGES];
  uint64_t aux_full[2], aux_empty[2];
  uint64_t d1_full[2], d1_free[2];
  uint64_t hid_full, hid_free;
  uint64_t d2_full, d2_free;
  uint32_t tmem_base;
  int abort;
  __align__(16) __half w3[2][16 * 16];
};

__device__ __forceinline__ void ft_wait(uint64_t* bar, uint32_t parity, volatile int* abort, int32_t* status,
                                        int where) {
  if (*abort) return;
  if (!mbar_wait(bar, parity)) {
    *abort = 1;
    set_status(status, kStatusTimeout, where);
  }
}

struct FtGeom {
  int npad;        // tokens per tile (GEMM1 N): 16, 32, 64 or 128
  int ntile;       // token tiles per (layer-head, map)
  int items;       // work items
  int nstage;      // ring stages
  uint32_t tmem_cols;
};

template <int R>
__global__ void __launch_bounds__(FT_THREADS) feature_tc_kernel(
    const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
    const __grid_constant__ CUtensorMap tm_w1phi, const __grid_constant__ CUtensorMap tm_w1psi,
    const __grid_constant__ CUtensorMap tm_w2phi, const __grid_constant__ CUtensorMap tm_w2psi, FmParams p,
    FtGeom gm, int32_t* status) {
  extern __shared__ __align__(1024) unsigned char ft_smem[];
  const int Rp = p.Rp, nchunk = Rp / FT_CHUNK, npad = gm.npad, nstage = gm.nstage;
  const uint32_t hbytes = (uint32_t)npad * 256;      // hi (or lo): npad/8 token blocks x 2 KB
  const uint32_t xbytes = (uint32_t)npad * 256;      // two 64-column halves of npad rows x 128 B
  const uint32_t w2bytes = (uint32_t)Rp * R * 2;
  unsigned char* hbuf = ft_smem;                     // hi, then lo
  unsigned char* xbuf = hbuf + 2 * hbytes;           // [2][xbytes]
  unsigned char* ring = xbuf + 2 * xbytes;           // [nstage][32 KB]
  unsigned char* w2buf = ring + (size_t)nstage * FT_STAGE_BYTES;   // [2][R/8 column blocks][Rp rows][16 B]
  FtShared* sh = reinterpret_cast<FtShared*>(w2buf + 2 * w2bytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < nstage; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh->aux_full[s], 1);
      mbar_init(&sh->aux_empty[s], 1 + FT_EPI_WARPS);
      mbar_init(&sh->d1_full[s], 1);
      mbar_init(&sh->d1_free[s], FT_EPI_THREADS);
    }
    mbar_init(&sh->hid_full, FT_EPI_THREADS);
    mbar_init(&sh->hid_free, 1);
    mbar_init(&sh->d2_full, 1);
    mbar_init(&sh->d2_free, FT_EPI_THREADS);
    // a CTA that starts after another one has given up skips every wait: the grid drains at once
    sh->abort = *reinterpret_cast<volatile int32_t*>(status) != 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&sh->tmem_base, gm.tmem_cols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh->tmem_base;
  const uint32_t d2col = 2u * (uint32_t)npad;
  volatile int* abortp = &sh->abort;
  const int my_items = blockIdx.x < gm.items ? (gm.items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      uint32_t g = 0;
      for (int n = 0; n < my_items; ++n) {
        const int it = blockIdx.x + n * gridDim.x;
        const int tile = it % gm.ntile, which = (it / gm.ntile) & 1, lh = it / (2 * gm.ntile);
        const int a = n & 1;
        ft_wait(&sh->aux_empty[a], ((n >> 1) & 1) ^ 1, abortp, status, 40);
        if (*abortp) break;
        const CUtensorMap* tx = which ? &tm_k : &tm_q;
        const CUtensorMap* tw1 = which ? &tm_w1psi : &tm_w1phi;
        const CUtensorMap* tw2 = which ? &tm_w2psi : &tm_w2phi;
        mbar_expect_tx(&sh->aux_full[a], xbytes + w2bytes + (which ? R * R * 2 : 0));
        unsigned char* xa = xbuf + a * xbytes;
        tma_load_2d(xa, tx, lh * kHeadDim, tile * npad, &sh->aux_full[a]);
        tma_load_2d(xa + xbytes / 2, tx, lh * kHeadDim + 64, tile * npad, &sh->aux_full[a]);
        const int wrows = Rp < 256 ? Rp : 256;           // rows per W2 box
        for (int nb = 0; nb < R / 8; ++nb)
          for (int r0 = 0; r0 < Rp; r0 += wrows)
            tma_load_2d(w2buf + a * w2bytes + ((size_t)nb * Rp + r0) * 16, tw2, nb * 8, lh * Rp + r0,
                        &sh->aux_full[a]);
        if (which) bulk_g2s(&sh->w3[a][0], p.w3 + (size_t)lh * R * R, R * R * 2, &sh->aux_full[a]);
        for (int c = 0; c < nchunk; ++c, ++g) {
          const int s = g % nstage;
          ft_wait(&sh->empty[s], ((g / nstage) & 1) ^ 1, abortp, status, 41);
          if (*abortp) break;
          mbar_expect_tx(&sh->full[s], FT_STAGE_BYTES);
          unsigned char* st = ring + (size_t)s * FT_STAGE_BYTES;
          tma_load_2d(st, tw1, c * FT_CHUNK, lh * kHeadDim, &sh->full[s]);
          tma_load_2d(st + FT_STAGE_BYTES / 2, tw1, c * FT_CHUNK + 64, lh * kHeadDim, &sh->full[s]);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0 && my_items > 0) {
      const uint32_t idesc1 = idesc_f16(128, npad, 1, 0);   // A = W1 chunk (M-major), B = x rows (K-major)
      constexpr uint32_t idesc2 = idesc_f16(128, 16, 1, 1); // A = hidden (M-major), B = W2 (N-major)
      const uint32_t ring_a = smem_u32(ring), x_a = smem_u32(xbuf), h_a = smem_u32(hbuf), w2_a = smem_u32(w2buf);
      const uint32_t Q = (uint32_t)my_items * nchunk;
      auto issue_gemm1 = [&](uint32_t qq) {
        const uint32_t n = qq / nchunk, c = qq % nchunk, a = n & 1, s = qq % nstage, b = qq & 1;
        if (c == 0) ft_wait(&sh->aux_full[a], (n >> 1) & 1, abortp, status, 42);
        ft_wait(&sh->full[s], (qq / nstage) & 1, abortp, status, 43);
        ft_wait(&sh->d1_free[b], ((qq >> 1) & 1) ^ 1, abortp, status, 44);
        if (*abortp) return;
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < kHeadDim / 16; ++ks) {
          const uint64_t ad = smem_desc(ring_a + s * FT_STAGE_BYTES + ks * 2048, FT_STAGE_BYTES / 2, 1024, kLayoutSw128);
          const uint64_t bd =
              smem_desc(x_a + a * xbytes + (ks >> 2) * (xbytes / 2) + (ks & 3) * 32, 16, 1024, kLayoutSw128);
          mma_f16_ss(tmem + b * npad, ad, bd, idesc1, ks ? 1u : 0u);
        }
        mma_commit(&sh->empty[s]);
        mma_commit(&sh->d1_full[b]);
      };
      issue_gemm1(0);
      for (uint32_t q = 0; q < Q && !*abortp; ++q) {
        if (q + 1 < Q) issue_gemm1(q + 1);
        const uint32_t n = q / nchunk, c = q % nchunk, a = n & 1;
        if (c == 0) ft_wait(&sh->d2_free, (n & 1) ^ 1, abortp, status, 45);
        ft_wait(&sh->hid_full, q & 1, abortp, status, 46);
        if (*abortp) break;
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < FT_CHUNK / 16; ++ks) {
          // R = 8 fills one 8-column block; the second block of the N = 16 tile then only has to
          // lie inside this CTA's shared memory (its columns of D2 are never read)
          const uint64_t bd = smem_desc(w2_a + a * w2bytes + (c * FT_CHUNK + ks * 16) * 16, 128,
                                        R == 16 ? (uint32_t)Rp * 16 : 128u, kLayoutNone);
          const uint64_t ah = smem_desc(h_a + ks * 256, 128, 2048, kLayoutNone);
          const uint64_t al = smem_desc(h_a + hbytes + ks * 256, 128, 2048, kLayoutNone);
          mma_f16_ss(tmem + d2col, ah, bd, idesc2, (c | ks) ? 1u : 0u);
          mma_f16_ss(tmem + d2col, al, bd, idesc2, 1u);
        }
        mma_commit(&sh->hid_free);
        if (c == (uint32_t)nchunk - 1) {
          mma_commit(&sh->d2_full);
          mma_commit(&sh->aux_empty[a]);
        }
      }
    }
  } else {
    // ---------------- epilogue warps ----------------
    const int ew = warp - 2;                   // 0..7
    const int quad = warp & 3;                 // tensor-memory lane quadrant this warp may read
    const int hf = ew >> 2;                    // which half of the token blocks
    const int j = quad * 32 + lane;            // hidden unit inside the chunk = accumulator lane
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    unsigned char* hrow = hbuf + (j >> 3) * 128 + (j & 7) * 16;
    uint32_t q = 0;
    for (int n = 0; n < my_items && !*abortp; ++n) {
      const int it = blockIdx.x + n * gridDim.x;
      const int tile = it % gm.ntile, which = (it / gm.ntile) & 1, lh = it / (2 * gm.ntile);
      const int a = n & 1;
      const int b0 = tile * npad, nb = min(npad, p.B - b0), nblk = (nb + 7) >> 3;
      float c1 = 1.f, c2 = 1.f;
      if (which && p.psi_scale) { c1 = __ldg(p.psi_scale + lh * 2); c2 = __ldg(p.psi_scale + lh * 2 + 1); }
      for (int c = 0; c < nchunk && !*abortp; ++c, ++q) {
        const int b = q & 1;
        ft_wait(&sh->d1_full[b], (q >> 1) & 1, abortp, status, 47);
        tc_fence_after_sync();
        // this warp's token blocks: hf, hf + 2, ...   (at most 8 of the 16 blocks of a 128-token tile)
        uint32_t acc[8][8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int blk = hf + 2 * i;
          if (blk < nblk) tmem_ld8(lane_addr + b * npad + blk * 8, acc[i]);
        }
        tmem_ld_wait();
        tc_fence_before_sync();
        mbar_arrive(&sh->d1_free[b]);
        uint4 hi[8], lo[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int blk = hf + 2 * i;
          if (blk < nblk) {
            uint32_t ph[4], pl[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float h0 = c1 * gelu_erf(__uint_as_float(acc[i][2 * e]));
              const float h1 = c1 * gelu_erf(__uint_as_float(acc[i][2 * e + 1]));
              const __half2 hh = __floats2half2_rn(h0, h1);
              const float2 hf2 = __half22float2(hh);
              const __half2 ll = __floats2half2_rn(h0 - hf2.x, h1 - hf2.y);
              ph[e] = *reinterpret_cast<const uint32_t*>(&hh);
              pl[e] = *reinterpret_cast<const uint32_t*>(&ll);
            }
            hi[i] = make_uint4(ph[0], ph[1], ph[2], ph[3]);
            lo[i] = make_uint4(pl[0], pl[1], pl[2], pl[3]);
          }
        }
        ft_wait(&sh->hid_free, (q & 1) ^ 1, abortp, status, 48);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int blk = hf + 2 * i;
          if (blk < nblk) {
            *reinterpret_cast<uint4*>(hrow + blk * 2048) = hi[i];
            *reinterpret_cast<uint4*>(hrow + hbytes + blk * 2048) = lo[i];
          }
        }
        fence_proxy_async_smem();
        mbar_arrive(&sh->hid_full);
      }
      if (*abortp) break;
      // ---- layer 2 result: token = accumulator lane ----
      ft_wait(&sh->d2_full, n & 1, abortp, status, 49);
      tc_fence_after_sync();
      const bool mine = hf == 0 && quad * 32 < nb;         // warp-uniform
      uint32_t g2[16];
      if (mine) {
#pragma unroll
        for (int r8 = 0; r8 < R / 8; ++r8) tmem_ld8(lane_addr + d2col + r8 * 8, g2 + r8 * 8);
        tmem_ld_wait();
      }
      tc_fence_before_sync();
      mbar_arrive(&sh->d2_free);
      if (mine && j < nb) {
        float gv[R], out[R];
#pragma unroll
        for (int r = 0; r < R; ++r) gv[r] = c2 * gelu_erf(__uint_as_float(g2[r]));
        if (which) {
          const __half* w3 = &sh->w3[a][0];
#pragma unroll
          for (int r = 0; r < R; ++r) {
            float s = 0.f;
#pragma unroll
            for (int rr = 0; rr < R; ++rr) s = fmaf(gv[rr], __half2float(w3[rr * R + r]), s);
            out[r] = fabsf(s);
          }
        } else {
#pragma unroll
          for (int r = 0; r < R; ++r) out[r] = fabsf(gv[r]);
        }
        float4* dst = reinterpret_cast<float4*>(p.out[which] + ((size_t)(b0 + j) * p.L * p.Hd + lh) * R);
#pragma unroll
        for (int r4 = 0; r4 < R / 4; ++r4) dst[r4] = make_float4(out[r4 * 4], out[r4 * 4 + 1], out[r4 * 4 + 2], out[r4 * 4 + 3]);
      }
      // this warp is done with the item's W3
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->aux_empty[a]);
    }
  }
  drain_after_abort(abortp);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, gm.tmem_cols);
}

bool feature_tc_supported(const Dims& d) {
  return (d.Rp == 128 || d.Rp == 256 || d.Rp == 512) && encode_tiled_fn() != nullptr;
}

static size_t ft_fixed_smem(const Dims& d, int npad) {
  return (size_t)4 * npad * 256 + (size_t)2 * d.Rp * d.R * 2 + sizeof(FtShared) + 1024;
}

int launch_feature_tc(less_ctx* c, const FmParams& p, cudaStream_t s) {
  const Dims& d = c->d;
  FtGeom gm;
  const int bt = d.B < 128 ? d.B : 128;
  gm.npad = bt <= 16 ? 16 : bt <= 32 ? 32 : bt <= 64 ? 64 : 128;
  gm.ntile = (d.B + gm.npad - 1) / gm.npad;
  gm.items = d.L * d.Hd * 2 * gm.ntile;
  const size_t fixed = ft_fixed_smem(d, gm.npad);
  int ns = (int)((FT_SMEM_LIMIT - fixed) / FT_STAGE_BYTES);
  gm.nstage = ns > FT_MAX_STAGES ? FT_MAX_STAGES : ns;
  if (gm.nstage < 2) return LESS_ERR_INVALID_CONFIG;
  const uint32_t need = 2u * gm.npad + 16u;
  gm.tmem_cols = need <= 64 ? 64 : need <= 128 ? 128 : need <= 256 ? 256 : 512;
  const size_t smem = fixed + (size_t)gm.nstage * FT_STAGE_BYTES;

  CUtensorMap tq, tk, tw1a, tw1b, tw2a, tw2b;
  const uint64_t lh = (uint64_t)d.L * d.Hd;
  // q, k: [B rows][L*Hd*128 columns]; a box is npad batch rows x 64 columns of one head
  if (!make_tmap_f16_2d(&tq, p.x[0], d.B, lh * kHeadDim, lh * kHeadDim * 2, gm.npad) ||
      !make_tmap_f16_2d(&tk, p.x[1], d.B, lh * kHeadDim, lh * kHeadDim * 2, gm.npad))
    return fail_cuda("tensor map of q / k");
  if (!make_tmap_f16_2d(&tw1a, p.w1[0], lh * kHeadDim, d.Rp, (uint64_t)d.Rp * 2, kHeadDim) ||
      !make_tmap_f16_2d(&tw1b, p.w1[1], lh * kHeadDim, d.Rp, (uint64_t)d.Rp * 2, kHeadDim))
    return fail_cuda("tensor map of W1");
  const uint32_t wrows = d.Rp < 256 ? d.Rp : 256;
  if (!make_tmap_f16_2d_box(&tw2a, p.w2[0], lh * d.Rp, d.R, (uint64_t)d.R * 2, wrows, 8, false) ||
      !make_tmap_f16_2d_box(&tw2b, p.w2[1], lh * d.Rp, d.R, (uint64_t)d.R * 2, wrows, 8, false))
    return fail_cuda("tensor map of W2");

  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
  const int grid = gm.items < sms ? gm.items : sms;
  LaunchScope scope(c, LESS_KERNEL_FEATURE_MAP, s);
  if (d.R == 8) {
    if (cudaFuncSetAttribute(feature_tc_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return fail_cuda("shared memory opt-in of feature_tc_kernel");
    feature_tc_kernel<8><<<grid, FT_THREADS, smem, s>>>(tq, tk, tw1a, tw1b, tw2a, tw2b, p, gm, c->a.status);
  } else {
    if (cudaFuncSetAttribute(feature_tc_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return fail_cuda("shared memory opt-in of feature_tc_kernel");
    feature_tc_kernel<16><<<grid, FT_THREADS, smem, s>>>(tq, tk, tw1a, tw1b, tw2a, tw2b, p, gm, c->a.status);
  }
  return check_launch("feature_tc_kernel");
}

}  // namespace less
