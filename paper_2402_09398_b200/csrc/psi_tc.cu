// psi(k_j) of every prompt token on the tensor cores (Eq. 2), fused with the prompt state build
// (Eq. 4 / Eq. 5 summed over the discarded set D_1):
//     psi(k) = | c2 * gelu( c1 * gelu(k W1) W2 ) W3 |,   H^T[D x R] = V_ev^T psi(K_ev),   z = 1^T psi(K_ev)
//
// One CTA = one token split of one instance; W1 of the instance's head (128 KB) stays in shared
// memory for all of the split's tiles.  Per 128-token tile:
//   GEMM1  D1[128 tok x 128] = Ktile[128 x 128] * W1[:, chunk]      chunks of 128 hidden units, D1
//                                                                   double-buffered in tensor memory
//   epilogue warps: tcgen05.ld 32 columns of D1 -> gelu -> fp16 hi + lo (a single fp16 rounding of the
//                   hidden layer costs ~2e-3 on individual psi vectors) -> tcgen05.st back over the
//                   same 32 columns of D1 (16 packed columns hi, 16 lo)
//   GEMM2  G2[128 x 16] += hidden[128 x 128] * W2[chunk rows, :]    A operand read from tensor memory,
//                                                                   so the hidden layer never touches shared memory
//   after the last chunk: tcgen05.ld G2 -> c2 * gelu(c1 * .) -> W3 on CUDA cores -> abs -> psi[token][R]
// With kState the tile's psi goes straight into the state build: rows of kept (or out-of-range)
// tokens are zeroed, the rest is scaled by a power of two taken from the tile's own maximum (so that
// fp16's range never matters, whatever the magnitude of the trained maps), split into fp16 hi + lo
// and laid out as the B operand of
//   Ht[128 dims x 2R] = Vtile^T[128 dims x 128 tok] * psi_hi|lo[128 tok x 2R]   (A = V tile by TMA, M-major)
//   Zt[128 x 2R]      = ones[128 x 128 tok] * psi_hi|lo                         (every row = the tile's z)
// into a fresh accumulator per tile; four warps read it back, undo the tile's scale (exact) and add
// it to fp32 registers that hold the split's H^T and z.  psi itself is written out only for kept
// tokens (their slots cache it).  finalize_kernel sums the splits in a fixed order.
// Without kState the kernel writes psi of every token and the instance's maximum (the parallel
// form), or evaluates phi(q) = | gelu( gelu(q W1) W2 ) | (Eq. 1) over rows of Q (PtMap::is_phi).
// Roles: warps 0-15 epilogue (lane quadrant = warp & 3, token row = tensor-memory lane; the four
// warps of a quadrant split a chunk's 128 columns), warp 16 TMA producer, warp 17 issues GEMM1,
// warp 18 GEMM2, warp 19 the state products.  Plain TMA tiled loads with the 128-byte swizzle.
// Every wait is bounded.
#include "prefill.cuh"
#include "tc_common.cuh"

namespace less {

constexpr int PT_WORKERS = 512;                    // 16 epilogue warps: four per tensor-memory lane quadrant
constexpr int PT_THREADS = PT_WORKERS + 128;       // + TMA producer, GEMM1, GEMM2 and state-product issuers: a warp each (two
                                                   // issuers in one warp would block each other in their waits)
constexpr int PT_TILE = 128;                       // tokens per tile
constexpr int PT_CHUNK = 128;                      // hidden units per GEMM1 chunk (64 when the hidden width is 64)
constexpr int PT_KBYTES = PT_TILE * kHeadDim * 2;  // one K (or V) tile
constexpr int PT_W2N = 16;                         // GEMM2 N (R padded to 16)
// tensor-memory columns: three D1 buffers of 128, G2 at 384, the per-tile state accumulators (H^T, then
// z 32 columns on) behind.  Three D1 buffers, not two: the chain "GEMM2 reads the hidden layer of chunk
// q - 1, GEMM1 refills that buffer" takes about as long as the epilogue of one chunk (a thread gets
// an MMA out every ~84 cycles), so with two buffers the epilogue warps waited for it at every chunk.
constexpr int PT_D1BUFS = 3;
constexpr uint32_t PT_G2COL = 384, PT_HCOL = 416, PT_TMEM = 512;

struct PtShared {
  uint64_t w1_full;
  uint64_t k_full, k_empty;
  uint64_t v_full, v_empty;
  uint64_t d1_full[PT_D1BUFS], d1_free[PT_D1BUFS];
  uint64_t hid_full[PT_D1BUFS];   // per D1 buffer: a warp cannot arrive for the buffer's next use before this one is consumed
  uint64_t g2_full, g2_free;
  uint64_t b_full, b_free;
  uint64_t h_full, h_free;
  uint64_t mx_bar;        // the four finishing warps meet here twice per tile
  uint32_t tmem_base;
  int abort;
  float w3[16 * 16];
  float c1, c2;
  float wmax[4];          // per quadrant: largest psi of the tile that enters the state
  float inv_scale[2];     // per state accumulator buffer: 1 / the tile's scale
  float zacc[16];         // the split's z (one thread adds a tile's z at a time)
};

__device__ __forceinline__ void pt_wait(uint64_t* bar, uint32_t parity, volatile int* abort, int32_t* status,
                                        int where) {
  if (mbar_try_wait(bar, parity)) return;
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

// gelu of two accumulator values -> fp16 hi pair, fp16 lo pair
__device__ __forceinline__ void gelu_split(uint32_t a0, uint32_t a1, uint32_t& hi, uint32_t& lo) {
  // c1 multiplies the layer-2 sums instead (same value): the fp16 hi + lo operand then never
  // depends on how small the learnable scalar is (the paper initialises it to 1e-4)
  float h0, h1;
  gelu_erf2(__uint_as_float(a0), __uint_as_float(a1), h0, h1);
  const __half2 hh = __floats2half2_rn(h0, h1);
  const float2 hf = __half22float2(hh);
  const __half2 ll = __floats2half2_rn(h0 - hf.x, h1 - hf.y);
  hi = *reinterpret_cast<const uint32_t*>(&hh);
  lo = *reinterpret_cast<const uint32_t*>(&ll);
}

template <int R, bool kState>
__global__ void __launch_bounds__(PT_THREADS) psi_tc_kernel(const __grid_constant__ CUtensorMap tmap_k,
                                                            const __grid_constant__ CUtensorMap tmap_v,
                                                            const __grid_constant__ CUtensorMap tmap_w1,
                                                            PfParams p, PtMap mp) {
  constexpr int NB = 2 * R;                          // state B operand: hi | lo columns
  constexpr uint32_t B_SBO = 128;                    // between 8-column blocks
  constexpr uint32_t B_LBO = (NB / 8) * 128;         // between 8-token groups
  extern __shared__ __align__(1024) unsigned char pt_smem[];
  if (smem_misaligned(pt_smem, p.a.status, 29)) return;
  const int Rp = p.Rp;
  const int chunk = Rp < PT_CHUNK ? Rp : PT_CHUNK;   // hidden units per chunk
  const int nchunk = Rp / chunk;
  const int cparts = chunk / 32;                     // epilogue warps per quadrant with work (4, or 2 at width 64)
  unsigned char* w1s = pt_smem;                                  // [Rp/64][128 k][64 n]  (16 KB each)
  unsigned char* kbuf = w1s + (size_t)(Rp / 64) * 16384;         // [2 kblocks][128 tok][64]
  unsigned char* w2s = kbuf + PT_KBYTES;                         // [Rp/8][2 nblocks][8 k][8 n] fp16
  unsigned char* vbuf = w2s + (size_t)Rp * PT_W2N * 2;           // kState: [2 dblocks][128 tok][64]
  unsigned char* bbuf = vbuf + (kState ? PT_KBYTES : 0);         // kState: psi hi | lo as B operand
  __half* ones = reinterpret_cast<__half*>(bbuf + (kState ? PT_TILE * NB * 2 : 0));   // kState: 4 KB of 1.0
  PtShared* sh = reinterpret_cast<PtShared*>(reinterpret_cast<unsigned char*>(ones) + (kState ? 4096 : 0));

  const int tid = threadIdx.x, warp = tid >> 5;
  const int split = blockIdx.x, g = blockIdx.y;
  // phi belongs to the query head: g then counts query heads (grp per KV instance), each with its own
  // rows of Q and its own weights
  InstMap im = map_instance(p, mp.is_phi ? g / p.grp : g);
  if (mp.is_phi) {
    im.in_row0 = map_query(p, g).q_row0;
    im.lh = im.lh * p.grp + g % p.grp;
  }
  const int jbeg = split * p.split_tokens, jend = min(p.S, jbeg + p.split_tokens);
  const int ntiles = (jend - jbeg + PT_TILE - 1) / PT_TILE;

  if (tid == 0) {
    mbar_init(&sh->w1_full, 1);
    mbar_init(&sh->k_full, 1);
    mbar_init(&sh->k_empty, 1);
    mbar_init(&sh->v_full, 1);
    mbar_init(&sh->v_empty, 1);
    for (int s = 0; s < PT_D1BUFS; ++s) {
      mbar_init(&sh->d1_full[s], 1);
      mbar_init(&sh->d1_free[s], 1);
      mbar_init(&sh->hid_full[s], PT_WORKERS / 32);
    }
    mbar_init(&sh->h_full, 1);
    mbar_init(&sh->h_free, 4);
    mbar_init(&sh->g2_full, 1);
    mbar_init(&sh->g2_free, 4);
    mbar_init(&sh->b_full, 4);
    mbar_init(&sh->b_free, 1);
    mbar_init(&sh->mx_bar, 4);
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
    if (kState)
      for (int e = tid; e < 2048; e += PT_THREADS) ones[e] = __float2half(1.0f);
  }
  if (warp == PT_WORKERS / 32 + 1) tmem_alloc(&sh->tmem_base, PT_TMEM);
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
      mbar_expect_tx(&sh->w1_full, (uint32_t)(Rp / 64) * 16384);
      for (int c = 0; c < Rp / 64; ++c)
        tma_load_2d(w1s + (size_t)c * 16384, &tmap_w1, c * 64, im.lh * kHeadDim, &sh->w1_full);
      for (int i = 0; i < ntiles; ++i) {
        const int row = (int)(im.in_row0 + jbeg + (size_t)i * PT_TILE);
        pt_wait(&sh->k_empty, (i & 1) ^ 1, abortp, status, 30);
        if (*abortp) break;                      // issue nothing more once the CTA has given up
        mbar_expect_tx(&sh->k_full, PT_KBYTES);
        tma_load_2d_hint(kbuf, &tmap_k, 0, row, &sh->k_full, stream_policy);
        tma_load_2d_hint(kbuf + PT_KBYTES / 2, &tmap_k, 64, row, &sh->k_full, stream_policy);
        if (kState) {
          pt_wait(&sh->v_empty, (i & 1) ^ 1, abortp, status, 39);
          if (*abortp) break;
          mbar_expect_tx(&sh->v_full, PT_KBYTES);
          tma_load_2d_hint(vbuf, &tmap_v, 0, row, &sh->v_full, stream_policy);
          tma_load_2d_hint(vbuf + PT_KBYTES / 2, &tmap_v, 64, row, &sh->v_full, stream_policy);
        }
      }
    }
  } else if (warp == PT_WORKERS / 32 + 1) {
    // ---------------- MMA issuer of GEMM1 ----------------
    // One issuing thread per product: a single thread gets an MMA out every ~84 cycles, and the streams
    // only meet at the barriers they need anyway.
    if (tid == PT_WORKERS + 32) {
      const uint32_t idesc1 = idesc_f16(128, chunk, 0, 1);          // A = K tile (K-major), B = W1 (N-major)
      const uint32_t w1a = smem_u32(w1s);
      pt_wait(&sh->w1_full, 0, abortp, status, 31);
      uint32_t b = 0, bph = 0;                                      // D1 buffer of the chunk and its phase: counted
      for (int i = 0; i < ntiles && !*abortp; ++i) {
        pt_wait(&sh->k_full, i & 1, abortp, status, 33);
        const uint32_t ka = smem_u32(kbuf);
        for (int c = 0; c < nchunk && !*abortp; ++c, (++b == PT_D1BUFS ? (b = 0, bph ^= 1) : 0u)) {
          pt_wait(&sh->d1_free[b], bph ^ 1, abortp, status, 32);   // GEMM2 has read the hidden layer this buffer held before
          if (*abortp) break;
          tc_fence_after_sync();
#pragma unroll
          for (int ks = 0; ks < kHeadDim / 16; ++ks) {
            const uint64_t ad = smem_desc(ka + (ks >> 2) * (PT_KBYTES / 2) + (ks & 3) * 32, 16, 1024, kLayoutSw128);
            // B: [128 k][chunk n], 64-column blocks 16 KB apart
            const uint64_t bd = smem_desc(w1a + c * (chunk / 64) * 16384 + ks * 2048, 16384, 1024, kLayoutSw128);
            mma_f16_ss(tmem + b * 128, ad, bd, idesc1, ks ? 1u : 0u);
          }
          mma_commit(&sh->d1_full[b]);
        }
        mma_commit(&sh->k_empty);                                   // all GEMM1s of this tile are issued
      }
    }
  } else if (warp == PT_WORKERS / 32 + 2) {
    // ---------------- MMA issuer of GEMM2: A = hidden hi / lo in tensor memory ----------------
    if (tid == PT_WORKERS + 64) {
      constexpr uint32_t idesc2 = idesc_f16(128, PT_W2N, 0, 1);     // A = hidden (tensor memory), B = W2 (N-major)
      const uint32_t w2a = smem_u32(w2s);
      uint32_t b = 0, bph = 0;
      for (int i = 0; i < ntiles && !*abortp; ++i) {
        for (int c = 0; c < nchunk; ++c, (++b == PT_D1BUFS ? (b = 0, bph ^= 1) : 0u)) {
          if (c == 0) pt_wait(&sh->g2_free, (i & 1) ^ 1, abortp, status, 34);
          pt_wait(&sh->hid_full[b], bph, abortp, status, 35);
          if (*abortp) break;
          tc_fence_after_sync();
          // part w of the chunk: hidden units 32 w .. 32 w + 31 sit in D1 columns 32 w .. 32 w + 31 as
          // 16 packed columns of hi, then 16 of lo; a k-step of 16 units is 8 packed columns
          for (int w = 0; w < cparts; ++w) {
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
              const uint64_t bd = smem_desc(w2a + ((c * chunk + w * 32 + ks * 16) >> 3) * 256, 256, 128, kLayoutNone);
              const uint32_t acol = tmem + b * 128 + w * 32 + ks * 8;
              mma_f16_ts(tmem + PT_G2COL, acol, bd, idesc2, (c | w | ks) ? 1u : 0u);
              mma_f16_ts(tmem + PT_G2COL, acol + 16, bd, idesc2, 1u);
            }
          }
          mma_commit(&sh->d1_free[b]);
        }
        if (*abortp) break;
        mma_commit(&sh->g2_full);
      }
    }
  } else if (warp == PT_WORKERS / 32 + 3) {
    // ---------------- MMA issuer of the state products ----------------
    if (kState && tid == PT_WORKERS + 96) {
      constexpr uint32_t idesc_h = idesc_f16(128, NB, 1, 1);   // A = V tile (M-major), B = psi (N-major)
      constexpr uint32_t idesc_z = idesc_f16(128, NB, 0, 1);   // A = ones (K-major)
      const uint32_t ones_addr = smem_u32(ones), va = smem_u32(vbuf), ba = smem_u32(bbuf);
      for (int i = 0; i < ntiles; ++i) {
        pt_wait(&sh->v_full, i & 1, abortp, status, 21);
        pt_wait(&sh->b_full, i & 1, abortp, status, 22);
        pt_wait(&sh->h_free, (i & 1) ^ 1, abortp, status, 23);      // the tile before has been collected
        if (*abortp) break;
        tc_fence_after_sync();
        const uint32_t hcol = tmem + PT_HCOL;
#pragma unroll
        for (int ks = 0; ks < PT_TILE / 16; ++ks) {
          const uint64_t bd = smem_desc(ba + ks * 2 * B_LBO, B_LBO, B_SBO, kLayoutNone);
          const uint64_t ad = smem_desc(va + ks * 2048, PT_KBYTES / 2, 1024, kLayoutSw128);
          mma_f16_ss(hcol, ad, bd, idesc_h, ks ? 1u : 0u);
          const uint64_t od = smem_desc(ones_addr, 128, 256, kLayoutNone);
          mma_f16_ss(hcol + 32, od, bd, idesc_z, ks ? 1u : 0u);
        }
        mma_commit(&sh->v_empty);
        mma_commit(&sh->b_free);
        mma_commit(&sh->h_full);
      }
    }
  } else {
    // ---------------- epilogue workers ----------------
    const float c1 = sh->c1, c2 = sh->c2;
    const int quad = warp & 3, part = warp >> 2;       // part: which 32 columns of a chunk
    const int lane = tid & 31;
    const int row = quad * 32 + lane;                  // token row of the tile = tensor-memory lane
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    float* psi = mp.out + (size_t)g * p.Sp * R;
    const int32_t* slot_of = p.a.ws_slot + (size_t)g * p.Sp;
    float pmax = 0.f;                                  // largest psi this thread has produced
    float hacc[kState ? R : 1];                        // part 1: column `row` of the split's H^T
#pragma unroll
    for (int r = 0; r < (kState ? R : 1); ++r) hacc[r] = 0.f;
    if (kState && part == 1 && row < R) sh->zacc[row] = 0.f;   // lanes of one warp (quadrant 0, part 1), which alone touches it afterwards
    __syncwarp();
    // the tile whose state products part 1 still has to collect
    auto collect = [&](int i) {
      pt_wait(&sh->h_full, i & 1, abortp, status, 24);
      tc_fence_after_sync();
      uint32_t hv[NB];
      const uint32_t hcol = lane_addr + PT_HCOL;
      const float inv = sh->inv_scale[i & 1];          // exact: a power of two
      if (NB == 32) tmem_ld32(hcol, hv); else tmem_ld16(hcol, hv);
      tmem_ld_wait();
#pragma unroll
      for (int r = 0; r < R; ++r) hacc[r] = fmaf(__uint_as_float(hv[r]) + __uint_as_float(hv[R + r]), inv, hacc[r]);
      if (quad == 0) {                                 // every row of the z accumulator holds the tile's z: lane 0 keeps the sum
        if (NB == 32) tmem_ld32(hcol + 32, hv); else tmem_ld16(hcol + 32, hv);
        tmem_ld_wait();
        if (lane == 0) {
#pragma unroll
          for (int r = 0; r < R; ++r) sh->zacc[r] = fmaf(__uint_as_float(hv[r]) + __uint_as_float(hv[R + r]), inv, sh->zacc[r]);
        }
      }
      tc_fence_before_sync();
      mbar_arrive_warp(&sh->h_free);
    };
    uint32_t b = 0, bph = 0;                           // D1 buffer of the chunk and its phase: counted
    for (int i = 0; i < ntiles && !*abortp; ++i) {
      for (int c = 0; c < nchunk && !*abortp; ++c, (++b == PT_D1BUFS ? (b = 0, bph ^= 1) : 0u)) {
        if (part < cparts) {
          pt_wait(&sh->d1_full[b], bph, abortp, status, 36);
          tc_fence_after_sync();
          uint32_t acc[32], hi[16], lo[16];              // this warp's 32 of the chunk's columns
          const uint32_t col = lane_addr + b * 128 + part * 32;
          tmem_ld32(col, acc);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 16; ++e) gelu_split(acc[2 * e], acc[2 * e + 1], hi[e], lo[e]);
          tmem_st16(col, hi);
          tmem_st16(col + 16, lo);
          tmem_st_wait();
          tc_fence_before_sync();
        }
        mbar_arrive_warp(&sh->hid_full[b]);
      }
      if (*abortp) break;
      if (kState && part == 1 && i > 0) collect(i - 1);          // while this tile's last GEMM2s run
      if (part != 0) continue;
      // ---- one warp per quadrant finishes the tile's rows ----
      pt_wait(&sh->g2_full, i & 1, abortp, status, 38);
      tc_fence_after_sync();
      uint32_t g2[PT_W2N];
      tmem_ld16(lane_addr + PT_G2COL, g2);
      tmem_ld_wait();
      tc_fence_before_sync();
      mbar_arrive_warp(&sh->g2_free);
      const int j = jbeg + i * PT_TILE + row;
      float out[R];
      {
        float gv[R];
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
        }
      }
      const bool live = j < jend;
      const bool kept = live && kState && slot_of[j] >= 0;
      if (live && (!kState || kept)) {
#pragma unroll
        for (int r4 = 0; r4 < R / 4; ++r4)
          reinterpret_cast<float4*>(psi + (size_t)j * R)[r4] =
              make_float4(out[r4 * 4], out[r4 * 4 + 1], out[r4 * 4 + 2], out[r4 * 4 + 3]);
      }
      if (!kState) {
        if (live)
#pragma unroll
          for (int r = 0; r < R; ++r) pmax = fmaxf(pmax, out[r]);
        continue;
      }
      // ---- the tile's psi as the B operand of the state products ----
      float tmax = 0.f;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (!live || kept) out[r] = 0.f;                 // only discarded prompt tokens enter H, z
        tmax = fmaxf(tmax, out[r]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
      pt_wait(&sh->b_free, (i & 1) ^ 1, abortp, status, 25);      // the products of the tile before have read bbuf (and wmax, inv_scale are theirs no more)
      if (lane == 0) sh->wmax[quad] = tmax;
      mbar_arrive_warp(&sh->mx_bar);                               // the four finishing warps meet (bounded, like every wait)
      pt_wait(&sh->mx_bar, 0, abortp, status, 26);
      tmax = fmaxf(fmaxf(sh->wmax[0], sh->wmax[1]), fmaxf(sh->wmax[2], sh->wmax[3]));
      // the largest value lands near 8192: hi parts far from fp16's overflow, lo parts as far from
      // its underflow as they can be
      float scale = 1.f;
      if (tmax > 0.f && tmax < INFINITY) scale = exp2f(fminf(fmaxf(floorf(log2f(8192.f / tmax)), -100.f), 100.f));
      if (tid == 0) sh->inv_scale[i & 1] = 1.0f / scale;
      __align__(16) __half hh[R], ll[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float x = out[r] * scale;
        hh[r] = __float2half_rn(x);
        ll[r] = __float2half_rn(x - __half2float(hh[r]));
      }
      unsigned char* brow = bbuf + (row >> 3) * B_LBO + (row & 7) * 16;
#pragma unroll
      for (int nb = 0; nb < R / 8; ++nb) {
        *reinterpret_cast<uint4*>(brow + nb * B_SBO) = *reinterpret_cast<const uint4*>(&hh[nb * 8]);
        *reinterpret_cast<uint4*>(brow + (R / 8 + nb) * B_SBO) = *reinterpret_cast<const uint4*>(&ll[nb * 8]);
      }
      fence_proxy_async_smem();
      mbar_arrive_warp(&sh->mx_bar);                               // wmax is read by all four before the next tile rewrites it
      pt_wait(&sh->mx_bar, 1, abortp, status, 27);
      mbar_arrive_warp(&sh->b_full);
    }
    if (kState && part == 1 && ntiles > 0 && !*abortp) {
      collect(ntiles - 1);
      float* hp = p.a.ws_hpart + ((size_t)g * kMaxSplit + split) * (R * kHeadDim + R);
#pragma unroll
      for (int r = 0; r < R; ++r) hp[r * kHeadDim + row] = hacc[r];
      if (row == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) hp[R * kHeadDim + r] = sh->zacc[r];
      }
    }
    if (!kState) {
      // maximum over the split, into the instance's cell: psi >= 0, so its bit pattern orders like an
      // integer, and a maximum does not depend on the order of the atomics
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) pmax = fmaxf(pmax, __shfl_xor_sync(0xffffffffu, pmax, o));
      if (lane == 0 && mp.pmax && pmax > 0.f && pmax < INFINITY) atomicMax(mp.pmax + g, __float_as_int(pmax));
    }
  }
  drain_after_abort(abortp);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == PT_WORKERS / 32 + 1) tmem_dealloc(tmem, PT_TMEM);
}

bool psi_tc_supported(const Dims& d) { return d.Rp == 512 || d.Rp == 256 || d.Rp == 128 || d.Rp == 64; }

template <int R, bool kState>
static int launch_variant(const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tw1, const PfParams& p,
                          const PtMap& mp, int G, size_t smem, cudaStream_t s) {
  auto kern = psi_tc_kernel<R, kState>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return fail_cuda("shared memory opt-in of psi_tc_kernel");
  kern<<<dim3(p.nsplit, G), PT_THREADS, smem, s>>>(tk, tv, tw1, p, mp);
  return check_launch("psi_tc_kernel");
}

// x: the rows the map is applied to ([B, layer_count, Hd, S, D]; for phi, Q with Hd * group heads); with_state: psi fused with the
// prompt state build (needs the kept / discarded map of select_kernel and V)
static int launch_map_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s, const __half* x, const void* w1,
                         const PtMap& mp, bool with_state) {
  const Dims& d = c->d;
  CUtensorMap tmap_k, tmap_v, tmap_w1;
  const uint64_t hg = mp.is_phi ? (uint64_t)p.grp : 1;            // query heads per KV head where the map is phi
  const uint64_t rows = (uint64_t)d.B * p.layer_count * d.Hd * p.S;
  if (!make_tmap_f16_2d(&tmap_k, x, rows * hg, kHeadDim, kHeadDim * 2, PT_TILE)) return fail_cuda("tensor map of K");
  if (!make_tmap_f16_2d(&tmap_v, with_state ? p.V : x, with_state ? rows : rows * hg, kHeadDim, kHeadDim * 2, PT_TILE))
    return fail_cuda("tensor map of V");
  if (!make_tmap_f16_2d(&tmap_w1, w1, (uint64_t)d.L * d.Hd * hg * kHeadDim, d.Rp, (uint64_t)d.Rp * 2, kHeadDim))
    return fail_cuda("tensor map of W1");
  const size_t smem = (size_t)(d.Rp / 64) * 16384 + PT_KBYTES + (size_t)d.Rp * PT_W2N * 2 +
                      (with_state ? PT_KBYTES + (size_t)PT_TILE * 2 * d.R * 2 + 4096 : 0) + sizeof(PtShared) + 64;
  char name[48];
  snprintf(name, sizeof name, "psi_tc_kernel<%d, %d>", d.R, (int)with_state);
  LaunchScope scope(c, LESS_KERNEL_PSI, s, name);
  if (d.R == 8)
    return with_state ? launch_variant<8, true>(tmap_k, tmap_v, tmap_w1, p, mp, G, smem, s)
                      : launch_variant<8, false>(tmap_k, tmap_v, tmap_w1, p, mp, G, smem, s);
  return with_state ? launch_variant<16, true>(tmap_k, tmap_v, tmap_w1, p, mp, G, smem, s)
                    : launch_variant<16, false>(tmap_k, tmap_v, tmap_w1, p, mp, G, smem, s);
}

// psi of every prompt token and the instance's maximum (the parallel form's operand pack reads both)
int launch_psi_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s) {
  PtMap mp;
  mp.w2 = p.w_psi2; mp.w3 = p.w_psi3; mp.out = p.a.ws_psi; mp.pmax = p.a.ws_pmax; mp.is_phi = 0;
  return launch_map_tc(c, p, G, s, p.K, p.w_psi1, mp, false);
}

// psi fused with the prompt state build: leaves psi of the kept tokens in the workspace and the
// splits' partial H, z for finalize_kernel
int launch_psi_state_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s) {
  PtMap mp;
  mp.w2 = p.w_psi2; mp.w3 = p.w_psi3; mp.out = p.a.ws_psi; mp.pmax = nullptr; mp.is_phi = 0;
  return launch_map_tc(c, p, G, s, p.K, p.w_psi1, mp, true);
}

// phi(q_i) of every row of Q into `out` [G][Sp][R]; G counts query heads (p.grp per KV instance)
int launch_phi_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s, float* out) {
  PtMap mp;
  mp.w2 = (const __half*)c->w.w_phi2; mp.w3 = nullptr; mp.out = out; mp.pmax = nullptr; mp.is_phi = 1;
  return launch_map_tc(c, p, G, s, p.Q, c->w.w_phi1, mp, false);
}

}  // namespace less
