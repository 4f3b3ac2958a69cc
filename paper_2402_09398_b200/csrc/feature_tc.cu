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
//                                   * X^T           (B, K-major, n = tokens padded to 16, 32 or 64)
// so the GELU work of the epilogue grows with the number of tokens, not with the
// 128-row tile, and a batch of one costs one GELU per thread and chunk.
// Epilogue warps (four per lane quadrant) read D1^T from tensor memory, apply
// gelu, split the result into fp16 hi + lo (one fp16 rounding of the hidden
// layer would cost ~2e-3 on psi) and store it, tokens contiguous, as the M-major
// A operand of
//     D2[tokens x 16] += H[tokens x 128 hidden] * W2[chunk rows, :]       (GEMM2)
// whose accumulator lives in tensor memory across the chunks.  After the last
// chunk: c2 * gelu(c1 * .), W3 (psi only) and the absolute value on CUDA cores.
// The hidden activations never leave the SM (the paper folds the activation into the preceding linear kernel,
// Section 3.2, taken to the whole MLP).  Plain TMA loads only; every wait is bounded.
#include "feature_gemv.cuh"
#include "tc_common.cuh"

namespace less {

constexpr int FT_EPI_WARPS = 8;
constexpr int FT_EPI_THREADS = FT_EPI_WARPS * 32;
constexpr int FT_THREADS = 96 + FT_EPI_THREADS;   // small-batch kernel: warp 0 TMA, warp 1 MMA, warps 2..9 epilogue, warp 10 input rows by plain loads
// The larger-batch kernel runs sixteen GELU warps (four per scheduler: with two the issue slots sat
// idle) in two groups of eight that take the 128-unit chunks in turn, each with its own accumulator
// buffer and its own hidden-layer operand: while one group is saturating the schedulers with GELUs,
// the other sits in the phases that issue little (waiting for GEMM1, loading the accumulator, storing
// the operand, the proxy fence).  In lockstep the sixteen warps spent 1 350 of a chunk's 3 200 cycles
// in the GELU phase and the rest with the schedulers mostly idle.  Four more warps, one per lane
// quadrant, finish the items (second layer's GELU, W3, output), so that the GELU warps never wait for it.
constexpr int FL_GROUPS = 2;
constexpr int FL_GROUP_WARPS = 8;
constexpr int FL_EPI_WARPS = FL_GROUPS * FL_GROUP_WARPS;
constexpr int FL_FIN_WARPS = 4;
constexpr int FL_THREADS = 64 + (FL_EPI_WARPS + FL_FIN_WARPS) * 32;
constexpr int FT_CHUNK = 128;                     // hidden units per GEMM1
constexpr int FT_STAGE_BYTES = FT_CHUNK * kHeadDim * 2;
constexpr int FT_MAX_STAGES = 6;
constexpr int FT_SMEM_LIMIT = 232448;             // 227 KB per CTA

struct FtShared {
  uint64_t full[FT_MAX_STAGES], empty[FT_MAX_STAGES];
  uint64_t aux_full[2], aux_empty[2];
  uint64_t d1_full[2], d1_free[2];
  uint64_t hid_full[FL_GROUPS], hid_free[FL_GROUPS];   // per epilogue group
  uint64_t d2_full, d2_free;
  uint32_t tmem_base;
  int abort;
  __align__(16) __half w3[2][16 * 16];
};

struct FtGeom {
  int npad;        // tokens per tile (GEMM1 N): 16, 32 or 64
  int ntile;       // token tiles per (layer-head, map)
  int items;       // work items
  int per_head;    // items per KV head: (G + 1) * ntile
  int G;           // query heads per KV head
  int kv0;         // first (layer, KV head) of this launch
  int nstage;      // ring stages
  uint32_t tmem_cols;
  int late_inputs; // the kernel may have started before the kernel before it in the stream was done (programmatic
                   // dependent launch): weights are fetched at once, the step's q, k only behind the wait for it
};


// Work item -> (token tile, map, layer-head of that map).  The items of one KV head are
// neighbours - its G phi items (one per query head), then its psi item, each times the token
// tiles - so that a head's feature maps are complete early and together: the decode kernel of the
// same step, which may already be running, needs exactly those.
struct FtItem { int tile, which, lh; };
__device__ __forceinline__ FtItem ft_item(int it, const FtGeom& gm) {
  FtItem r;
  const int kvi = it / gm.per_head, rest = it - kvi * gm.per_head, kv = gm.kv0 + kvi;
  const int sub = rest / gm.ntile;
  r.tile = rest - sub * gm.ntile;
  r.which = sub == gm.G;
  r.lh = r.which ? kv : kv * gm.G + sub;
  return r;
}

// A warp that has written its share of an item's phi / psi publishes it: every lane's stores are
// fenced, the warp converges, one lane bumps the head's counter.  The decode kernel compares the
// counter with the number of writer warps the head has had once this step is complete.
__device__ __forceinline__ void publish_rows(const FmParams& p, int which, int lh) {
  if (p.feat_flag == nullptr) return;
  __threadfence();
  __syncwarp();
  if ((threadIdx.x & 31) == 0) atomicAdd(p.feat_flag + (which ? p.flag_stride : 0) + lh, 1u);
}

// The producer thread of both kernels: per item the input rows, W2 and W3 into the item's aux
// buffers, then W1 in 32-KB chunks through the ring.  Ring positions advance by counting, not by
// dividing: this thread's instruction latency is on the critical path of the whole stream.
template <int R>
__device__ __forceinline__ void ft_produce(const CUtensorMap* tm_q, const CUtensorMap* tm_k, const CUtensorMap* tm_w1phi,
                                           const CUtensorMap* tm_w1psi, const FmParams& p, const FtGeom& gm, int my_items,
                                           int nchunk, unsigned char* xbuf, uint32_t xbytes, unsigned char* w2dst,
                                           uint32_t w2bytes, __half* w3buf /* [2][256] */, unsigned char* ring,
                                           uint64_t* full, uint64_t* empty, uint64_t* aux_full, uint64_t* aux_empty,
                                           int naux, volatile int* abortp, int32_t* status) {
  uint32_t s = 0, sph = 0, a = 0, aph = 0;
  const uint64_t stream_policy = l2_evict_first_policy();
  // The first item of a kernel that may have started early: its weights (W2, W3 and as many W1 chunks as the
  // ring takes) are asked for at once, its input rows only once the kernels before this one are done.
  bool inputs_later = gm.late_inputs != 0;
  for (int n = 0; n < my_items; ++n, (++a == (uint32_t)naux ? (a = 0, aph ^= 1) : 0u)) {
    const FtItem im = ft_item(blockIdx.x + n * gridDim.x, gm);
    wait_or_give_up(&aux_empty[a], aph ^ 1, abortp, status, 40);
    if (*abortp) return;                                 // issue nothing more once the CTA has given up
    const CUtensorMap* tx = im.which ? tm_k : tm_q;
    const CUtensorMap* tw1 = im.which ? tm_w1psi : tm_w1phi;
    mbar_expect_tx(&aux_full[a], (p.x_plain ? 0u : xbytes) + w2bytes + (im.which ? R * R * 2 : 0));
    unsigned char* xa = xbuf + a * xbytes;
    auto load_inputs = [&]() {
      if (p.x_plain) return;
      tma_load_2d(xa, tx, im.lh * kHeadDim, im.tile * gm.npad, &aux_full[a]);
      tma_load_2d(xa + xbytes / 2, tx, im.lh * kHeadDim + 64, im.tile * gm.npad, &aux_full[a]);
    };
    if (!inputs_later) load_inputs();
    // W2 comes as one contiguous copy (a tiled load of 16-byte rows is far slower)
    bulk_g2s(w2dst + a * w2bytes, p.w2[im.which] + (size_t)im.lh * p.Rp * R, w2bytes, &aux_full[a]);
    if (im.which) bulk_g2s(w3buf + a * 256, p.w3 + (size_t)im.lh * R * R, R * R * 2, &aux_full[a]);
    const int ahead = nchunk < gm.nstage ? nchunk : gm.nstage;   // chunks whose ring stages are free without the consumer
    for (int c = 0; c < nchunk; ++c) {
      if (inputs_later && c == ahead) {
        pdl_wait_primary();
        pdl_launch_dependents();                         // only now: the step's decode kernel reads the arena before it waits
        load_inputs();
        inputs_later = false;
      }
      wait_or_give_up(&empty[s], sph ^ 1, abortp, status, 41);
      if (*abortp) return;
      mbar_expect_tx(&full[s], FT_STAGE_BYTES);
      unsigned char* st = ring + (size_t)s * FT_STAGE_BYTES;
      tma_load_2d_hint(st, tw1, c * FT_CHUNK, im.lh * kHeadDim, &full[s], stream_policy);
      tma_load_2d_hint(st + FT_STAGE_BYTES / 2, tw1, c * FT_CHUNK + 64, im.lh * kHeadDim, &full[s], stream_policy);
      if (++s == (uint32_t)gm.nstage) { s = 0; sph ^= 1; }
    }
    if (inputs_later) {                                  // every chunk of the first item fitted the ring
      pdl_wait_primary();
      pdl_launch_dependents();
      load_inputs();
      inputs_later = false;
    }
  }
}

template <int R>
__global__ void __launch_bounds__(FL_THREADS, 1) feature_tc_kernel(
    const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
    const __grid_constant__ CUtensorMap tm_w1phi, const __grid_constant__ CUtensorMap tm_w1psi, FmParams p,
    FtGeom gm, int32_t* status) {
  extern __shared__ __align__(1024) unsigned char ft_smem[];
  if (smem_misaligned(ft_smem, status, 60)) return;
  const int Rp = p.Rp, nchunk = Rp / FT_CHUNK, npad = gm.npad, nstage = gm.nstage;
  const uint32_t hbytes = (uint32_t)npad * 256;      // hi (or lo): npad/8 token blocks x 2 KB
  const uint32_t xbytes = (uint32_t)npad * 256;      // two 64-column halves of npad rows x 128 B
  const uint32_t w2bytes = (uint32_t)Rp * R * 2;
  unsigned char* hbuf = ft_smem;                     // per group: hi, then lo
  unsigned char* xbuf = hbuf + FL_GROUPS * 2 * hbytes;   // [2][xbytes]
  unsigned char* ring = xbuf + 2 * xbytes;           // [nstage][32 KB]
  unsigned char* w2buf = ring + (size_t)nstage * FT_STAGE_BYTES;   // [2][R/8 column blocks][Rp rows][16 B]
  unsigned char* w2raw = w2buf + 2 * w2bytes;        // R = 16 only: [2][Rp rows][32 B] as it lies in HBM
  FtShared* sh = reinterpret_cast<FtShared*>(w2raw + (R == 16 ? 2 * w2bytes : 0));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < nstage; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh->aux_full[s], 1);
      mbar_init(&sh->aux_empty[s], 1 + FL_FIN_WARPS);
      mbar_init(&sh->d1_full[s], 1);
      mbar_init(&sh->d1_free[s], FL_GROUP_WARPS);
      mbar_init(&sh->hid_full[s], FL_GROUP_WARPS);
      mbar_init(&sh->hid_free[s], 1);
    }
    mbar_init(&sh->d2_full, 1);
    mbar_init(&sh->d2_free, FL_FIN_WARPS);
    // a CTA that starts after another one has given up skips every wait: the grid drains at once
    sh->abort = *reinterpret_cast<volatile int32_t*>(status) != 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&sh->tmem_base, gm.tmem_cols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (!gm.late_inputs) pdl_launch_dependents();   // else by the producer thread, behind its wait for the kernels before
  const uint32_t tmem = sh->tmem_base;
  const uint32_t d2col = 2u * (uint32_t)npad;
  volatile int* abortp = &sh->abort;
  const int my_items = blockIdx.x < gm.items ? (gm.items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  const uint32_t total = (uint32_t)my_items * nchunk;   // chunks of this CTA, counted across its items

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0)
      ft_produce<R>(&tm_q, &tm_k, &tm_w1phi, &tm_w1psi, p, gm, my_items, nchunk, xbuf, xbytes,
                    R == 16 ? w2raw : w2buf, w2bytes, &sh->w3[0][0], ring, sh->full, sh->empty, sh->aux_full,
                    sh->aux_empty, 2, abortp, status);
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0 && my_items > 0) {
      const uint32_t idesc1 = idesc_f16(128, npad, 1, 0);   // A = W1 chunk (M-major), B = x rows (K-major)
      constexpr uint32_t idesc2 = idesc_f16(128, 16, 1, 1); // A = hidden (M-major), B = W2 (N-major)
      // Descriptors are built once; afterwards only the start address (bits [0, 14), in 16-byte
      // units) moves.  Every index below advances by counting: a division on this thread would
      // sit on the critical path of the stream.
      const uint64_t ad_ring = smem_desc(smem_u32(ring), FT_STAGE_BYTES / 2, 1024, kLayoutSw128);
      const uint64_t bd_x = smem_desc(smem_u32(xbuf), 16, 1024, kLayoutSw128);
      // R = 8 fills one 8-column block; the second block of the N = 16 tile then only has to
      // lie inside this CTA's shared memory (its columns of D2 are never read)
      const uint64_t bd_w2 = smem_desc(smem_u32(w2buf), 128, R == 16 ? (uint32_t)Rp * 16 : 128u, kLayoutNone);
      const uint64_t ad_hid = smem_desc(smem_u32(hbuf), 128, 2048, kLayoutNone);
      // GEMM1 runs two chunks ahead of GEMM2: one chunk per epilogue group is in work at any time.
      // Chunk qq (counted over the CTA's items) lives in accumulator buffer qq & 1 and belongs to group qq & 1.
      uint32_t s = 0, sph = 0, c1 = 0, n1 = 0, issued = 0;
      auto issue_gemm1 = [&]() {
        const uint32_t a = n1 & 1, b1 = issued & 1;
        if (c1 == 0) wait_or_give_up(&sh->aux_full[a], (n1 >> 1) & 1, abortp, status, 42);
        wait_or_give_up(&sh->full[s], sph, abortp, status, 43);
        wait_or_give_up(&sh->d1_free[b1], ((issued >> 1) & 1) ^ 1, abortp, status, 44);   // the group has loaded the buffer's last chunk
        if (*abortp) return;
        tc_fence_after_sync();
        const uint64_t ad0 = ad_ring + (uint64_t)(s * (FT_STAGE_BYTES >> 4));
        const uint64_t bd0 = bd_x + (uint64_t)(a * (xbytes >> 4));
        const uint64_t bd1 = bd0 + (uint64_t)(xbytes >> 5);
#pragma unroll
        for (int ks = 0; ks < kHeadDim / 16; ++ks)
          mma_f16_ss(tmem + b1 * npad, ad0 + (uint64_t)(ks * (2048 >> 4)), (ks < 4 ? bd0 : bd1) + (uint64_t)((ks & 3) * 2),
                     idesc1, ks ? 1u : 0u);
        mma_commit(&sh->empty[s]);
        mma_commit(&sh->d1_full[b1]);
        if (++s == (uint32_t)nstage) { s = 0; sph ^= 1; }
        if (++c1 == (uint32_t)nchunk) { c1 = 0; ++n1; }
        ++issued;
      };
      issue_gemm1();
      if (issued < total && !*abortp) issue_gemm1();
      uint32_t qq = 0;
      for (uint32_t n = 0; n < (uint32_t)my_items && !*abortp; ++n) {
        const uint32_t a = n & 1;
        for (uint32_t c = 0; c < (uint32_t)nchunk; ++c, ++qq) {
          const uint32_t g = qq & 1;
          // the chunk two ahead first: its accumulator buffer is free as soon as group g has loaded chunk qq
          if (issued < total) issue_gemm1();
          if (c == 0) wait_or_give_up(&sh->d2_free, (n & 1) ^ 1, abortp, status, 45);
          wait_or_give_up(&sh->hid_full[g], (qq >> 1) & 1, abortp, status, 46);
          if (*abortp) break;
          tc_fence_after_sync();
          const uint64_t bd0 = bd_w2 + (uint64_t)(a * (w2bytes >> 4) + c * (FT_CHUNK * 16 >> 4));
          const uint64_t ad_hi = ad_hid + (uint64_t)(g * (2 * hbytes >> 4));
          const uint64_t ad_lo = ad_hi + (uint64_t)(hbytes >> 4);
#pragma unroll
          for (int ks = 0; ks < FT_CHUNK / 16; ++ks) {
            mma_f16_ss(tmem + d2col, ad_hi + (uint64_t)(ks * 16), bd0 + (uint64_t)(ks * 16), idesc2, (c | ks) ? 1u : 0u);
            mma_f16_ss(tmem + d2col, ad_lo + (uint64_t)(ks * 16), bd0 + (uint64_t)(ks * 16), idesc2, 1u);
          }
          mma_commit(&sh->hid_free[g]);
        }
        if (*abortp) break;
        mma_commit(&sh->d2_full);
        mma_commit(&sh->aux_empty[a]);
      }
    }
  } else if (warp < 2 + FL_EPI_WARPS) {
    // ---------------- GELU warps: group g takes the chunks qq = g, g + 2, ... ----------------
    const int ew = warp - 2;                   // 0..15
    const int g = ew >> 3;                     // group = accumulator buffer = hidden operand buffer
    const int quad = warp & 3;                 // tensor-memory lane quadrant this warp may read
    const int hf = (ew & 7) >> 2;              // which half of the token blocks (blocks hf, hf + 2, hf + 4, hf + 6)
    const int j = quad * 32 + lane;            // hidden unit inside the chunk = accumulator lane
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    unsigned char* hrow = hbuf + (size_t)g * 2 * hbytes + (j >> 3) * 128 + (j & 7) * 16;
    int n_cur = -1, nb = 0, nblk = 0, a = 0;
    int n = g / nchunk, c = g % nchunk;        // item and chunk of qq, advanced by counting
    for (uint32_t qq = g, u = 0; qq < total && !*abortp; qq += FL_GROUPS, ++u) {
      if (n != n_cur) {
        n_cur = n;
        const FtItem im = ft_item(blockIdx.x + n * gridDim.x, gm);
        nb = min(npad, p.B - im.tile * npad);
        nblk = (nb + 7) >> 3;
        a = n & 1;
      }
      if (R == 16 && c == 0) {
        // the item's W2: 32-byte rows -> two blocks of 16-byte rows, by the group that has the item's first
        // chunk; the GEMM2s that read this buffer two items ago are complete (the producer waited for them
        // before refilling the raw copy), and this group's hid_full arrival below publishes it
        wait_or_give_up(&sh->aux_full[a], (n >> 1) & 1, abortp, status, 50);
        const uint4* src = reinterpret_cast<const uint4*>(w2raw + a * w2bytes);
        unsigned char* dst = w2buf + a * w2bytes;
        for (int x = (ew & 7) * 32 + lane; x < Rp * 2; x += FL_GROUP_WARPS * 32)
          *reinterpret_cast<uint4*>(dst + ((size_t)(x & 1) * Rp + (x >> 1)) * 16) = src[x];
      }
      wait_or_give_up(&sh->d1_full[g], u & 1, abortp, status, 47);
      // the GEMM2 of this group's chunk before has read the hidden operand (two chunks ago: long done)
      wait_or_give_up(&sh->hid_free[g], (u & 1) ^ 1, abortp, status, 48);
      if (*abortp) break;
      tc_fence_after_sync();
      // this warp's four token blocks (a tile has at most 8 blocks of 8 tokens), all in registers at once:
      // sixteen independent GELU chains per thread keep a scheduler with two such warps issuing
      {
        uint32_t acc[4][8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int blk = hf + 2 * i;
          if (blk < nblk) tmem_ld8(lane_addr + g * npad + blk * 8, acc[i]);
        }
        tmem_ld_wait();
        tc_fence_before_sync();                // the accumulator buffer is in registers: GEMM1 may refill it
        mbar_arrive_warp(&sh->d1_free[g]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int blk = hf + 2 * i;
          if (blk < nblk) {
            uint32_t ph[4], pl[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              // columns past the last token hold products with zero-filled rows: no GELU spent on them
              // (c1 multiplies the layer-2 sums instead: the fp16 operand must not depend on how
              // small that learnable scalar is)
              float h0 = 0.f, h1 = 0.f;
              if (blk * 8 + 2 * e + 1 < nb) gelu_erf2(__uint_as_float(acc[i][2 * e]), __uint_as_float(acc[i][2 * e + 1]), h0, h1);
              else if (blk * 8 + 2 * e < nb) h0 = gelu_erf(__uint_as_float(acc[i][2 * e]));
              const __half2 hh = __floats2half2_rn(h0, h1);
              const float2 hf2 = __half22float2(hh);
              const __half2 ll = __floats2half2_rn(h0 - hf2.x, h1 - hf2.y);
              ph[e] = *reinterpret_cast<const uint32_t*>(&hh);
              pl[e] = *reinterpret_cast<const uint32_t*>(&ll);
            }
            *reinterpret_cast<uint4*>(hrow + blk * 2048) = make_uint4(ph[0], ph[1], ph[2], ph[3]);
            *reinterpret_cast<uint4*>(hrow + hbytes + blk * 2048) = make_uint4(pl[0], pl[1], pl[2], pl[3]);
          }
        }
      }
      fence_proxy_async_smem();
      mbar_arrive_warp(&sh->hid_full[g]);
      c += FL_GROUPS;
      while (c >= nchunk) { c -= nchunk; ++n; }
    }
  } else {
    // ---------------- finishing warps, one per lane quadrant: layer 2's result, token = accumulator lane ----------------
    const int quad = warp & 3;
    const int j = quad * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    for (int n = 0; n < my_items && !*abortp; ++n) {
      const FtItem im = ft_item(blockIdx.x + n * gridDim.x, gm);
      const int which = im.which, lh = im.lh;
      const int a = n & 1;
      const int b0 = im.tile * npad, nb = min(npad, p.B - b0);
      float c1 = 1.f, c2 = 1.f;
      if (which && p.psi_scale) { c1 = __ldg(p.psi_scale + lh * 2); c2 = __ldg(p.psi_scale + lh * 2 + 1); }
      wait_or_give_up(&sh->aux_full[a], (n >> 1) & 1, abortp, status, 51);   // the item's W3
      wait_or_give_up(&sh->d2_full, n & 1, abortp, status, 49);
      if (*abortp) break;
      tc_fence_after_sync();
      const bool mine = quad * 32 < nb;                    // warp-uniform
      uint32_t g2[16];
      if (mine) {
#pragma unroll
        for (int r8 = 0; r8 < R / 8; ++r8) tmem_ld8(lane_addr + d2col + r8 * 8, g2 + r8 * 8);
        tmem_ld_wait();
      }
      tc_fence_before_sync();
      mbar_arrive_warp(&sh->d2_free);
      if (mine && j < nb) {
        float gv[R], out[R];
#pragma unroll
        for (int r = 0; r < R; ++r) gv[r] = c2 * gelu_erf(c1 * __uint_as_float(g2[r]));
        if (which) {
          const __half* w3 = &sh->w3[a][0];
#pragma unroll
          for (int r = 0; r < R; ++r) {
            float sacc = 0.f;
#pragma unroll
            for (int rr = 0; rr < R; ++rr) sacc = fmaf(gv[rr], __half2float(w3[rr * R + r]), sacc);
            out[r] = fabsf(sacc);
          }
        } else {
#pragma unroll
          for (int r = 0; r < R; ++r) out[r] = fabsf(gv[r]);
        }
        float4* dst = reinterpret_cast<float4*>(p.out[which] + ((size_t)(b0 + j) * p.L * p.Hh[which] + lh) * R);
#pragma unroll
        for (int r4 = 0; r4 < R / 4; ++r4) dst[r4] = make_float4(out[r4 * 4], out[r4 * 4 + 1], out[r4 * 4 + 2], out[r4 * 4 + 3]);
      }
      if (mine) publish_rows(p, which, lh);              // ceil(nb / 32) writer warps per item
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

// --------------------------------------------------------------------------- //
// Small batches (at most 8 tokens per head): the same weight stream and the same
// transposed GEMM1, but layer 2 stays on CUDA cores.  A tensor-core instruction
// with a 128-row operand costs about a hundred cycles however narrow it is, and
// GEMM2 needs 64 of them per item (hi and lo halves of 512 hidden units); with a
// handful of tokens the epilogue thread that owns hidden unit j multiplies its
// activations with row j of W2 in fp32 registers instead, and one shuffle
// reduction per item replaces the second GEMM.
// --------------------------------------------------------------------------- //
constexpr int FS_BUFS = 4;        // D1^T buffers in tensor memory (16 columns each)
constexpr int FS_NPAD = 16;       // GEMM1 N (the narrowest a 128-row MMA takes)
constexpr int FS_XROWS = 8;       // input rows really loaded: the other 8 columns of D1^T are never read
constexpr int FS_XBYTES = FS_XROWS * 256;
constexpr int FS_AUX = 3;         // items whose inputs, W2 and W3 may be in flight

template <int V>
struct FsShared {
  uint64_t full[FT_MAX_STAGES], empty[FT_MAX_STAGES];
  uint64_t aux_full[FS_AUX], aux_empty[FS_AUX];
  uint64_t d1_full[FS_BUFS], d1_free[FS_BUFS];
  uint32_t tmem_base;
  int abort;
  __align__(16) __half w3[FS_AUX][16 * 16];
  float red[2][FT_EPI_WARPS][V];        // per item parity, per warp: partial layer-2 sums [token][r]
  float g[2][V];                        // c2 * gelu(layer-2 sums)
};

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, %0;" ::"n"(FT_EPI_THREADS) : "memory"); }

// Sum over the 32 lanes of V values per lane, V a power of two: every exchange halves the
// values a lane keeps, so it costs about V shuffles instead of 5 V.  Afterwards v[0 .. count)
// are complete sums of the indices base .. base + count, and lanes with `owner` false hold copies.
template <int V>
__device__ __forceinline__ void lane_reduce_scatter(float (&v)[V], int lane, int& base, int& count, bool& owner) {
  int n = V;
  base = 0;
  owner = true;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const bool up = (lane & o) != 0;
    if (n > 1) {
      n >>= 1;
#pragma unroll
      for (int i = 0; i < V / 2; ++i) {
        if (i < n) {
          const float keep = up ? v[i + n] : v[i];
          const float send = up ? v[i] : v[i + n];
          v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
        }
      }
      if (up) base += n;
    } else {
      v[0] += __shfl_xor_sync(0xffffffffu, v[0], o);
      if (up) owner = false;
    }
  }
  count = n;
}

template <int R, int NT>
__global__ void __launch_bounds__(FT_THREADS) feature_tc_small_kernel(
    const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
    const __grid_constant__ CUtensorMap tm_w1phi, const __grid_constant__ CUtensorMap tm_w1psi, FmParams p,
    FtGeom gm, int32_t* status) {
  extern __shared__ __align__(1024) unsigned char ft_smem[];
  if (smem_misaligned(ft_smem, status, 60)) return;
  constexpr int V = NT * R;
  const int Rp = p.Rp, nchunk = Rp / FT_CHUNK, nstage = gm.nstage;
  const uint32_t w2bytes = (uint32_t)Rp * R * 2;
  // x: [FS_AUX][2 halves][8 rows x 128 B], padded to 8 KB.  GEMM1 reads 16 rows per half; rows 8..15
  // are whatever follows in shared memory (the other half, the next buffer, the pad) and only feed
  // D1^T columns that no one reads.
  unsigned char* xbuf = ft_smem;
  unsigned char* ring = xbuf + 8192;                               // [nstage][32 KB]
  unsigned char* w2raw = ring + (size_t)nstage * FT_STAGE_BYTES;   // [FS_AUX][Rp rows][R] as it lies in HBM
  FsShared<V>* sh = reinterpret_cast<FsShared<V>*>(w2raw + FS_AUX * w2bytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < nstage; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], 1);
    }
    for (int s = 0; s < FS_AUX; ++s) {
      mbar_init(&sh->aux_full[s], p.x_plain ? 2 : 1);    // the producer's copies, and the row loader's arrival
      mbar_init(&sh->aux_empty[s], 1 + FT_EPI_WARPS);
    }
    for (int s = 0; s < FS_BUFS; ++s) {
      mbar_init(&sh->d1_full[s], 1);
      mbar_init(&sh->d1_free[s], FT_EPI_WARPS / 2);
    }
    sh->abort = *reinterpret_cast<volatile int32_t*>(status) != 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&sh->tmem_base, FS_BUFS * FS_NPAD);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  // The decode kernel of this step may start now - unless this kernel itself started early (late_inputs):
  // the decode kernel reads the arena before it waits for anything, so it is let go only once the
  // kernels before this one are known to be done (the producer thread does that, behind its own wait).
  if (!gm.late_inputs) pdl_launch_dependents();
  const uint32_t tmem = sh->tmem_base;
  volatile int* abortp = &sh->abort;
  const int my_items = blockIdx.x < gm.items ? (gm.items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0)
      ft_produce<R>(&tm_q, &tm_k, &tm_w1phi, &tm_w1psi, p, gm, my_items, nchunk, xbuf, FS_XBYTES, w2raw, w2bytes,
                    &sh->w3[0][0], ring, sh->full, sh->empty, sh->aux_full, sh->aux_empty, FS_AUX, abortp, status);
  } else if (warp == 2 + FT_EPI_WARPS) {
    // ---------------- input rows by plain loads ----------------
    // Used when q and k lie in pinned host memory (the host entry point): the rows come over PCIe
    // while the weights stream, no staging copy in front of the step.  The warp writes what the
    // tiled load would have written: per half of 64 columns, 8 rows of 128 bytes, the 16-byte chunk c
    // of row r at chunk position c ^ r (128-byte swizzle); rows past the batch are zeros.
    if (p.x_plain) {
      if (gm.late_inputs) pdl_wait_primary();           // the rows may be written by the kernel before this one
      uint32_t a = 0, aph = 0;
      for (int n = 0; n < my_items; ++n, (++a == FS_AUX ? (a = 0, aph ^= 1) : 0u)) {
        const FtItem im = ft_item(blockIdx.x + n * gridDim.x, gm);
        wait_or_give_up(&sh->aux_empty[a], aph ^ 1, abortp, status, 67);
        if (*abortp) break;
        unsigned char* xa = xbuf + a * FS_XBYTES;
        const __half* src = p.x[im.which] + (size_t)im.lh * kHeadDim;
        const size_t row_stride = (size_t)p.L * p.Hh[im.which] * kHeadDim;
        const int b0 = im.tile * FS_NPAD;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int e = lane + 32 * i;                 // 128 chunks: (half, row, chunk)
          const int h = e >> 6, r = (e >> 3) & 7, c = e & 7;
          uint4 v = make_uint4(0, 0, 0, 0);
          if (b0 + r < p.B) v = *reinterpret_cast<const uint4*>(src + (size_t)(b0 + r) * row_stride + h * 64 + c * 8);
          *reinterpret_cast<uint4*>(xa + h * (FS_XBYTES / 2) + r * 128 + ((c ^ r) << 4)) = v;
        }
        fence_proxy_async_smem();
        mbar_arrive_warp(&sh->aux_full[a]);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: GEMM1 only ----------------
    if (lane == 0) {
      constexpr uint32_t idesc1 = idesc_f16(128, FS_NPAD, 1, 0);
      const uint64_t ad_ring = smem_desc(smem_u32(ring), FT_STAGE_BYTES / 2, 1024, kLayoutSw128);
      const uint64_t bd_x = smem_desc(smem_u32(xbuf), 16, 1024, kLayoutSw128);
      uint32_t s = 0, sph = 0, b = 0, bph = 0;      // ring stage / D1 buffer and their phases: counted, never divided
      uint32_t a = 0, aph = 0;
      for (int n = 0; n < my_items; ++n, (++a == FS_AUX ? (a = 0, aph ^= 1) : 0u)) {
        wait_or_give_up(&sh->aux_full[a], aph, abortp, status, 62);
        const uint64_t bd0 = bd_x + (uint64_t)(a * (FS_XBYTES >> 4));
        const uint64_t bd1 = bd0 + (uint64_t)(FS_XBYTES >> 5);
        for (int c = 0; c < nchunk; ++c) {
          wait_or_give_up(&sh->full[s], sph, abortp, status, 63);
          wait_or_give_up(&sh->d1_free[b], bph ^ 1, abortp, status, 64);
          if (*abortp) break;
          tc_fence_after_sync();
          const uint64_t ad0 = ad_ring + (uint64_t)(s * (FT_STAGE_BYTES >> 4));
#pragma unroll
          for (int ks = 0; ks < kHeadDim / 16; ++ks)
            mma_f16_ss(tmem + b * FS_NPAD, ad0 + (uint64_t)(ks * (2048 >> 4)),
                       (ks < 4 ? bd0 : bd1) + (uint64_t)((ks & 3) * 2), idesc1, ks ? 1u : 0u);
          mma_commit(&sh->empty[s]);
          mma_commit(&sh->d1_full[b]);
          if (++s == (uint32_t)nstage) { s = 0; sph ^= 1; }
          if (++b == FS_BUFS) { b = 0; bph ^= 1; }
        }
        if (*abortp) break;
        mma_commit(&sh->aux_empty[a]);
      }
    }
  } else {
    // ---------------- epilogue warps ----------------
    // No early exit here: the warps meet at named barriers, so after a timed-out wait they keep
    // walking their items (every later wait returns at once) and the CTA ends normally.
    const int ew = warp - 2, quad = warp & 3, hf = ew >> 2;
    const int j = quad * 32 + lane;            // hidden unit inside a chunk = accumulator lane
    const int et = tid - 64;                   // 0..255
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    uint32_t a = 0, aph = 0;
    for (int n = 0; n < my_items; ++n, (++a == FS_AUX ? (a = 0, aph ^= 1) : 0u)) {
      const int it = blockIdx.x + n * gridDim.x;
      const FtItem im = ft_item(it, gm);
      const int tile = im.tile, which = im.which, lh = im.lh;
      const int b0 = tile * FS_NPAD, nb = min(NT, p.B - b0);
      float c1 = 1.f, c2 = 1.f;
      if (which && p.psi_scale) { c1 = __ldg(p.psi_scale + lh * 2); c2 = __ldg(p.psi_scale + lh * 2 + 1); }
      wait_or_give_up(&sh->aux_full[a], aph, abortp, status, 65);
      float part[V];
#pragma unroll
      for (int e = 0; e < V; ++e) part[e] = 0.f;
      // the two warps of a lane quadrant take alternate chunks
      for (int c = hf; c < nchunk; c += 2) {
        const uint32_t q = (uint32_t)n * nchunk + c, b = q % FS_BUFS;
        wait_or_give_up(&sh->d1_full[b], (q / FS_BUFS) & 1, abortp, status, 66);
        tc_fence_after_sync();
        uint32_t acc[8];
        tmem_ld8(lane_addr + b * FS_NPAD, acc);
        tmem_ld_wait();
        tc_fence_before_sync();
        mbar_arrive_warp(&sh->d1_free[b]);
        float w[R];
        const uint4* wr = reinterpret_cast<const uint4*>(w2raw + a * w2bytes + (size_t)(c * FT_CHUNK + j) * R * 2);
#pragma unroll
        for (int r8 = 0; r8 < R / 8; ++r8) half8_to_float(wr[r8], w + r8 * 8);
#pragma unroll
        for (int t = 0; t < NT; ++t) {
          const float h = t < nb ? c1 * gelu_erf(__uint_as_float(acc[t])) : 0.f;
#pragma unroll
          for (int r = 0; r < R; ++r) part[t * R + r] = fmaf(h, w[r], part[t * R + r]);
        }
      }
      int base, count;
      bool owner;
      lane_reduce_scatter<V>(part, lane, base, count, owner);
      float* red = &sh->red[n & 1][ew][0];
      if (owner) {
#pragma unroll
        for (int i = 0; i < (V >= 32 ? V / 32 : 1); ++i) red[base + i] = part[i];
      }
      epi_sync();
      float gv = 0.f;
      if (et < V) {
        float sum = 0.f;
#pragma unroll
        for (int wq = 0; wq < FT_EPI_WARPS; ++wq) sum += sh->red[n & 1][wq][et];   // fixed order
        gv = c2 * gelu_erf(sum);
      }
      const int t = et / R, r = et % R;
      if (which) {
        if (et < V) sh->g[n & 1][et] = gv;
        epi_sync();
        if (et < V) {
          const __half* w3 = &sh->w3[a][0];
          float sacc = 0.f;
#pragma unroll
          for (int rr = 0; rr < R; ++rr) sacc = fmaf(sh->g[n & 1][t * R + rr], __half2float(w3[rr * R + r]), sacc);
          gv = sacc;
        }
      }
      if (et < V && t < nb) p.out[which][((size_t)(b0 + t) * p.L * p.Hh[which] + lh) * R + r] = fabsf(gv);
      if (ew * 32 < V) publish_rows(p, which, lh);         // ceil(V / 32) writer warps per item
      // this warp is done with the item's W2 and W3
      mbar_arrive_warp(&sh->aux_empty[a]);
    }
  }
  drain_after_abort(abortp);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, FS_BUFS * FS_NPAD);
}

template <int R, int NT>
static int launch_small(less_ctx* c, const FmParams& p, const FtGeom& gm, const CUtensorMap& tq, const CUtensorMap& tk,
                        const CUtensorMap& tw1a, const CUtensorMap& tw1b, size_t smem, int grid, cudaStream_t s) {
  auto kern = feature_tc_small_kernel<R, NT>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return fail_cuda("shared memory opt-in of feature_tc_small_kernel");
  if (!gm.late_inputs) {
    kern<<<grid, FT_THREADS, smem, s>>>(tq, tk, tw1a, tw1b, p, gm, c->a.status);
    return check_launch("feature_tc_small_kernel");
  }
  // as a programmatic dependent of the kernel before it in the stream (the decode kernel of the step before,
  // typically): its CTAs come up and fetch their first weights while that kernel finishes
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(FT_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int32_t* status = c->a.status;
  if (cudaLaunchKernelEx(&cfg, kern, tq, tk, tw1a, tw1b, p, gm, status) != cudaSuccess)
    return fail_cuda("launch of feature_tc_small_kernel");
  return check_launch("feature_tc_small_kernel");
}

// whether a decode step of this context runs a tensor-core feature kernel (they take a layer range), and
// whether it is the small-batch one (which can fetch the step's q, k rows with plain loads)
bool feature_tc_path(const less_ctx* c) {
  const Dims& d = c->d;
  return !d.general && !(d.flags & LESS_NO_STATE) && (c->feature_path == 2 || d.G > 1) && feature_tc_supported(d);
}
bool feature_small_tc_path(const less_ctx* c) { return feature_tc_path(c) && c->d.B <= 8; }

bool feature_tc_supported(const Dims& d) {
  return (d.Rp == 128 || d.Rp == 256 || d.Rp == 512) && encode_tiled_fn() != nullptr;
}

static size_t ft_fixed_smem(const Dims& d, int npad) {
  return (size_t)(2 * FL_GROUPS + 2) * npad * 256 + (size_t)(d.R == 16 ? 4 : 2) * d.Rp * d.R * 2 + sizeof(FtShared) + 1024;
}

int launch_feature_tc(less_ctx* c, const FmParams& p_in, cudaStream_t s) {
  const Dims& d = c->d;
  FmParams p = p_in;
  FtGeom gm;
  // token tiles of at most 64: larger tiles leave too little shared memory for the weight ring
  gm.npad = d.B <= 16 ? 16 : d.B <= 32 ? 32 : 64;
  gm.ntile = (d.B + gm.npad - 1) / gm.npad;
  gm.G = d.G;
  gm.per_head = (d.G + 1) * gm.ntile;
  gm.kv0 = p.lh0;
  gm.items = p.nlh * gm.per_head;
  // The kernel is launched as a programmatic dependent of the kernel before it in the stream - the decode
  // kernel of the step before, typically, which lets its dependents go when it starts: the CTAs come up on
  // multiprocessors as that kernel drains from them (they need most of a multiprocessor's shared memory, so
  // they never displace its CTAs) and fetch their first weights meanwhile.
  gm.late_inputs = (c->pdl && !c->profile && !c->head_counters) ? 1 : 0;
  const size_t fixed = ft_fixed_smem(d, gm.npad);
  int ns = (int)((FT_SMEM_LIMIT - fixed) / FT_STAGE_BYTES);
  gm.nstage = ns > FT_MAX_STAGES ? FT_MAX_STAGES : ns;
  // With the overlap on, the ring gives up stages so that decode CTAs of the same step fit beside
  // this kernel's CTA on every SM (at these batch sizes the kernel is bound by its epilogue, not
  // by the weight stream: three stages feed it).
  const int cap_l = c->feature_stages >= 2 ? c->feature_stages : (c->pdl && (c->head_counters || d.I <= 8 * c->sms) ? 3 : FT_MAX_STAGES);
  if (gm.nstage > cap_l) gm.nstage = cap_l;
  if (gm.nstage < 2) return LESS_ERR_INVALID_CONFIG;
  const uint32_t need = 2u * gm.npad + 16u;
  gm.tmem_cols = need <= 64 ? 64 : need <= 128 ? 128 : need <= 256 ? 256 : 512;
  const size_t smem = fixed + (size_t)gm.nstage * FT_STAGE_BYTES;

  static_assert(sizeof(CUtensorMap) <= 128, "tensor map cache slot");
  CUtensorMap* tmc = reinterpret_cast<CUtensorMap*>(c->tm_cache);
  CUtensorMap &tq = tmc[0], &tk = tmc[1], &tw1a = tmc[2], &tw1b = tmc[3];
  const uint64_t lhq = (uint64_t)d.L * p.Hh[0], lhk = (uint64_t)d.L * p.Hh[1];   // layer-heads of phi / psi
  // q, k: [B rows][L*Hd*128 columns]; a box is `box` batch rows x 64 columns of one head (the small
  // kernel loads 8 input rows per half tile).  The maps are kept in the context between steps.
  const int box = d.B <= 8 ? FS_XROWS : gm.npad;
  if (c->tm_box != box || c->tm_q != p.x[0] || c->tm_k != p.x[1]) {
    c->tm_box = 0;
    if (!make_tmap_f16_2d(&tq, p.x[0], d.B, lhq * kHeadDim, lhq * kHeadDim * 2, box) ||
        !make_tmap_f16_2d(&tk, p.x[1], d.B, lhk * kHeadDim, lhk * kHeadDim * 2, box))
      return fail_cuda("tensor map of q / k");
    c->tm_q = p.x[0]; c->tm_k = p.x[1]; c->tm_box = box;
  }
  if (!c->tm_w_ok) {
    if (!make_tmap_f16_2d(&tw1a, p.w1[0], lhq * kHeadDim, d.Rp, (uint64_t)d.Rp * 2, kHeadDim) ||
        !make_tmap_f16_2d(&tw1b, p.w1[1], lhk * kHeadDim, d.Rp, (uint64_t)d.Rp * 2, kHeadDim))
      return fail_cuda("tensor map of W1");
    c->tm_w_ok = true;
  }
  int sms = c->sms;
  if (c->feature_ctas > 0 && c->feature_ctas < sms) sms = c->feature_ctas;
  const int grid = gm.items < sms ? gm.items : sms;
  const int nt = d.B <= 1 ? 1 : d.B <= 2 ? 2 : d.B <= 4 ? 4 : 8;
  // Per-head counters, so that any number of decode CTAs can follow this kernel as programmatic
  // dependents, each waiting for its own head's feature maps only.  Off unless LESS_HEAD_COUNTERS is
  // set: measured on 64 x 1024 heads x 204 slots the overlap gains nothing (1.337 ms per step with it,
  // 1.325 ms without; feature grids of 24 to 148 CTAs all within 1 %) - at that size the decode kernel
  // is bound by what the SMs can keep in flight, not by HBM, so every SM-microsecond the feature
  // kernel takes is lost to it wherever it is scheduled - and with grouped query heads it costs
  // (8192 KV heads x 2 query heads: 1.02 ms against 0.86 ms).  Direct calls only (a captured step
  // would replay a stale target).  Never behind the small-batch kernel with more instances than fit
  // the GPU at once: that kernel is bound by its weight stream, and successive waves of decode CTAs
  // take so much of the bandwidth from it that the feature maps they wait for arrive later than
  // without the overlap (measured, 4 x 1600 heads x 654 slots: 533 us per step against 486).
  // Every flagged launch adds the same number of writer warps to every head's counter, so the target
  // is one running total.
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  cudaStreamIsCapturing(s, &capturing);
  const bool many = d.I > 8 * c->sms;
  if (capturing == cudaStreamCaptureStatusNone && c->pdl && c->head_counters && many && d.B > 8) {
    uint32_t writers = 0;
    if (d.B <= 8) writers = (uint32_t)(nt * d.R + 31) / 32;
    else
      for (int t = 0; t < gm.ntile; ++t) writers += (uint32_t)(((d.B - t * gm.npad < gm.npad ? d.B - t * gm.npad : gm.npad) + 31) / 32);
    p.feat_flag = c->a.feat_flag;
    c->flag_target[0] += writers;
    c->flag_target[1] += writers;
    c->flags_this_step = true;
  }
  char name[64];
  if (d.B <= 8) snprintf(name, sizeof name, "feature_tc_small_kernel<%d, %d>", d.R, nt);
  else snprintf(name, sizeof name, "feature_tc_kernel<%d>", d.R);
  LaunchScope scope(c, LESS_KERNEL_FEATURE_MAP, s, name);
  if (d.B <= 8) {
    const size_t shared_struct = sizeof(FsShared<1>) + (size_t)(2 * FT_EPI_WARPS + 2) * (nt * d.R - 1) * 4;
    const size_t fx = 8192 + (size_t)FS_AUX * d.Rp * d.R * 2 + shared_struct + 256;
    const int nsm = (int)((FT_SMEM_LIMIT - fx) / FT_STAGE_BYTES);
    gm.nstage = nsm > FT_MAX_STAGES ? FT_MAX_STAGES : nsm;
    // With the overlap on, one stage of the ring is given up so that the decode kernel's CTAs of
    // the same step fit beside this kernel's CTA on every SM (measured on the Llama-2-7B shape at
    // batch 1: 83.5 us per step with 6 stages and no room, 74.5 us with 5, 74.2 us with 4).
    const int cap = c->feature_stages >= 2 ? c->feature_stages : (c->pdl && !many ? 5 : FT_MAX_STAGES);
    if (gm.nstage > cap) gm.nstage = cap;
    if (gm.nstage < 2) return LESS_ERR_INVALID_CONFIG;
    const size_t sm = fx + (size_t)gm.nstage * FT_STAGE_BYTES;
    if (d.R == 8) {
      if (nt == 1) return launch_small<8, 1>(c, p, gm, tq, tk, tw1a, tw1b, sm, grid, s);
      if (nt == 2) return launch_small<8, 2>(c, p, gm, tq, tk, tw1a, tw1b, sm, grid, s);
      if (nt == 4) return launch_small<8, 4>(c, p, gm, tq, tk, tw1a, tw1b, sm, grid, s);
      return launch_small<8, 8>(c, p, gm, tq, tk, tw1a, tw1b, sm, grid, s);
    }
    if (nt == 1) return launch_small<16, 1>(c, p, gm, tq, tk, tw1a, tw1b, sm, grid, s);
    if (nt == 2) return launch_small<16, 2>(c, p, gm, tq, tk, tw1a, tw1b, sm, grid, s);
    if (nt == 4) return launch_small<16, 4>(c, p, gm, tq, tk, tw1a, tw1b, sm, grid, s);
    return launch_small<16, 8>(c, p, gm, tq, tk, tw1a, tw1b, sm, grid, s);
  }
  auto kern = d.R == 8 ? feature_tc_kernel<8> : feature_tc_kernel<16>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return fail_cuda("shared memory opt-in of feature_tc_kernel");
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(FL_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = gm.late_inputs ? 1 : 0;
  int32_t* status = c->a.status;
  if (cudaLaunchKernelEx(&cfg, kern, tq, tk, tw1a, tw1b, p, gm, status) != cudaSuccess)
    return fail_cuda("launch of feature_tc_kernel");
  return check_launch("feature_tc_kernel");
}

}  // namespace less
