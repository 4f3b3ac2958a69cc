// Prompt scoring on the tensor cores (Section 3.1: the prompt phase is regular causal
// attention; Section 2.1: H2O accumulates the attention probabilities):
//   rowstat_tc_kernel   m_i, 1 / l_i of causal row i of Q K^T / sqrt(D)
//   colsum_tc_kernel    acc_j = sum_{i >= j} exp(s_ij - m_i) / l_i
//
// Both stream 256-row tiles of the other operand past one resident 128-row tile and
// compute 128 x 256 tiles of raw dot products with tcgen05 (kind::f16, fp16 inputs used
// exactly, fp32 accumulators double-buffered in tensor memory); sixteen epilogue warps read
// the tiles back (lane = row of the resident tile) and reduce them.
//
// Row statistics: resident Q tile, streamed K tiles up to the diagonal, online max / sum.
//
// Column sums: resident K tile (lane = key j), streamed Q tiles from the diagonal on.  The
// per-row constants are folded into the contraction, so the epilogue is one multiply, one
// exp2 and one add per element:
//     p_ij = exp2( c (q_i . k_j - b_i) ),   c = log2(e) / sqrt(D),   b_i = m_i sqrt(D) - log2(1 / l_i) / c
// A ninth k-step multiplies a column of ones on the key side with (-b_i), split into three
// fp16 parts, on the query side; the row-statistics kernel leaves those parts in the workspace
// in operand layout (16 bytes per row), so they arrive with one bulk copy per tile.  Rows past
// the prompt get b = +60000, which turns them into exact zeros.  Only the tile on the diagonal
// needs a per-element causal test.
// Every wait is bounded (pipeline.cuh).
#include "prefill.cuh"
#include "tc_common.cuh"

namespace less {

constexpr int SC_EPI_WARPS = 16;                   // four per lane quadrant: with two, the tensor-memory loads of a
                                                  // tile's column groups were exposed and the XU idled a fifth of the time
constexpr int SC_PARTS = SC_EPI_WARPS / 4;        // warps that split a tile's 256 columns
constexpr int SC_PART_COLS = 256 / SC_PARTS;      // columns per warp (64)
constexpr int SC_PART_GROUPS = SC_PART_COLS / 32; // 32-column loads per warp and tile
constexpr int SC_EPI_THREADS = SC_EPI_WARPS * 32;
constexpr int SC_TILE_M = 128;                    // rows of the resident tile
constexpr int SC_TILE_N = 256;                    // rows of a streamed tile
constexpr int SC_RES_BYTES = SC_TILE_M * kHeadDim * 2;
constexpr int SC_STAGE_BYTES = SC_TILE_N * kHeadDim * 2;
constexpr int SC_STAGES = 2;
constexpr float kRawScale = 0.08838834764831845f;             // 1 / sqrt(128)
constexpr float kExpScale = 0.12751743074602468f;             // log2(e) / sqrt(128)

struct ScShared {
  uint64_t res_full;
  uint64_t full[SC_STAGES], empty[SC_STAGES];
  uint64_t d_full[2], d_free[2];
  uint32_t tmem_base;
  int abort;
  float merge[SC_PARTS][SC_TILE_M][2];
};

__device__ __forceinline__ void sc_epi_sync() { asm volatile("bar.sync 1, %0;" ::"n"(SC_EPI_THREADS) : "memory"); }

// -b as three fp16 parts (k = 0, 1, 2 of the ninth k-step), the row's other 5 halves zero
__device__ __forceinline__ uint4 pack_neg_b(float nb) {
  const __half h0 = __float2half_rn(nb);
  const float r1 = nb - __half2float(h0);
  const __half h1 = __float2half_rn(r1);
  const __half h2 = __float2half_rn(r1 - __half2float(h1));
  return make_uint4((uint32_t)__half_as_ushort(h0) | ((uint32_t)__half_as_ushort(h1) << 16),
                    (uint32_t)__half_as_ushort(h2), 0u, 0u);
}

// three-input maximum (one instruction on sm_100): halves the instructions of the row-maximum pass
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ------------------------------------------------------------------------------------------- //
// P1: row statistics.  warp 0 TMA, warp 1 MMA, warps 2..9 epilogue.
// ------------------------------------------------------------------------------------------- //
constexpr int RS_THREADS = 64 + SC_EPI_THREADS;

__global__ void __launch_bounds__(RS_THREADS) rowstat_tc_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                                const __grid_constant__ CUtensorMap tm_k, PfParams p) {
  extern __shared__ __align__(1024) unsigned char sc_smem[];
  if (smem_misaligned(sc_smem, p.a.status, 80)) return;
  unsigned char* qres = sc_smem;                                 // [2 halves][128 rows][128 B]
  unsigned char* ring = qres + SC_RES_BYTES;                     // [stages][2 halves][256 rows][128 B]
  ScShared* sh = reinterpret_cast<ScShared*>(ring + SC_STAGES * SC_STAGE_BYTES);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles = (p.S + SC_TILE_M - 1) / SC_TILE_M;
  const int tile = tiles - 1 - (int)blockIdx.x;                  // long rows first
  const int g = blockIdx.y;                                      // query head (KV instance * grp + head of the group)
  const QueryMap qm = map_query(p, g);
  const int i0 = tile * SC_TILE_M;
  const int ncol = min(p.S, i0 + SC_TILE_M);                     // causal: columns [0, ncol)
  const int ntile = (ncol + SC_TILE_N - 1) / SC_TILE_N;
  int32_t* status = p.a.status;

  if (tid == 0) {
    mbar_init(&sh->res_full, 1);
    for (int s = 0; s < SC_STAGES; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh->d_full[s], 1);
      mbar_init(&sh->d_free[s], SC_EPI_WARPS);
    }
    sh->abort = *reinterpret_cast<volatile int32_t*>(status) != 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&sh->tmem_base, 512);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh->tmem_base;
  volatile int* abortp = &sh->abort;

  if (warp == 0) {
    if (lane == 0) {
      const int row0 = (int)(qm.q_row0 + i0);
      mbar_expect_tx(&sh->res_full, SC_RES_BYTES);
      tma_load_2d(qres, &tm_q, 0, row0, &sh->res_full);
      tma_load_2d(qres + SC_RES_BYTES / 2, &tm_q, 64, row0, &sh->res_full);
      uint32_t s = 0, ph = 0;
      for (int t = 0; t < ntile; ++t) {
        wait_or_give_up(&sh->empty[s], ph ^ 1, abortp, status, 80);
        if (*abortp) break;
        const int krow = (int)(qm.kv_row0 + (size_t)t * SC_TILE_N);
        unsigned char* st = ring + s * SC_STAGE_BYTES;
        mbar_expect_tx(&sh->full[s], SC_STAGE_BYTES);
        tma_load_2d(st, &tm_k, 0, krow, &sh->full[s]);
        tma_load_2d(st + SC_STAGE_BYTES / 2, &tm_k, 64, krow, &sh->full[s]);
        if (++s == SC_STAGES) { s = 0; ph ^= 1; }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_f16(SC_TILE_M, SC_TILE_N, 0, 0);
      const uint64_t ad0 = smem_desc(smem_u32(qres), 16, 1024, kLayoutSw128);
      const uint64_t bd_ring = smem_desc(smem_u32(ring), 16, 1024, kLayoutSw128);
      wait_or_give_up(&sh->res_full, 0, abortp, status, 81);
      uint32_t s = 0, ph = 0, b = 0, bph = 0;
      for (int t = 0; t < ntile; ++t) {
        wait_or_give_up(&sh->full[s], ph, abortp, status, 82);
        wait_or_give_up(&sh->d_free[b], bph ^ 1, abortp, status, 83);
        if (*abortp) break;
        tc_fence_after_sync();
        const uint64_t bd0 = bd_ring + (uint64_t)(s * (SC_STAGE_BYTES >> 4));
#pragma unroll
        for (int ks = 0; ks < kHeadDim / 16; ++ks)
          mma_f16_ss(tmem + b * SC_TILE_N, ad0 + (uint64_t)((ks >> 2) * (SC_RES_BYTES >> 5) + (ks & 3) * 2),
                     bd0 + (uint64_t)((ks >> 2) * (SC_STAGE_BYTES >> 5) + (ks & 3) * 2), idesc, ks ? 1u : 0u);
        mma_commit(&sh->empty[s]);
        mma_commit(&sh->d_full[b]);
        if (++s == SC_STAGES) { s = 0; ph ^= 1; }
        if (b ^= 1, b == 0) bph ^= 1;
      }
    }
  } else {
    // ---- epilogue: lane = row of the Q tile; the four warps of a lane quadrant split the columns ----
    const int quad = warp & 3, half = (warp - 2) >> 2;      // half: which SC_PART_COLS columns of a tile
    const int r = quad * 32 + lane, i = i0 + r;
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16) + half * SC_PART_COLS;
    float m = -INFINITY, l = 0.f;                      // m in raw dot-product units
    uint32_t b = 0, bph = 0;
    for (int t = 0; t < ntile; ++t) {
      wait_or_give_up(&sh->d_full[b], bph, abortp, status, 84);
      tc_fence_after_sync();
      const int c0 = t * SC_TILE_N + half * SC_PART_COLS;
      const bool edge = t == ntile - 1;                // only the last tile meets the diagonal or the prompt's end
#pragma unroll 1
      for (int cg = 0; cg < SC_PART_GROUPS; ++cg) {
        uint32_t v[32];
        tmem_ld32(lane_addr + b * SC_TILE_N + cg * 32, v);
        tmem_ld_wait();
        const int cbase = c0 + cg * 32;
        float tmax = -INFINITY;
        if (edge) {
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const int j = cbase + e;
            if (j > i || j >= p.S) v[e] = 0xff800000u;   // -inf: outside the causal row
            tmax = fmaxf(tmax, __uint_as_float(v[e]));
          }
        } else {
#pragma unroll
          for (int e = 0; e < 32; e += 2) tmax = max3(tmax, __uint_as_float(v[e]), __uint_as_float(v[e + 1]));
        }
        if (tmax > m) {
          l *= ex2_approx((m - tmax) * kExpScale);       // m = -inf the first time: l = 0 stays 0
          m = tmax;
        }
        if (m > -INFINITY) {
          const float mc = m * kExpScale;
          float acc = 0.f;
#pragma unroll
          for (int e = 0; e < 32; ++e) acc += ex2_approx(fmaf(__uint_as_float(v[e]), kExpScale, -mc));
          l += acc;
        }
      }
      tc_fence_before_sync();
      mbar_arrive_warp(&sh->d_free[b]);
      if (b ^= 1, b == 0) bph ^= 1;
    }
    // merge the column parts of a row
    sh->merge[half][r][0] = m;
    sh->merge[half][r][1] = l;
    sc_epi_sync();
    if (half == 0 && i < p.S && !*abortp) {
      float mm = -INFINITY;
#pragma unroll
      for (int h = 0; h < SC_PARTS; ++h) mm = fmaxf(mm, sh->merge[h][r][0]);
      float lt = 0.f;
#pragma unroll
      for (int h = 0; h < SC_PARTS; ++h) {
        const float mh = sh->merge[h][r][0];
        if (mh > -INFINITY) lt += sh->merge[h][r][1] * ex2_approx((mh - mm) * kExpScale);
      }
      const float il = 1.0f / lt;
      p.a.ws_m[(size_t)g * p.Sp + i] = mm * kRawScale;
      p.a.ws_invl[(size_t)g * p.Sp + i] = il;
      p.a.ws_bx[(size_t)g * p.Sbx + i] = pack_neg_b(-(mm - log2f(il) * (1.0f / kExpScale)));
    }
    // rows between the prompt's end and the end of its last 256-row tile: exact zeros in the column sums
    if (half == 0 && tile == tiles - 1 && !*abortp)
      for (int x = p.S + r; x < ((p.S + SC_TILE_N - 1) & ~(SC_TILE_N - 1)); x += SC_TILE_M)
        p.a.ws_bx[(size_t)g * p.Sbx + x] = pack_neg_b(-60000.f);
  }
  drain_after_abort(abortp);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------- //
// P2: column sums.  warp 0 TMA, warp 1 MMA, warps 2..9 epilogue.
// ------------------------------------------------------------------------------------------- //
constexpr int CS_THREADS = 64 + SC_EPI_THREADS;
constexpr int SC_BX_BYTES = SC_TILE_N * 16;        // one stage: [32 row groups][8 rows][16 B], k = 0..7 of the ninth k-step
constexpr int SC_BXZ_BYTES = SC_STAGES * SC_BX_BYTES;   // zeros: k = 8..15, at the same offset behind every stage
constexpr int SC_ONES_BYTES = SC_TILE_M * 32;      // [16 row groups][2 k halves][8 rows][16 B]

__global__ void __launch_bounds__(CS_THREADS) colsum_tc_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                               const __grid_constant__ CUtensorMap tm_k, PfParams p) {
  extern __shared__ __align__(1024) unsigned char sc_smem[];
  if (smem_misaligned(sc_smem, p.a.status, 80)) return;
  unsigned char* kres = sc_smem;                                 // resident K tile
  unsigned char* ring = kres + SC_RES_BYTES;                     // streamed Q tiles
  unsigned char* bx = ring + SC_STAGES * SC_STAGE_BYTES;         // [stages] (-b_i) columns of the Q tiles, then zeros
  unsigned char* ones = bx + SC_STAGES * SC_BX_BYTES + SC_BXZ_BYTES;   // ones columns of the K tile
  ScShared* sh = reinterpret_cast<ScShared*>(ones + SC_ONES_BYTES);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x, g = blockIdx.y;                   // low key tiles (long columns) first
  const InstMap im = map_instance(p, g);
  const int j0 = tile * SC_TILE_M;
  const int t0 = j0 / SC_TILE_N;                                 // first Q tile: the one that holds row j0
  const int ntile = (p.S + SC_TILE_N - 1) / SC_TILE_N - t0;      // Q tiles of one query head
  const int nstream = ntile * p.grp;                             // the heads of the group one after the other
  int32_t* status = p.a.status;

  if (tid == 0) {
    mbar_init(&sh->res_full, 1);
    for (int s = 0; s < SC_STAGES; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh->d_full[s], 1);
      mbar_init(&sh->d_free[s], SC_EPI_WARPS);
    }
    sh->abort = *reinterpret_cast<volatile int32_t*>(status) != 0;
    mbar_fence_init();
  }
  // constant parts of the ninth k-step: zeros for k = 8..15 of the query side; on the key side
  // ones (1, 1, 1, 0 ...) for k = 0..7 and zeros for k = 8..15
  for (int e = tid; e < (SC_BXZ_BYTES + SC_ONES_BYTES) / 16; e += CS_THREADS) {
    uint4 v = make_uint4(0, 0, 0, 0);
    const int unit = e - SC_BXZ_BYTES / 16;                      // 16-byte unit inside the ones block
    if (unit >= 0 && ((unit >> 3) & 1) == 0) v = make_uint4(0x3c003c00u, 0x00003c00u, 0, 0);   // fp16 1, 1, 1, 0 ...
    *reinterpret_cast<uint4*>(bx + SC_STAGES * SC_BX_BYTES + e * 16) = v;
  }
  if (warp == 1) tmem_alloc(&sh->tmem_base, 512);
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh->tmem_base;
  volatile int* abortp = &sh->abort;

  if (warp == 0) {
    if (lane == 0) {
      const int row0 = (int)(im.in_row0 + j0);
      mbar_expect_tx(&sh->res_full, SC_RES_BYTES);
      tma_load_2d(kres, &tm_k, 0, row0, &sh->res_full);
      tma_load_2d(kres + SC_RES_BYTES / 2, &tm_k, 64, row0, &sh->res_full);
      uint32_t s = 0, ph = 0;
      for (int qg = 0; qg < p.grp; ++qg) {
        const int gq = g * p.grp + qg;
        const size_t q_row0 = map_query(p, gq).q_row0;
        for (int t = 0; t < ntile; ++t) {
          wait_or_give_up(&sh->empty[s], ph ^ 1, abortp, status, 85);
          if (*abortp) break;
          const int qrow = (int)(q_row0 + (size_t)(t0 + t) * SC_TILE_N);
          unsigned char* st = ring + s * SC_STAGE_BYTES;
          mbar_expect_tx(&sh->full[s], SC_STAGE_BYTES + SC_BX_BYTES);
          tma_load_2d(st, &tm_q, 0, qrow, &sh->full[s]);
          tma_load_2d(st + SC_STAGE_BYTES / 2, &tm_q, 64, qrow, &sh->full[s]);
          bulk_g2s(bx + s * SC_BX_BYTES, p.a.ws_bx + (size_t)gq * p.Sbx + (size_t)(t0 + t) * SC_TILE_N, SC_BX_BYTES,
                   &sh->full[s]);
          if (++s == SC_STAGES) { s = 0; ph ^= 1; }
        }
        if (*abortp) break;
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_f16(SC_TILE_M, SC_TILE_N, 0, 0);
      const uint64_t ad0 = smem_desc(smem_u32(kres), 16, 1024, kLayoutSw128);
      const uint64_t bd_ring = smem_desc(smem_u32(ring), 16, 1024, kLayoutSw128);
      const uint64_t ad_ones = smem_desc(smem_u32(ones), 128, 256, kLayoutNone);
      const uint64_t bd_bx = smem_desc(smem_u32(bx), SC_STAGES * SC_BX_BYTES, 128, kLayoutNone);
      wait_or_give_up(&sh->res_full, 0, abortp, status, 86);
      uint32_t s = 0, ph = 0, b = 0, bph = 0;
      for (int t = 0; t < nstream; ++t) {
        wait_or_give_up(&sh->full[s], ph, abortp, status, 87);
        wait_or_give_up(&sh->d_free[b], bph ^ 1, abortp, status, 89);
        if (*abortp) break;
        tc_fence_after_sync();
        const uint64_t bd0 = bd_ring + (uint64_t)(s * (SC_STAGE_BYTES >> 4));
#pragma unroll
        for (int ks = 0; ks < kHeadDim / 16; ++ks)
          mma_f16_ss(tmem + b * SC_TILE_N, ad0 + (uint64_t)((ks >> 2) * (SC_RES_BYTES >> 5) + (ks & 3) * 2),
                     bd0 + (uint64_t)((ks >> 2) * (SC_STAGE_BYTES >> 5) + (ks & 3) * 2), idesc, ks ? 1u : 0u);
        mma_f16_ss(tmem + b * SC_TILE_N, ad_ones, bd_bx + (uint64_t)(s * (SC_BX_BYTES >> 4)), idesc, 1u);
        mma_commit(&sh->empty[s]);
        mma_commit(&sh->d_full[b]);
        if (++s == SC_STAGES) { s = 0; ph ^= 1; }
        if (b ^= 1, b == 0) bph ^= 1;
      }
    }
  } else {
    // ---- epilogue: lane = key of the K tile; the four warps of a lane quadrant split the rows i ----
    const int quad = warp & 3, half = (warp - 2) >> 2;
    const int r = quad * 32 + lane, j = j0 + r;
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16) + half * SC_PART_COLS;
    float acc = 0.f;
    uint32_t b = 0, bph = 0;
    for (int ts = 0, t = 0; ts < nstream; ++ts, t = (t + 1 == ntile ? 0 : t + 1)) {   // t: tile within the head
      wait_or_give_up(&sh->d_full[b], bph, abortp, status, 91);
      tc_fence_after_sync();
      const int c0 = (t0 + t) * SC_TILE_N + half * SC_PART_COLS;
#pragma unroll 1
      for (int cg = 0; cg < SC_PART_GROUPS; ++cg) {
        uint32_t v[32];
        tmem_ld32(lane_addr + b * SC_TILE_N + cg * 32, v);
        tmem_ld_wait();
        const int ibase = c0 + cg * 32;
        float a = 0.f;
        if (t == 0) {                                   // the tile that holds the diagonal
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float pe = ex2_approx(__uint_as_float(v[e]) * kExpScale);
            a += (ibase + e >= j) ? pe : 0.f;
          }
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) a += ex2_approx(__uint_as_float(v[e]) * kExpScale);
        }
        acc += a;
      }
      tc_fence_before_sync();
      mbar_arrive_warp(&sh->d_free[b]);
      if (b ^= 1, b == 0) bph ^= 1;
    }
    sh->merge[half][r][0] = acc;
    sc_epi_sync();
    if (half == 0 && j < p.S && !*abortp) {
      float total = 0.f;
#pragma unroll
      for (int h = 0; h < SC_PARTS; ++h) total += sh->merge[h][r][0];      // fixed order
      p.a.ws_acc[(size_t)g * p.Sp + j] = total;
    }
  }
  drain_after_abort(abortp);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

bool score_tc_supported() { return encode_tiled_fn() != nullptr; }

int launch_score_tc(less_ctx* c, const PfParams& p, int G, cudaStream_t s, bool with_column_sums) {
  const Dims& d = c->d;
  CUtensorMap tq, tk;
  const uint64_t rows = (uint64_t)d.B * p.layer_count * d.Hd * p.S, qrows = rows * p.grp;
  if (!make_tmap_f16_2d(&tq, p.Q, qrows, kHeadDim, kHeadDim * 2, SC_TILE_N) ||
      !make_tmap_f16_2d(&tk, p.K, rows, kHeadDim, kHeadDim * 2, SC_TILE_N))
    return fail_cuda("tensor maps of Q / K");
  CUtensorMap tq_res, tk_res;
  if (!make_tmap_f16_2d(&tq_res, p.Q, qrows, kHeadDim, kHeadDim * 2, SC_TILE_M) ||
      !make_tmap_f16_2d(&tk_res, p.K, rows, kHeadDim, kHeadDim * 2, SC_TILE_M))
    return fail_cuda("tensor maps of Q / K");
  const int tiles = (p.S + SC_TILE_M - 1) / SC_TILE_M;
  const size_t smem1 = SC_RES_BYTES + SC_STAGES * SC_STAGE_BYTES + sizeof(ScShared) + 1024;
  const size_t smem2 = smem1 + SC_STAGES * SC_BX_BYTES + SC_BXZ_BYTES + SC_ONES_BYTES;
  if (cudaFuncSetAttribute(rowstat_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1) != cudaSuccess ||
      cudaFuncSetAttribute(colsum_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2) != cudaSuccess)
    return fail_cuda("shared memory opt-in of the scoring kernels");
  {
    LaunchScope scope(c, LESS_KERNEL_ROWSTAT, s, "rowstat_tc_kernel");
    rowstat_tc_kernel<<<dim3(tiles, G * p.grp), RS_THREADS, smem1, s>>>(tq_res, tk, p);   // one row of CTAs per query head
  }
  if (with_column_sums) {
    LaunchScope scope(c, LESS_KERNEL_COLSUM, s, "colsum_tc_kernel");
    colsum_tc_kernel<<<dim3(tiles, G), CS_THREADS, smem2, s>>>(tq, tk_res, p);
  }
  return check_launch("scoring kernels");
}

}  // namespace less
