// The parallel form on the tensor cores (Section 3.2, Inexpensive Training; Section 4.1): all rows
// of a sequence's causal attention matrix at once, entries the sparse policy has discarded
// replaced by phi(q_i) psi(k_j)^T, one normalisation per row (Eq. 3):
//
//     A_ij = exp(q_i . k_j / sqrt(D))     if i < exact_until[j]          (key j still cached)
//            phi(q_i) psi(k_j)^T          otherwise                      (j <= i)
//     out_i = sum_j A_ij v_j / sum_j A_ij
//
// Key tiles whose keys have all been discarded before a Q tile's first row never stream past it: their
// share of a row is phi(q_i) times the summed state of those tiles (see masked_tile_state_kernel).
// Steps (launch_masked_form): psi(K) and phi(Q) come from the MLP kernel (psi_tc.cu);
// masked_pack_kernel scales them by powers of two (phi per row, psi per instance), splits them into
// fp16 hi + lo and writes them as operand tiles; masked_out_tc_kernel then works like the
// prompt-output kernel, with a second accumulator:
//   S = Q K^T                       tcgen05, fp32 in tensor memory (double-buffered)
//   L = phi~ psi~^T                 tcgen05, hi hi + lo hi + hi lo of the scaled fp16 splits
//   P_ij = i < exact_until[j] ? exp2(c S_ij - E_i) : L_ij 2^(lscale_i - E_i)     (epilogue warps, lane = row)
//   O += P V                        tcgen05, P read from tensor memory;   r_i += sum_j P_ij (fp32, before rounding P to fp16)
//   out_i = O_i / r_i
// The key tiles stream past the Q tile twice.  The first sweep only takes maxima: the row's largest
// exact dot product and its largest kernel value give E_i = log2 of the row's largest entry.  The
// second sweep forms P against it, so every entry is at most 1 and the largest is 1 when P is
// rounded to fp16 for P V, whatever share of the plain softmax's mass the policy has left exact
// (a row whose dominant key has been discarded keeps ~1e-6 of it: formed against the plain
// normaliser its entries would sink into fp16's subnormals).
// With grouped query heads (Section 3.2, multi-query attention) the query heads of a group share the
// key side (K, V, psi, exact_until, the dead-tile sums); each has its own Q rows, phi and output.
// Every wait is bounded (pipeline.cuh).
#include "prefill.cuh"
#include "tc_common.cuh"

namespace less {

constexpr int MF_TILE = 128;
constexpr int MF_TILE_BYTES = MF_TILE * kHeadDim * 2;
constexpr int MF_OP_BYTES = 8192;                   // operand tile: [4 chunks of 8 k][16 row groups][8 rows][16 B]
constexpr int MF_EU_BYTES = MF_TILE * 4;
constexpr int MF_STAGES = 2;
constexpr int MF_EU_SLOTS = 4;                      // exact_until tiles in flight: the epilogue frees them, later than the K stage
constexpr int MF_STAGE_BYTES = 2 * MF_TILE_BYTES;   // K tile, then V tile
constexpr int MF_EPI_WARPS = 16;                   // four per lane quadrant, 32 keys of a tile each
constexpr int MF_EPI_THREADS = MF_EPI_WARPS * 32;
constexpr int MF_THREADS = 64 + MF_EPI_THREADS + 64;   // warp 0 TMA (Q, K, operands), warp 1 MMA (scores), warps 2..17 epilogue, warp 18 TMA (V), warp 19 MMA (P V)
constexpr float kMfExpScale = 0.12751743074602468f; // log2(e) / sqrt(128)

struct MfParams {
  const int32_t* exact_until;   // [B, layer_count, Hd, S]
  float* out;                   // [B, layer_count, Hd * grp, S, D]
  int St;                       // operand tiles per instance in the workspace
  const float* phi;             // [Iw * grp][Sp][R] phi(q_i), unscaled
  const float* hsum;            // [Iw][St][R*D + R] per Q tile: H, z summed over the key tiles that are dead for it
  const int32_t* bucket;        // [Iw][St] first Q tile for which a key tile is dead (all its keys discarded before it)
};

// ------------------------------------------------------------------------------------------- //
// Operand tiles and row constants.  One CTA = one 128-row tile of one query head, one thread per row;
// the group's first query head also writes the key side (psi operand, exact_until).
// ------------------------------------------------------------------------------------------- //
__device__ __forceinline__ float pow2_scale_exponent(float vmax) {
  // exponent e with vmax * 2^e in [8192, 16384): hi parts far from fp16's overflow, lo parts far from its underflow
  if (!(vmax > 0.f) || !(vmax < INFINITY)) return 0.f;
  return fminf(fmaxf(floorf(log2f(8192.f / vmax)), -100.f), 100.f);
}

template <int R>
__device__ __forceinline__ void split_row(const float* x, float scale, uint4* hi, uint4* lo) {
  // x[R] * scale -> fp16 hi and lo parts, 8 values per 16-byte chunk
  uint32_t h[R / 2], l[R / 2];
#pragma unroll
  for (int e = 0; e < R / 2; ++e) {
    const float a = x[2 * e] * scale, b = x[2 * e + 1] * scale;
    const __half2 hh = __floats2half2_rn(a, b);
    const float2 hf = __half22float2(hh);
    const __half2 ll = __floats2half2_rn(a - hf.x, b - hf.y);
    h[e] = *reinterpret_cast<const uint32_t*>(&hh);
    l[e] = *reinterpret_cast<const uint32_t*>(&ll);
  }
#pragma unroll
  for (int c = 0; c < R / 8; ++c) {
    hi[c] = make_uint4(h[c * 4], h[c * 4 + 1], h[c * 4 + 2], h[c * 4 + 3]);
    lo[c] = make_uint4(l[c * 4], l[c * 4 + 1], l[c * 4 + 2], l[c * 4 + 3]);
  }
}

template <int R>
__global__ void __launch_bounds__(MF_TILE) masked_pack_kernel(PfParams p, MfParams mf) {
  const int T = blockIdx.x, gq = blockIdx.y, r = threadIdx.x;
  const int g = gq / p.grp;                              // the KV instance of this query head
  const bool first = gq == g * p.grp;
  const int i = T * MF_TILE + r;
  const bool valid = i < p.S;
  const InstMap im = map_instance(p, g);
  const float pmax = __int_as_float(p.a.ws_pmax[g]);
  const float epsi = pow2_scale_exponent(pmax);

  float ph[R], ps[R];
#pragma unroll
  for (int e = 0; e < R; ++e) ph[e] = ps[e] = 0.f;
  if (valid) {
    const float4* a = reinterpret_cast<const float4*>(p.a.ws_phi + ((size_t)gq * p.Sp + i) * R);
    const float4* b = reinterpret_cast<const float4*>(p.a.ws_psi + ((size_t)g * p.Sp + i) * R);
#pragma unroll
    for (int e = 0; e < R / 4; ++e) {
      const float4 x = a[e], y = b[e];
      ph[4 * e] = x.x; ph[4 * e + 1] = x.y; ph[4 * e + 2] = x.z; ph[4 * e + 3] = x.w;
      ps[4 * e] = y.x; ps[4 * e + 1] = y.y; ps[4 * e + 2] = y.z; ps[4 * e + 3] = y.w;
    }
  }
  float phmax = 0.f;
#pragma unroll
  for (int e = 0; e < R; ++e) {
    phmax = fmaxf(phmax, ph[e]);
  }
  const float ephi = pow2_scale_exponent(phmax);

  // operand tiles.  The k-steps the MMA issues pair the chunks as
  //   R = 8 :  phi (hi, lo) x psi (hi, hi),   phi (hi, 0) x psi (lo, 0)
  //   R = 16:  phi hi x psi hi,  phi lo x psi hi,  phi hi x psi lo          (each 16 wide = 2 chunks)
  uint4 fh[R / 8], fl[R / 8], sh_[R / 8], sl[R / 8];
  split_row<R>(ph, exp2f(ephi), fh, fl);
  split_row<R>(ps, exp2f(epsi), sh_, sl);
  const int off = (r >> 3) * 128 + (r & 7) * 16;
  uint4* fo = reinterpret_cast<uint4*>(p.a.ws_phiop + ((size_t)gq * mf.St + T) * MF_OP_BYTES + off);
  uint4* so = reinterpret_cast<uint4*>(p.a.ws_psiop + ((size_t)g * mf.St + T) * MF_OP_BYTES + off);
  const uint4 zero = make_uint4(0, 0, 0, 0);
  constexpr int CH = 2048 / 16;                        // chunk stride in uint4
  if (R == 8) {
    fo[0] = fh[0]; fo[CH] = fl[0]; fo[2 * CH] = fh[0]; fo[3 * CH] = zero;
    if (first) { so[0] = sh_[0]; so[CH] = sh_[0]; so[2 * CH] = sl[0]; so[3 * CH] = zero; }
  } else {
    fo[0] = fh[0]; fo[CH] = fh[R / 8 - 1]; fo[2 * CH] = fl[0]; fo[3 * CH] = fl[R / 8 - 1];
    if (first) { so[0] = sh_[0]; so[CH] = sh_[R / 8 - 1]; so[2 * CH] = sl[0]; so[3 * CH] = sl[R / 8 - 1]; }
  }

  // what turns a scaled kernel value back into phi(q_i) psi(k_j)^T, as a power of two; the key's mask
  p.a.ws_g[(size_t)gq * mf.St * MF_TILE + i] = -(ephi + epsi);
  if (first) p.a.ws_eu[(size_t)g * mf.St * MF_TILE + i] = valid ? mf.exact_until[im.in_row0 + i] : 0;
}

// ------------------------------------------------------------------------------------------- //
// Dead key tiles.  A key tile T is dead for a Q tile q once every one of its keys has been discarded
// before the Q tile's first row (max exact_until over the tile <= 128 q): then all its entries are kernel
// values for all 128 rows, and its share of row i is phi(q_i) H_T and phi(q_i) z_T with
// H_T = sum_j psi(k_j)^T v_j, z_T = sum_j psi(k_j) over the tile (Eq. 4, Eq. 5 for a block).  A tile that
// is dead for q stays dead for every later Q tile, so Hsum_q = sum of H_T over the tiles dead for q is a
// running sum over "buckets" (the first Q tile a key tile is dead for).  The attention kernel streams
// only the tiles that are not dead; for an H2O-like schedule that is a band below the diagonal plus the
// tiles that hold keys kept for good, instead of the whole triangle.
// ------------------------------------------------------------------------------------------- //
template <int R>
__global__ void __launch_bounds__(MF_TILE) masked_tile_state_kernel(PfParams p, MfParams mf, float* ht, int32_t* bucket) {
  const int T = blockIdx.x, g = blockIdx.y, d = threadIdx.x;
  const InstMap im = map_instance(p, g);
  const int j0 = T * MF_TILE, nj = min(MF_TILE, p.S - j0);
  __shared__ float ps[MF_TILE][R];
  __shared__ int s_death[MF_TILE / 32];
  int death = 0;
  if (d < nj) {
#pragma unroll
    for (int q = 0; q < R; ++q) ps[d][q] = p.a.ws_psi[((size_t)g * p.Sp + j0 + d) * R + q];
    death = mf.exact_until[im.in_row0 + j0 + d];
  }
  death = __reduce_max_sync(0xffffffffu, death);
  if ((d & 31) == 0) s_death[d >> 5] = death;
  __syncthreads();
  float h[R];
#pragma unroll
  for (int q = 0; q < R; ++q) h[q] = 0.f;
  const __half* vcol = p.V + (im.in_row0 + j0) * kHeadDim + d;
  for (int j = 0; j < nj; ++j) {
    const float v = __half2float(vcol[(size_t)j * kHeadDim]);
#pragma unroll
    for (int q = 0; q < R; ++q) h[q] = fmaf(ps[j][q], v, h[q]);
  }
  float* dst = ht + ((size_t)g * mf.St + T) * (R * kHeadDim + R);
#pragma unroll
  for (int q = 0; q < R; ++q) dst[q * kHeadDim + d] = h[q];
  if (d < R) {
    float z = 0.f;
    for (int j = 0; j < nj; ++j) z += ps[j][d];
    dst[R * kHeadDim + d] = z;
  }
  if (d == 0) {
    int dm = s_death[0];
#pragma unroll
    for (int w = 1; w < MF_TILE / 32; ++w) dm = max(dm, s_death[w]);
    // first Q tile whose first row is >= every exact_until of the tile; never before the tile below the diagonal
    const long long b = ((long long)dm + MF_TILE - 1) / MF_TILE;
    bucket[(size_t)g * mf.St + T] = (int)min(max(b, (long long)T + 1), (long long)0x7fffffff);
  }
}

// Hsum_q = sum of H_T, z_T over the key tiles with bucket <= q: one thread per element, key tiles in order
// (a fixed order of additions), then a running sum over q.
template <int R>
__global__ void __launch_bounds__(256) masked_prefix_kernel(int tiles, int St, const float* ht, const int32_t* bucket, float* hsum) {
  const int g = blockIdx.y, e = blockIdx.x * 256 + threadIdx.x;
  constexpr int E = R * kHeadDim + R;
  if (e >= E) return;
  const float* src = ht + (size_t)g * St * E + e;
  float* dst = hsum + (size_t)g * St * E + e;
  const int32_t* bk = bucket + (size_t)g * St;
  for (int q = 0; q < tiles; ++q) dst[(size_t)q * E] = 0.f;
  for (int T = 0; T < tiles; ++T) {
    const int b = bk[T];
    if (b < tiles) dst[(size_t)b * E] += src[(size_t)T * E];
  }
  float run = 0.f;
  for (int q = 0; q < tiles; ++q) {
    run += dst[(size_t)q * E];
    dst[(size_t)q * E] = run;
  }
}

// ------------------------------------------------------------------------------------------- //
// One CTA = one 128-row Q tile of one query head; the key tiles 0 .. diagonal that are not dead stream past it.
// ------------------------------------------------------------------------------------------- //
struct MfShared {
  uint64_t res_full;
  uint64_t k_full[MF_STAGES], k_empty[MF_STAGES];     // K tile + psi operand tile
  uint64_t v_full[MF_STAGES], v_empty[MF_STAGES];
  uint64_t eu_full[MF_EU_SLOTS], eu_empty[MF_EU_SLOTS];   // exact_until of the key tile
  uint64_t s_full[2], s_free[2];                      // S buffer (and L) written / read
  uint64_t l_free;                                    // the single L buffer has been read
  uint64_t p_full[2];                                 // per S / P buffer: one barrier for both would let two phases pass unseen
  uint64_t pv_done[2];                                // the P V that read the S buffer's P has completed
  uint64_t o_full;
  uint32_t tmem_base;
  int abort;
  float rsum[4][MF_TILE];
  float rmax[4][MF_TILE];
  int nlive;                                          // key tiles of this Q tile that are not dead
};

__device__ __forceinline__ float mf_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void mf_epi_sync() { asm volatile("bar.sync 1, %0;" ::"n"(MF_EPI_THREADS) : "memory"); }

template <int R>
__global__ void __launch_bounds__(MF_THREADS) masked_out_tc_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                                   const __grid_constant__ CUtensorMap tm_k,
                                                                   const __grid_constant__ CUtensorMap tm_v,
                                                                   PfParams p, MfParams mf) {
  extern __shared__ __align__(1024) unsigned char mf_smem[];
  if (smem_misaligned(mf_smem, p.a.status, 120)) return;
  unsigned char* qres = mf_smem;                                   // Q tile: [2 halves][128 rows][128 B]
  unsigned char* ring = qres + MF_TILE_BYTES;                      // [stages][K tile, V tile]
  unsigned char* phires = ring + MF_STAGES * MF_STAGE_BYTES;       // phi operand tile of the rows
  unsigned char* psiring = phires + MF_OP_BYTES;                   // [stages] psi operand tiles of the keys
  unsigned char* euring = psiring + MF_STAGES * MF_OP_BYTES;       // [slots] exact_until of the keys
  MfShared* sh = reinterpret_cast<MfShared*>(euring + MF_EU_SLOTS * MF_EU_BYTES);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles = (p.S + MF_TILE - 1) / MF_TILE;
  const int tile = tiles - 1 - (int)blockIdx.x;                    // long rows first
  const int gq = blockIdx.y, g = gq / p.grp;                      // query head, its KV instance
  const InstMap im = map_instance(p, g);
  const QueryMap qm = map_query(p, gq);
  const int i0 = tile * MF_TILE;
  const int ntile = tile + 1;                                      // key tiles 0 .. tile (the last holds the diagonal)
  int32_t* status = p.a.status;
  const size_t op0 = (size_t)g * mf.St * MF_OP_BYTES;              // the KV instance's operand tiles (psi)
  const size_t rc0 = (size_t)g * mf.St * MF_TILE;                  // ... and exact_until
  const size_t op0q = (size_t)gq * mf.St * MF_OP_BYTES;            // the query head's operand tiles (phi)
  const size_t rc0q = (size_t)gq * mf.St * MF_TILE;                // ... and row constants

  if (tid == 0) {
    mbar_init(&sh->res_full, 1);
    for (int s = 0; s < MF_STAGES; ++s) {
      mbar_init(&sh->k_full[s], 1);
      mbar_init(&sh->k_empty[s], 1);
      mbar_init(&sh->v_full[s], 1);
      mbar_init(&sh->v_empty[s], 1);
    }
    for (int s = 0; s < MF_EU_SLOTS; ++s) {
      mbar_init(&sh->eu_full[s], 1);
      mbar_init(&sh->eu_empty[s], MF_EPI_WARPS);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh->s_full[s], 1);
      mbar_init(&sh->s_free[s], MF_EPI_WARPS);
      mbar_init(&sh->pv_done[s], 1);
    }
    mbar_init(&sh->l_free, MF_EPI_WARPS);
    mbar_init(&sh->p_full[0], MF_EPI_WARPS);
    mbar_init(&sh->p_full[1], MF_EPI_WARPS);
    mbar_init(&sh->o_full, 1);
    sh->abort = *reinterpret_cast<volatile int32_t*>(status) != 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&sh->tmem_base, 512);
  // A key tile all of whose keys were discarded before this Q tile's first row is dead for it: its
  // entries are phi(q_i) psi(k_j)^T for every row, so its whole contribution is phi(q_i) (sum psi^T v) and
  // phi(q_i) (sum psi), which masked_prefix_kernel has added up per Q tile (Eq. 6 for a block of keys).
  // Only the other tiles stream past the Q tile; every role skips the dead ones by the same test.
  const int32_t* bucket = mf.bucket + (size_t)g * mf.St;
  if (warp == 0) {
    int c = 0;
    for (int t = lane; t <= tile; t += 32) c += __ldg(bucket + t) > tile;
    c = __reduce_add_sync(0xffffffffu, c);
    if (lane == 0) sh->nlive = c;
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh->tmem_base;
  const int nlive = sh->nlive;
  const uint32_t ocol = 2 * MF_TILE, lcol = 3 * MF_TILE;           // O and L behind the two S buffers
  volatile int* abortp = &sh->abort;

  if (warp == 0) {
    // ---------------- producer: Q and its phi operand, then K + psi operand + exact_until per key tile ----------------
    if (lane == 0) {
      const int row0 = (int)(qm.q_row0 + i0);
      mbar_expect_tx(&sh->res_full, MF_TILE_BYTES + MF_OP_BYTES);
      tma_load_2d(qres, &tm_q, 0, row0, &sh->res_full);
      tma_load_2d(qres + MF_TILE_BYTES / 2, &tm_q, 64, row0, &sh->res_full);
      bulk_g2s(phires, p.a.ws_phiop + op0q + (size_t)tile * MF_OP_BYTES, MF_OP_BYTES, &sh->res_full);
      uint32_t s = 0, ph = 0;
      int u = 0;                                         // live tiles issued so far, both sweeps
      for (int sweep = 0; sweep < 2 && !*abortp; ++sweep)
      for (int t = 0; t < ntile; ++t) {
        if (__ldg(bucket + t) <= tile) continue;         // dead for this Q tile
        wait_or_give_up(&sh->k_empty[s], ph ^ 1, abortp, status, 110);
        const int es = u % MF_EU_SLOTS;
        wait_or_give_up(&sh->eu_empty[es], ((u / MF_EU_SLOTS) & 1) ^ 1, abortp, status, 111);
        if (*abortp) break;
        const int krow = (int)(im.in_row0 + (size_t)t * MF_TILE);
        unsigned char* st = ring + s * MF_STAGE_BYTES;
        mbar_expect_tx(&sh->k_full[s], MF_TILE_BYTES + MF_OP_BYTES);
        tma_load_2d(st, &tm_k, 0, krow, &sh->k_full[s]);
        tma_load_2d(st + MF_TILE_BYTES / 2, &tm_k, 64, krow, &sh->k_full[s]);
        bulk_g2s(psiring + s * MF_OP_BYTES, p.a.ws_psiop + op0 + (size_t)t * MF_OP_BYTES, MF_OP_BYTES, &sh->k_full[s]);
        mbar_expect_tx(&sh->eu_full[es], MF_EU_BYTES);
        bulk_g2s(euring + es * MF_EU_BYTES, p.a.ws_eu + rc0 + (size_t)t * MF_TILE, MF_EU_BYTES, &sh->eu_full[es]);
        if (++s == MF_STAGES) { s = 0; ph ^= 1; }
        ++u;
      }
    }
  } else if (warp == 2 + MF_EPI_WARPS) {
    // ---------------- producer of the V tiles ----------------
    if (lane == 0) {
      uint32_t s = 0, ph = 0;
      for (int t = 0; t < ntile; ++t) {
        if (__ldg(bucket + t) <= tile) continue;
        wait_or_give_up(&sh->v_empty[s], ph ^ 1, abortp, status, 112);
        if (*abortp) break;
        const int krow = (int)(im.in_row0 + (size_t)t * MF_TILE);
        unsigned char* st = ring + s * MF_STAGE_BYTES + MF_TILE_BYTES;
        mbar_expect_tx(&sh->v_full[s], MF_TILE_BYTES);
        tma_load_2d(st, &tm_v, 0, krow, &sh->v_full[s]);
        tma_load_2d(st + MF_TILE_BYTES / 2, &tm_v, 64, krow, &sh->v_full[s]);
        if (++s == MF_STAGES) { s = 0; ph ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer of the scores and kernel values (both sweeps) ----------------
    // Two threads issue the MMAs, one per product: a single thread gets an M = 128, N = 128, K = 16 MMA
    // out every ~84 cycles, two threads together one every ~65 (the tensor pipe's own rate).
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_f16(MF_TILE, MF_TILE, 0, 0);   // A = Q (K-major), B = K (K-major); also phi x psi
      const uint64_t ad_q = smem_desc(smem_u32(qres), 16, 1024, kLayoutSw128);
      // operand tiles without swizzle: chunks of 8 k are 2048 bytes apart, 8-row groups 128 bytes
      const uint64_t ad_phi = smem_desc(smem_u32(phires), 2048, 128, kLayoutNone);
      const uint64_t bd_psi = smem_desc(smem_u32(psiring), 2048, 128, kLayoutNone);
      const uint64_t bd_ring = smem_desc(smem_u32(ring), 16, 1024, kLayoutSw128);
      constexpr uint64_t kPair = 4096 >> 4;                             // two chunks = one 16-wide k-step further
      wait_or_give_up(&sh->res_full, 0, abortp, status, 113);
      uint32_t s1 = 0, ph1 = 0;
      for (int u = 0; u < 2 * nlive; ++u) {            // u counts live tiles; which tile it is does not matter here
        const int b1 = u & 1;
        wait_or_give_up(&sh->k_full[s1], ph1, abortp, status, 114);
        // buffer b1 held tile u - 2: read by the epilogue (s_free) and, in the second sweep, rewritten
        // with P and read by that tile's P V (pv_done); the single L buffer held tile u - 1 (l_free)
        if (u >= 2) wait_or_give_up(&sh->s_free[b1], ((u >> 1) - 1) & 1, abortp, status, 115);
        if (u - 2 >= nlive) wait_or_give_up(&sh->pv_done[b1], ((u - 2 - nlive) >> 1) & 1, abortp, status, 123);
        if (*abortp) break;
        tc_fence_after_sync();
        const uint64_t bd0 = bd_ring + (uint64_t)(s1 * (MF_STAGE_BYTES >> 4));
#pragma unroll
        for (int ks = 0; ks < kHeadDim / 16; ++ks)
          mma_f16_ss(tmem + b1 * MF_TILE, ad_q + (uint64_t)((ks >> 2) * (MF_TILE_BYTES >> 5) + (ks & 3) * 2),
                     bd0 + (uint64_t)((ks >> 2) * (MF_TILE_BYTES >> 5) + (ks & 3) * 2), idesc_s, ks ? 1u : 0u);
        // the scores are under way before the single L buffer is waited for: the epilogue of tile u - 1
        // reads it while these eight MMAs run
        if (u >= 1) wait_or_give_up(&sh->l_free, (u - 1) & 1, abortp, status, 116);
        if (*abortp) break;
        tc_fence_after_sync();
        const uint64_t bp = bd_psi + (uint64_t)(s1 * (MF_OP_BYTES >> 4));
        if (R == 8) {
          mma_f16_ss(tmem + lcol, ad_phi, bp, idesc_s, 0u);                   // (hi, lo) x (hi, hi)
          mma_f16_ss(tmem + lcol, ad_phi + kPair, bp + kPair, idesc_s, 1u);   // (hi, 0) x (lo, 0)
        } else {
          mma_f16_ss(tmem + lcol, ad_phi, bp, idesc_s, 0u);                   // hi x hi
          mma_f16_ss(tmem + lcol, ad_phi + kPair, bp, idesc_s, 1u);           // lo x hi
          mma_f16_ss(tmem + lcol, ad_phi, bp + kPair, idesc_s, 1u);           // hi x lo
        }
        mma_commit(&sh->k_empty[s1]);
        mma_commit(&sh->s_full[b1]);
        if (++s1 == MF_STAGES) { s1 = 0; ph1 ^= 1; }
      }
    }
  } else if (warp == 3 + MF_EPI_WARPS) {
    // ---------------- MMA issuer of P V (second sweep) ----------------
    if (lane == 0) {
      constexpr uint32_t idesc_o = idesc_f16(MF_TILE, kHeadDim, 0, 1);  // A = P (tensor memory), B = V (N-major)
      const uint64_t bd_vring = smem_desc(smem_u32(ring) + MF_TILE_BYTES, MF_TILE_BYTES / 2, 1024, kLayoutSw128);
      uint32_t s2 = 0, vph = 0;
      for (int t = 0; t < nlive; ++t) {                // t counts the live tiles of the second sweep
        const int bt = (nlive + t) & 1;                  // the S buffer this tile's P lives in
        wait_or_give_up(&sh->v_full[s2], vph, abortp, status, 117);
        wait_or_give_up(&sh->p_full[bt], (t >> 1) & 1, abortp, status, 118);   // the buffer's (t / 2)-th P
        if (*abortp) break;
        tc_fence_after_sync();
        const uint64_t bv0 = bd_vring + (uint64_t)(s2 * (MF_STAGE_BYTES >> 4));
#pragma unroll
        for (int ks = 0; ks < MF_TILE / 16; ++ks)
          // A = P from tensor memory: k-step ks is 8 packed columns inside the S columns of part ks / 2
          mma_f16_ts(tmem + ocol, tmem + bt * MF_TILE + 32 * (ks >> 1) + 8 * (ks & 1),
                     bv0 + (uint64_t)(ks * (2048 >> 4)), idesc_o, (t | ks) ? 1u : 0u);
        mma_commit(&sh->v_empty[s2]);
        mma_commit(&sh->pv_done[bt]);
        if (++s2 == MF_STAGES) { s2 = 0; vph ^= 1; }
      }
      mma_commit(&sh->o_full);
    }
  } else {
    // ---------------- epilogue warps: lane = query row, the four warps of a quadrant split the keys ----------------
    const int quad = warp & 3, part = (warp - 2) >> 2;               // part: 32 of the tile's 128 keys
    const int r = quad * 32 + lane, i = i0 + r;
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    // sweep 1: the row's largest exact dot product and largest kernel value (scaled operands);
    // sweep 2: P against the largest entry, so that every entry is <= 1 and the largest is 1
    const float lscale = p.a.ws_g[rc0q + i];            // log2 of (true kernel value / scaled kernel value)
    const bool live = i < p.S;
    float mx = -INFINITY, ml = 0.f;
    float nb = 0.f, gi = 0.f, rsum = 0.f, rsum2 = 0.f;
    uint32_t b = 0, bph = 0;
    int u = 0;                                           // live tiles done so far, both sweeps
    for (int sweep = 0; sweep < 2; ++sweep)
    for (int t = 0; t < ntile; ++t) {
      const bool second = sweep == 1;
      if (second && t == 0) {
        // between the sweeps: E = log2 of the row's largest entry; exact entries become
        // exp2(c S - E), kernel entries L 2^(lscale - E)
        sh->rsum[part][r] = mx;
        sh->rmax[part][r] = ml;
        mf_epi_sync();
        mx = fmaxf(fmaxf(sh->rsum[0][r], sh->rsum[1][r]), fmaxf(sh->rsum[2][r], sh->rsum[3][r]));
        ml = fmaxf(fmaxf(sh->rmax[0][r], sh->rmax[1][r]), fmaxf(sh->rmax[2][r], sh->rmax[3][r]));
        mf_epi_sync();                                   // rsum is used again at the end
        const float ea = mx * kMfExpScale;               // -inf without exact entries
        const float el = ml > 0.f ? log2f(ml) + lscale : -INFINITY;
        const float E = fmaxf(ea, el);
        if (live && E < INFINITY) {
          // a row with nothing in its live tiles (E = -inf) keeps scale 1 for the dead tiles' part
          const float Es = E > -INFINITY ? E : 0.f;
          nb = -Es;
          gi = exp2f(fminf(lscale - Es, 120.f));
        } else {                                         // a row past the sequence, or one with nothing in it: all zeros
          nb = -INFINITY;
          gi = 0.f;
        }
      }
      if (__ldg(bucket + t) <= tile) continue;           // dead for this Q tile
      wait_or_give_up(&sh->s_full[b], bph, abortp, status, 119);
      const int es = u % MF_EU_SLOTS;
      wait_or_give_up(&sh->eu_full[es], (u / MF_EU_SLOTS) & 1, abortp, status, 120);
      tc_fence_after_sync();
      const int j0 = t * MF_TILE + part * 32;
      const int4* eu4 = reinterpret_cast<const int4*>(euring + es * MF_EU_BYTES) + part * 8;
      const bool diag = t == ntile - 1;
      uint32_t pk[16];
      uint32_t v[32], w[32];
      tmem_ld32(lane_addr + b * MF_TILE + part * 32, v);
      tmem_ld32(lane_addr + lcol + part * 32, w);
      tmem_ld_wait();
      tc_fence_before_sync();                            // both accumulators of this tile are in registers
      mbar_arrive_warp(&sh->s_free[b]);
      mbar_arrive_warp(&sh->l_free);
      if (!second) {
        // four independent chains per maximum
        float a0 = -INFINITY, a1 = -INFINITY, a2 = -INFINITY, a3 = -INFINITY, l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
        if (diag) {
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const int4 eu = eu4[e];
            const int j = j0 + 4 * e;
            const bool x0 = i < eu.x, x1 = i < eu.y, x2 = i < eu.z, x3 = i < eu.w;
            const bool c0 = j <= i, c1 = j + 1 <= i, c2 = j + 2 <= i, c3 = j + 3 <= i;     // causal
            a0 = fmaxf(a0, (c0 && x0) ? __uint_as_float(v[4 * e]) : -INFINITY);
            a1 = fmaxf(a1, (c1 && x1) ? __uint_as_float(v[4 * e + 1]) : -INFINITY);
            a2 = fmaxf(a2, (c2 && x2) ? __uint_as_float(v[4 * e + 2]) : -INFINITY);
            a3 = fmaxf(a3, (c3 && x3) ? __uint_as_float(v[4 * e + 3]) : -INFINITY);
            l0 = fmaxf(l0, (c0 && !x0) ? __uint_as_float(w[4 * e]) : 0.f);
            l1 = fmaxf(l1, (c1 && !x1) ? __uint_as_float(w[4 * e + 1]) : 0.f);
            l2 = fmaxf(l2, (c2 && !x2) ? __uint_as_float(w[4 * e + 2]) : 0.f);
            l3 = fmaxf(l3, (c3 && !x3) ? __uint_as_float(w[4 * e + 3]) : 0.f);
          }
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const int4 eu = eu4[e];
            const bool x0 = i < eu.x, x1 = i < eu.y, x2 = i < eu.z, x3 = i < eu.w;
            a0 = fmaxf(a0, x0 ? __uint_as_float(v[4 * e]) : -INFINITY);
            a1 = fmaxf(a1, x1 ? __uint_as_float(v[4 * e + 1]) : -INFINITY);
            a2 = fmaxf(a2, x2 ? __uint_as_float(v[4 * e + 2]) : -INFINITY);
            a3 = fmaxf(a3, x3 ? __uint_as_float(v[4 * e + 3]) : -INFINITY);
            l0 = fmaxf(l0, x0 ? 0.f : __uint_as_float(w[4 * e]));
            l1 = fmaxf(l1, x1 ? 0.f : __uint_as_float(w[4 * e + 1]));
            l2 = fmaxf(l2, x2 ? 0.f : __uint_as_float(w[4 * e + 2]));
            l3 = fmaxf(l3, x3 ? 0.f : __uint_as_float(w[4 * e + 3]));
          }
        }
        mx = fmaxf(mx, fmaxf(fmaxf(a0, a1), fmaxf(a2, a3)));
        ml = fmaxf(ml, fmaxf(fmaxf(l0, l1), fmaxf(l2, l3)));
      } else {
        const int2* eu2 = reinterpret_cast<const int2*>(eu4);
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const int2 eu = eu2[e];
          const int j = j0 + 2 * e;
          float p0 = i < eu.x ? mf_ex2(fmaf(__uint_as_float(v[2 * e]), kMfExpScale, nb)) : __uint_as_float(w[2 * e]) * gi;
          float p1 = i < eu.y ? mf_ex2(fmaf(__uint_as_float(v[2 * e + 1]), kMfExpScale, nb))
                              : __uint_as_float(w[2 * e + 1]) * gi;
          if (diag) {
            p0 = j <= i ? p0 : 0.f;
            p1 = j + 1 <= i ? p1 : 0.f;
          }
          if (e & 1) rsum2 += p0 + p1; else rsum += p0 + p1;
          const __half2 h = __floats2half2_rn(p0, p1);
          pk[e] = *reinterpret_cast<const uint32_t*>(&h);
        }
      }
      mbar_arrive_warp(&sh->eu_empty[es]);
      if (second) {
        // P, rounded to fp16, over the first 16 of this warp's own 32 S columns (they are in registers):
        // it inherits the double buffering of S, and the scores that overwrite the buffer are issued
        // after the P V that reads it (the tensor pipe runs in issue order)
        tmem_st16(lane_addr + b * MF_TILE + part * 32, pk);
        tmem_st_wait();
        tc_fence_before_sync();
        mbar_arrive_warp(&sh->p_full[b]);
      }
      if (b ^= 1, b == 0) bph ^= 1;
      ++u;
    }
    // ---- the row's normaliser: the four parts' sums ----
    sh->rsum[part][r] = rsum + rsum2;
    mf_epi_sync();
    float total = (sh->rsum[0][r] + sh->rsum[1][r]) + (sh->rsum[2][r] + sh->rsum[3][r]);
    // the dead key tiles: phi(q_i) Hsum and phi(q_i) zsum, in the scale of P (2^-E_i = 2^nb)
    const float* hs = mf.hsum + ((size_t)g * mf.St + tile) * (R * kHeadDim + R);
    float ph[R], dead[32];
    const float f = live ? exp2f(fminf(nb, 120.f)) : 0.f;           // nb = -inf for an empty row: 0
#pragma unroll
    for (int e = 0; e < 32; ++e) dead[e] = 0.f;
    if (live) {
      float dz = 0.f;
#pragma unroll
      for (int q = 0; q < R; ++q) {
        ph[q] = mf.phi[((size_t)gq * p.Sp + i) * R + q] * f;
        dz = fmaf(ph[q], __ldg(hs + R * kHeadDim + q), dz);
      }
      total += dz;
#pragma unroll
      for (int q = 0; q < R; ++q) {
        const float4* hrow = reinterpret_cast<const float4*>(hs + q * kHeadDim + part * 32);
#pragma unroll
        for (int e4 = 0; e4 < 8; ++e4) {
          const float4 h = __ldg(hrow + e4);
          dead[e4 * 4] = fmaf(ph[q], h.x, dead[e4 * 4]);
          dead[e4 * 4 + 1] = fmaf(ph[q], h.y, dead[e4 * 4 + 1]);
          dead[e4 * 4 + 2] = fmaf(ph[q], h.z, dead[e4 * 4 + 2]);
          dead[e4 * 4 + 3] = fmaf(ph[q], h.w, dead[e4 * 4 + 3]);
        }
      }
    }
    const float inv = total > 0.f ? 1.0f / total : 0.f;
    // ---- the finished rows: O[row][32 columns of this warp] / r_i ----
    wait_or_give_up(&sh->o_full, 0, abortp, status, 122);
    tc_fence_after_sync();
    float* orow = mf.out + (qm.q_row0 + i) * kHeadDim + part * 32;
    {
      uint32_t o[32];
      tmem_ld32(lane_addr + ocol + part * 32, o);
      tmem_ld_wait();
      if (i < p.S && !*abortp) {
#pragma unroll
        for (int e = 0; e < 32; e += 4)
          *reinterpret_cast<float4*>(orow + e) =
              make_float4((__uint_as_float(o[e]) + dead[e]) * inv, (__uint_as_float(o[e + 1]) + dead[e + 1]) * inv,
                          (__uint_as_float(o[e + 2]) + dead[e + 2]) * inv, (__uint_as_float(o[e + 3]) + dead[e + 3]) * inv);
      }
    }
  }
  drain_after_abort(abortp);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

int launch_masked_form(less_ctx* c, int layer0, int nl, int lj0, int layer_count, int S, const void* Q,
                       const void* K, const void* V, const int32_t* exact_until, void* out, cudaStream_t s) {
  const Dims& d = c->d;
  if (!score_tc_supported() || !psi_tc_supported(d) || c->score_path != 1) return LESS_ERR_INVALID_CONFIG;
  PfParams p;
  p.Q = (const __half*)Q; p.K = (const __half*)K; p.V = (const __half*)V;
  p.attn_out = nullptr;
  p.a = c->a;
  p.w_psi1 = (const __half*)c->w.w_psi1;
  p.w_psi2 = (const __half*)c->w.w_psi2;
  p.w_psi3 = (const __half*)c->w.w_psi3;
  p.psi_scale = c->w.psi_scale;
  p.S = S; p.Sp = d.Sp; p.Sbx = d.Sbx;
  p.layer0 = layer0; p.nl = nl; p.lj0 = lj0; p.layer_count = layer_count;
  p.B = d.B; p.L = d.L; p.Hd = d.Hd; p.N = d.N; p.Np = d.Np;
  p.heavy = d.heavy; p.recent = d.recent; p.Rp = d.Rp;
  p.flags = d.flags;
  p.grp = d.G;
  const int G = d.B * nl * d.Hd, Gq = G * d.G;       // KV instances, query heads
  // token splits of the MLP kernel, as in the prompt phase
  int split_tokens = 1024;
  while (split_tokens > 128 && (long long)G * ((S + split_tokens - 1) / split_tokens) < 148) split_tokens >>= 1;
  if ((S + split_tokens - 1) / split_tokens > kMaxSplit)
    split_tokens = ((S + kMaxSplit - 1) / kMaxSplit + 127) / 128 * 128;
  p.nsplit = (S + split_tokens - 1) / split_tokens;
  p.split_tokens = split_tokens;
  MfParams mf;
  mf.exact_until = exact_until;
  mf.out = (float*)out;
  mf.St = d.St;

  int rc;
  if (cudaMemsetAsync(c->a.ws_pmax, 0, (size_t)G * 4, s) != cudaSuccess) return fail_cuda("clearing the psi maxima");
  rc = launch_psi_tc(c, p, G, s);
  if (rc != LESS_OK) return rc;
  rc = launch_phi_tc(c, p, Gq, s, c->a.ws_phi);
  if (rc != LESS_OK) return rc;
  const int tiles = (S + MF_TILE - 1) / MF_TILE;
  {
    LaunchScope scope(c, LESS_KERNEL_MASKED_PACK, s);
    if (d.R == 8) masked_pack_kernel<8><<<dim3(tiles, Gq), MF_TILE, 0, s>>>(p, mf);
    else masked_pack_kernel<16><<<dim3(tiles, Gq), MF_TILE, 0, s>>>(p, mf);
  }
  mf.phi = c->a.ws_phi;
  mf.hsum = c->a.ws_hsum;
  mf.bucket = c->a.ws_bucket;
  {
    LaunchScope scope(c, LESS_KERNEL_MASKED_PACK, s);
    if (d.R == 8) masked_tile_state_kernel<8><<<dim3(tiles, G), MF_TILE, 0, s>>>(p, mf, c->a.ws_ht, c->a.ws_bucket);
    else masked_tile_state_kernel<16><<<dim3(tiles, G), MF_TILE, 0, s>>>(p, mf, c->a.ws_ht, c->a.ws_bucket);
  }
  {
    LaunchScope scope(c, LESS_KERNEL_MASKED_PACK, s);
    const int E = d.R * kHeadDim + d.R;
    if (d.R == 8) masked_prefix_kernel<8><<<dim3((E + 255) / 256, G), 256, 0, s>>>(tiles, d.St, c->a.ws_ht, c->a.ws_bucket, c->a.ws_hsum);
    else masked_prefix_kernel<16><<<dim3((E + 255) / 256, G), 256, 0, s>>>(tiles, d.St, c->a.ws_ht, c->a.ws_bucket, c->a.ws_hsum);
  }
  CUtensorMap tq, tk, tv;
  const uint64_t rows = (uint64_t)d.B * layer_count * d.Hd * S;
  if (!make_tmap_f16_2d(&tq, p.Q, rows * d.G, kHeadDim, kHeadDim * 2, MF_TILE) ||
      !make_tmap_f16_2d(&tk, p.K, rows, kHeadDim, kHeadDim * 2, MF_TILE) ||
      !make_tmap_f16_2d(&tv, p.V, rows, kHeadDim, kHeadDim * 2, MF_TILE))
    return fail_cuda("tensor maps of Q / K / V");
  const size_t smem = (size_t)MF_TILE_BYTES + MF_STAGES * MF_STAGE_BYTES + MF_OP_BYTES + MF_STAGES * MF_OP_BYTES +
                      MF_EU_SLOTS * MF_EU_BYTES + sizeof(MfShared) + 1024;
  LaunchScope scope(c, LESS_KERNEL_MASKED_OUT, s, "masked_out_tc_kernel");
  if (d.R == 8) {
    if (cudaFuncSetAttribute(masked_out_tc_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return fail_cuda("shared memory opt-in of masked_out_tc_kernel");
    masked_out_tc_kernel<8><<<dim3(tiles, Gq), MF_THREADS, smem, s>>>(tq, tk, tv, p, mf);
  } else {
    if (cudaFuncSetAttribute(masked_out_tc_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return fail_cuda("shared memory opt-in of masked_out_tc_kernel");
    masked_out_tc_kernel<16><<<dim3(tiles, Gq), MF_THREADS, smem, s>>>(tq, tk, tv, p, mf);
  }
  return check_launch("the parallel-form kernels");
}

}  // namespace less
