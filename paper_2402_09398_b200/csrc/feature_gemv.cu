// Feature maps phi(q_t), psi(k_t) (Eq. 1, Eq. 2) for small batches: a GEMV per
// (layer, head, map), bound by streaming the per-head weights from HBM once.
//
// Persistent kernel: each CTA walks a strided list of work items; one producer
// warp streams the item's weights (W1 in 16-KB row chunks, then W2) into a
// shared-memory ring with bulk asynchronous copies, eight consumer warps do
// the arithmetic.  The hidden activations never leave shared memory (the
// paper folds the activation into the preceding linear kernel, Section 3.2, taken to the whole MLP).
#include "feature_gemv.cuh"
#include "pipeline.cuh"

namespace less {

constexpr int GV_CONSUMERS = 256;
constexpr int GV_THREADS = GV_CONSUMERS + 32;
constexpr int GV_STAGE_BYTES = 16384;

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(GV_CONSUMERS) : "memory"); }

struct GvShared {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t aux_full[2];
  uint64_t aux_empty[2];
  int abort;
};

// waits unless the CTA has already given up; a wait that runs out makes the CTA give up
// (it keeps going through its barriers with meaningless data, so nothing can hang)
__device__ __forceinline__ void wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort,
                                              int32_t* status, int where) {
  if (*abort) return;
  if (!mbar_wait(bar, parity)) {
    *abort = 1;
    set_status(status, kStatusTimeout, where);
  }
}

// per item, double-buffered: the input rows (fp16) and W3
template <int R, int BR>
struct GvAux {
  __half x[BR][kHeadDim];
  __half w3[R * R];
};

template <int R, int BR, int NS>
__global__ void __launch_bounds__(GV_THREADS) feature_gemv_kernel(FmParams p, int nchunk_b, int items,
                                                                  int32_t* status) {
  extern __shared__ __align__(128) unsigned char gv_smem[];
  const int Rp = p.Rp;
  unsigned char* ring = gv_smem;                                        // NS x 16 KB
  GvAux<R, BR>* aux = reinterpret_cast<GvAux<R, BR>*>(ring + NS * GV_STAGE_BYTES);   // [2]
  float* hs = reinterpret_cast<float*>(aux + 2);                        // [BR][Rp]
  float* part = hs + BR * Rp;                                           // [ndg][BR][Rp]
  float* l2p = part + (GV_CONSUMERS / (Rp >> 3)) * BR * Rp;             // [8][BR][R]
  GvShared* sh = reinterpret_cast<GvShared*>(l2p + 8 * BR * R);

  const int tid = threadIdx.x;
  const int n_w1 = Rp >> 6;                       // W1 chunks per item (16 KB each)
  const uint32_t w2_bytes = (uint32_t)Rp * R * 2;
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], GV_CONSUMERS / 32);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh->aux_full[s], 1);
      mbar_init(&sh->aux_empty[s], GV_CONSUMERS / 32);
    }
    // a CTA that starts after another one has given up skips every wait: the grid drains at once
    sh->abort = *reinterpret_cast<volatile int32_t*>(status) != 0;
    mbar_fence_init();
  }
  __syncthreads();
  pdl_launch_dependents();
  volatile int* abortp = &sh->abort;

  if (tid >= GV_CONSUMERS) {
    // ---------------- producer warp: one lane issues the copies ----------------
    if (tid == GV_CONSUMERS) {
      uint32_t g = 0, n = 0;
      for (int it = blockIdx.x; it < items; it += gridDim.x, ++n) {
        const int lh = it / (2 * nchunk_b), which = (it / nchunk_b) & 1, bc = it % nchunk_b;
        const int layer = lh / p.Hd, head = lh % p.Hd;
        const int b0 = bc * BR, nb = min(BR, p.B - b0);
        const int a = n & 1;
        wait_or_abort(&sh->aux_empty[a], ((n >> 1) & 1) ^ 1, abortp, status, 13);
        mbar_expect_tx(&sh->aux_full[a], (uint32_t)(nb * kHeadDim * 2 + R * R * 2));
        for (int b = 0; b < nb; ++b)
          bulk_g2s(&aux[a].x[b][0],
                   p.x[which] + (((size_t)(b0 + b) * p.L + layer) * p.Hd + head) * kHeadDim,
                   kHeadDim * 2, &sh->aux_full[a]);
        bulk_g2s(&aux[a].w3[0], p.w3 + (size_t)lh * R * R, R * R * 2, &sh->aux_full[a]);
        const unsigned char* w1 = reinterpret_cast<const unsigned char*>(p.w1[which]) +
                                  (size_t)lh * kHeadDim * Rp * 2;
        const unsigned char* w2 = reinterpret_cast<const unsigned char*>(p.w2[which]) +
                                  (size_t)lh * Rp * R * 2;
        for (int c = 0; c <= n_w1; ++c, ++g) {
          const int s = g % NS;
          wait_or_abort(&sh->empty[s], ((g / NS) & 1) ^ 1, abortp, status, 10);
          const uint32_t bytes = c < n_w1 ? GV_STAGE_BYTES : w2_bytes;
          mbar_expect_tx(&sh->full[s], bytes);
          bulk_g2s(ring + s * GV_STAGE_BYTES, c < n_w1 ? w1 + (size_t)c * GV_STAGE_BYTES : w2, bytes,
                   &sh->full[s]);
        }
      }
    }
    return;
  }

  // ---------------- consumers ----------------
  const int warp = tid >> 5, lane = tid & 31;
  const int ncg = Rp >> 3, ndg = GV_CONSUMERS / ncg;
  const int cg = tid % ncg, dg = tid / ncg;
  const int rows_per_chunk = GV_STAGE_BYTES / (Rp * 2);
  uint32_t g = 0, n = 0;
  for (int it = blockIdx.x; it < items; it += gridDim.x, ++n) {
    const int lh = it / (2 * nchunk_b), which = (it / nchunk_b) & 1, bc = it % nchunk_b;
    const int layer = lh / p.Hd, head = lh % p.Hd;
    const int b0 = bc * BR, nb = min(BR, p.B - b0);
    const int a = n & 1;
    float c1 = 1.f, c2 = 1.f;
    if (which == 1 && p.psi_scale) { c1 = __ldg(p.psi_scale + lh * 2); c2 = __ldg(p.psi_scale + lh * 2 + 1); }
    wait_or_abort(&sh->aux_full[a], (n >> 1) & 1, abortp, status, 14);
    const __half* xr = &aux[a].x[0][0];
    // layer 1: every thread owns 8 hidden units and every ndg-th row of each chunk
    float acc[BR][8];
#pragma unroll
    for (int b = 0; b < BR; ++b)
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[b][c] = 0.f;
    for (int c = 0; c < n_w1; ++c, ++g) {
      const int s = g % NS;
      wait_or_abort(&sh->full[s], (g / NS) & 1, abortp, status, 11);
      const __half* stage = reinterpret_cast<const __half*>(ring + s * GV_STAGE_BYTES);
#pragma unroll
      for (int rr = 0; rr < 4; ++rr) {
        const int row = dg + rr * ndg;                 // row inside the chunk
        float wf[8];
        half8_to_float(*reinterpret_cast<const uint4*>(stage + (size_t)row * Rp + cg * 8), wf);
        const int d = c * rows_per_chunk + row;
#pragma unroll
        for (int b = 0; b < BR; ++b) {
          const float xv = b < nb ? __half2float(xr[b * kHeadDim + d]) : 0.f;
#pragma unroll
          for (int k = 0; k < 8; ++k) acc[b][k] = fmaf(xv, wf[k], acc[b][k]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->empty[s]);
    }
#pragma unroll
    for (int b = 0; b < BR; ++b) {
      float4* dst = reinterpret_cast<float4*>(part + ((size_t)dg * BR + b) * Rp + cg * 8);
      dst[0] = make_float4(acc[b][0], acc[b][1], acc[b][2], acc[b][3]);
      dst[1] = make_float4(acc[b][4], acc[b][5], acc[b][6], acc[b][7]);
    }
    consumer_sync();
    for (int e = tid; e < BR * Rp; e += GV_CONSUMERS) {
      float s = 0.f;
      for (int gq = 0; gq < ndg; ++gq) s += part[(size_t)gq * BR * Rp + e];   // fixed order
      hs[e] = c1 * gelu_erf(s);
    }
    consumer_sync();
    // layer 2: warp w covers hidden units [w*Rp/8, (w+1)*Rp/8)
    {
      const int s = g % NS;
      wait_or_abort(&sh->full[s], (g / NS) & 1, abortp, status, 12);
      const __half* w2s = reinterpret_cast<const __half*>(ring + s * GV_STAGE_BYTES);
      float a2[BR][R];
#pragma unroll
      for (int b = 0; b < BR; ++b)
#pragma unroll
        for (int r = 0; r < R; ++r) a2[b][r] = 0.f;
      const int jper = Rp >> 3;
      for (int j = warp * jper + lane; j < (warp + 1) * jper; j += 32) {
        float wf[R];
#pragma unroll
        for (int r8 = 0; r8 < R / 8; ++r8)
          half8_to_float(*reinterpret_cast<const uint4*>(w2s + (size_t)j * R + r8 * 8), wf + r8 * 8);
#pragma unroll
        for (int b = 0; b < BR; ++b) {
          const float hv = hs[b * Rp + j];
#pragma unroll
          for (int r = 0; r < R; ++r) a2[b][r] = fmaf(hv, wf[r], a2[b][r]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->empty[s]);
      ++g;
#pragma unroll
      for (int b = 0; b < BR; ++b)
#pragma unroll
        for (int r = 0; r < R; ++r) {
          float v = a2[b][r];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          if (lane == 0) l2p[(warp * BR + b) * R + r] = v;
        }
    }
    consumer_sync();
    if (warp < nb) {
      const int b = warp;
      float gv = 0.f;
      if (lane < R) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += l2p[(w * BR + b) * R + lane];         // fixed order
        gv = c2 * gelu_erf(s);
      }
      float res;
      if (which == 0) {
        res = fabsf(gv);
      } else {
        const __half* w3 = &aux[a].w3[0];
        float s = 0.f;
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const float gr = __shfl_sync(0xffffffffu, gv, r);
          if (lane < R) s = fmaf(gr, __half2float(w3[r * R + lane]), s);
        }
        res = fabsf(s);
      }
      if (lane < R) {
        const size_t inst = ((size_t)(b0 + b) * p.L + layer) * p.Hd + head;
        p.out[which][inst * R + lane] = res;
      }
    }
    // this warp is done with the item's input rows and W3
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh->aux_empty[a]);
    // No barrier here: part is next written after this warp's next layer 1 and was last read
    // before the second barrier above; hs and l2p are next written after the next item's
    // first and second barrier, which a warp reaches only after finishing this item.
  }
}

template <int R, int BR, int NS>
static int launch_one(less_ctx* c, const FmParams& p, cudaStream_t s) {
  const Dims& d = c->d;
  const int nchunk_b = (d.B + BR - 1) / BR;
  const int items = d.L * d.Hd * 2 * nchunk_b;
  const int ndg = GV_CONSUMERS / (d.Rp / 8);
  const size_t smem = (size_t)NS * GV_STAGE_BYTES + 2 * sizeof(GvAux<R, BR>) +
                      (size_t)(BR * d.Rp + ndg * BR * d.Rp + 8 * BR * R) * 4 + sizeof(GvShared) + 16;
  auto kern = feature_gemv_kernel<R, BR, NS>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return fail_cuda("tensor map or shared memory opt-in");
  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
  int per_sm = 1;
  cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, GV_THREADS, smem);
  if (per_sm < 1) per_sm = 1;
  const int grid = items < sms * per_sm ? items : sms * per_sm;
  LaunchScope scope(c, LESS_KERNEL_FEATURE_MAP, s, "feature_gemv_kernel");
  kern<<<grid, GV_THREADS, smem, s>>>(p, nchunk_b, items, c->a.status);
  return check_launch("feature_gemv_kernel");
}

bool feature_gemv_supported(const Dims& d) { return d.Rp <= 512 && d.Rp >= 64; }

int launch_feature_gemv(less_ctx* c, const FmParams& p, cudaStream_t s) {
  const Dims& d = c->d;
  if (d.R == 8) {
    if (d.B == 1) return launch_one<8, 1, 6>(c, p, s);
    if (d.B == 2) return launch_one<8, 2, 5>(c, p, s);
    return launch_one<8, 4, 4>(c, p, s);
  }
  if (d.B == 1) return launch_one<16, 1, 6>(c, p, s);
  if (d.B == 2) return launch_one<16, 2, 5>(c, p, s);
  return launch_one<16, 4, 4>(c, p, s);
}

}  // namespace less
