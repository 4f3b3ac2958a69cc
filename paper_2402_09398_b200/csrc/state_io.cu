// Records of less_export_state / less_import_state (Algorithm 1's "save K, V, H, z") gathered on
// the device: one CTA per listed instance packs its fields into (or unpacks them from) one
// contiguous record in a staging buffer, so that the host sees one copy per batch of records
// instead of eight small ones per instance.
#include "less_internal.cuh"

namespace less {

struct StateIo {
  Arena a;
  const int32_t* inst;      // device: the listed instances
  uint32_t* records;        // device staging: n records of rec_words 32-bit words
  int N, Np, D, R;
  int rec_words;
  int to_records;           // 1 pack (export), 0 unpack (import)
};

__device__ __forceinline__ void move_words(uint32_t* rec, uint32_t* field, int nwords, int to_records) {
  for (int i = threadIdx.x; i < nwords; i += blockDim.x) {
    if (to_records) rec[i] = field[i];
    else field[i] = rec[i];
  }
}

__global__ void __launch_bounds__(256) state_io_kernel(StateIo p) {
  const size_t I = (size_t)p.inst[blockIdx.x];
  uint32_t* rec = p.records + (size_t)blockIdx.x * p.rec_words;
  const int N = p.N, D = p.D, R = p.R;
  // header: live slots, then three words the host fills (position, reserved)
  if (threadIdx.x == 0) {
    if (p.to_records) { rec[0] = (uint32_t)p.a.count[I]; rec[1] = rec[2] = rec[3] = 0u; }
    else p.a.count[I] = (int32_t)rec[0];
  }
  int off = 4;
  move_words(rec + off, reinterpret_cast<uint32_t*>(p.a.pos + I * p.Np), N, p.to_records);            off += N;
  move_words(rec + off, reinterpret_cast<uint32_t*>(p.a.acc + I * p.Np), N, p.to_records);            off += N;
  move_words(rec + off, reinterpret_cast<uint32_t*>(p.a.kslots + I * N * D), N * D / 2, p.to_records); off += N * D / 2;
  move_words(rec + off, reinterpret_cast<uint32_t*>(p.a.vslots + I * N * D), N * D / 2, p.to_records); off += N * D / 2;
  move_words(rec + off, reinterpret_cast<uint32_t*>(p.a.psic + I * N * R), N * R, p.to_records);       off += N * R;
  move_words(rec + off, reinterpret_cast<uint32_t*>(p.a.H + I * R * D), R * D, p.to_records);          off += R * D;
  move_words(rec + off, reinterpret_cast<uint32_t*>(p.a.z + I * R), R, p.to_records);
}

// n records between the arena and `records_dev` (n * rec_bytes bytes); inst_dev: n instance ids
int launch_state_io(less_ctx* c, const int32_t* inst_dev, int n, void* records_dev, size_t rec_bytes, bool to_records,
                    cudaStream_t s) {
  StateIo p;
  p.a = c->a;
  p.inst = inst_dev;
  p.records = reinterpret_cast<uint32_t*>(records_dev);
  p.N = c->d.N; p.Np = c->d.Np; p.D = c->d.D; p.R = c->d.R;
  p.rec_words = (int)(rec_bytes / 4);
  p.to_records = to_records ? 1 : 0;
  state_io_kernel<<<n, 256, 0, s>>>(p);
  return check_launch("state_io_kernel");
}

}  // namespace less
