// Self-test of the bounded waits every pipeline of this library is built on.  One small CTA sets up
// an mbarrier that no producer ever arrives at and lets a consumer wait on it through the same
// helper the kernels use, with a poll limit given by the caller.  The wait runs out, the CTA marks
// itself as given up, records where in the context's status word, pauses as the kernels do before
// they release their resources, and returns: nothing hangs and the context stays readable
// (less_poll_status answers LESS_ERR_DEVICE_TIMEOUT, less_last_status_where the code below).
#include "less_internal.cuh"
#include "pipeline.cuh"

namespace less {

constexpr int kProbeWhere = 90;

__global__ void __launch_bounds__(64) wait_probe_kernel(int32_t* status, uint32_t polls) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = *reinterpret_cast<volatile int32_t*>(status) != 0;   // a context that already gave up skips the wait
    mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 32) wait_or_give_up(&bar, 0, &abort_flag, status, kProbeWhere, polls);   // phase 0 never completes
  __syncthreads();
  drain_after_abort(&abort_flag);
}

}  // namespace less

extern "C" int less_selftest_wait_timeout(less_ctx* c, uint32_t polls, void* stream) {
  if (!c) return LESS_ERR_NULL_POINTER;
  if (polls < 1 || polls > (1u << 20)) return LESS_ERR_INVALID_CONFIG;
  less::wait_probe_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(c->a.status, polls);
  return less::check_launch("wait_probe_kernel");
}
