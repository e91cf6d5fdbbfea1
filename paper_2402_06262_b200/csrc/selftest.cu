// A check of the bounded-wait mechanism every kernel of the library relies on: one CTA waits on a shared-memory
// barrier that nothing ever completes.  The wait must run out (after kWaitLimitNs), record
// ROCO_DEV_WAIT_TIMEOUT in the caller's status word and let the kernel return normally -- no trap, no hang.
#include "common.cuh"

namespace roco {

__global__ void wait_timeout_probe_kernel(int32_t *status, int32_t *waited_ms) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    mbar_init_fence();
  }
  __syncthreads();
  const uint64_t t0 = global_timer_ns();
  mbar_wait(&bar, 0, &abort_flag, status);  // no thread arrives and no copy completes on this barrier
  __syncthreads();
  if (threadIdx.x == 0 && waited_ms) *waited_ms = (int32_t)((global_timer_ns() - t0) / 1000000ull);
}

}  // namespace roco

extern "C" roco_status roco_selftest_wait_timeout(int32_t *status, int32_t *waited_ms, void *stream) {
  if (!status) return ROCO_ERR_INVALID_ARG;
  roco::wait_timeout_probe_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(status, waited_ms);
  return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}
