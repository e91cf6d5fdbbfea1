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

// A read-only stream over a buffer: every thread sums 16-byte loads, eight in flight, grid-stride.  The measured
// rate of this kernel is the ceiling a read-dominated kernel (the decode step: 97 % reads) can be held against;
// a device-to-device copy, half reads and half writes, runs somewhat below it.
__global__ void __launch_bounds__(256) read_stream_kernel(const uint4 *src, size_t n16, unsigned long long *sink) {
  constexpr int kInFlight = 8;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint32_t acc = 0;
  for (; i + (kInFlight - 1) * stride < n16; i += kInFlight * stride) {
    uint4 v[kInFlight];
#pragma unroll
    for (int k = 0; k < kInFlight; ++k) v[k] = __ldcs(src + i + k * stride);
#pragma unroll
    for (int k = 0; k < kInFlight; ++k) acc += v[k].x ^ v[k].y ^ v[k].z ^ v[k].w;
  }
  for (; i < n16; i += stride) {
    const uint4 v = __ldcs(src + i);
    acc += v.x ^ v.y ^ v.z ^ v.w;
  }
  acc = __reduce_add_sync(0xffffffffu, acc);
  if ((threadIdx.x & 31) == 0 && sink) atomicAdd(sink, (unsigned long long)acc);
}

}  // namespace roco

extern "C" roco_status roco_selftest_read_stream(const void *buf, size_t bytes, unsigned long long *sink,
                                                 void *stream) {
  if (!buf || bytes < 16 || (reinterpret_cast<uintptr_t>(buf) & 15u)) return ROCO_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return ROCO_ERR_CUDA;
  roco::read_stream_kernel<<<sms * 8, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4 *>(buf), bytes / 16, sink);
  return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

extern "C" roco_status roco_selftest_wait_timeout(int32_t *status, int32_t *waited_ms, void *stream) {
  if (!status) return ROCO_ERR_INVALID_ARG;
  roco::wait_timeout_probe_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(status, waited_ms);
  return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}
