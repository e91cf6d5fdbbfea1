// roco_prefill_static: the prefill entry point for callers that have no way to hand over a workspace.
//
// Some users of this library run where device memory cannot be requested at call time: a plug-in inside a
// serving runtime whose memory pool already owns the whole GPU (so cudaMalloc simply fails), or a latency
// critical loop that may not call cudaMalloc/cudaFree because those calls synchronise the device and stall
// every other stream.  roco_prefill needs scratch (row log-sum-exps, pre-eviction column statistics,
// destination slots, the device copy of the prompt lengths); here that scratch is a fixed array that lives
// in the library image itself, so the call allocates nothing -- no cudaMalloc, no cudaFree, no allocating
// library routine.  The price is a size limit and 8 MiB of device memory held by every GPU that loads the
// library, until the process exits.
#include <mutex>

#include "common.cuh"
#include "launch.h"

namespace {

constexpr size_t kScratchBytes = ROCO_PREFILL_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a stand-in for the symbol, not a device address;
// the address a kernel can use comes from cudaGetSymbolAddress, asked once per device (below).
static __device__ __align__(256) unsigned char g_prefill_scratch[kScratchBytes];

std::mutex g_mutex;
void *g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device (nullptr on failure).
void *scratch_on_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_addr[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_prefill_scratch) != cudaSuccess) return nullptr;
    g_scratch_addr[dev] = p;
  }
  return g_scratch_addr[dev];
}

}  // namespace

extern "C" roco_status roco_prefill_static(const void *Q, const void *K, const void *V, const int32_t *lens_host,
                                           int Lmax, int B, int r, int scope_mode, int count_self, float scale,
                                           roco_cache *cache, float *lse_out, float *s_full, float *q_full,
                                           void *stream) {
  if (!cache || Lmax < 1) return ROCO_ERR_INVALID_ARG;
  const size_t need = roco_prefill_workspace_bytes(cache, Lmax);
  if (need == 0) return ROCO_ERR_INVALID_ARG;
  if (need > kScratchBytes) return ROCO_ERR_WORKSPACE;  // S*G*Lmax too large for the built-in scratch
  void *scratch = scratch_on_current_device();
  if (!scratch) return ROCO_ERR_CUDA;
  // Every buffer in the scratch is written before it is read within one call (nothing has to start at
  // zero), so the previous call's contents need no clearing.
  return roco_prefill(Q, K, V, lens_host, Lmax, B, r, scope_mode, count_self, scale, cache, lse_out, s_full, q_full,
                      scratch, kScratchBytes, stream);
}
