// Consistency of a budgeted cache with a full cache (Sec. 4.3, preliminary experiments): how many of the B most
// important tokens of the full cache -- by the policy's own importance score (Sec. 4.1; mean attention score:
// Sec. 4.3) -- the budgeted cache still holds.  The two sets have B elements each, so their Jaccard similarity is
// overlap / (2B - overlap).
//
// One CTA per unit.  The full cache's tokens become 64-bit keys (ordered score bits, position): the policy evicts
// in (score asc, position asc) order, so the B most important tokens are the B largest keys, and the keys are
// distinct because positions are.  The B-th largest key is found bit by bit (64 counting passes over shared
// memory); the overlap is then counted by comparing positions.
#include "common.cuh"
#include "launch.h"

namespace roco {

constexpr int kConsistencyThreads = 256;

struct ConsistencyParams {
  const float *s, *q;  // full cache statistics [U][Bf]
  const int *n, *pos, *live;
  const int *kept_pos, *kept_live;  // budgeted cache [U][Bs], [U]
  int Bf, Bs, policy;
  int *overlap;        // [U]
  float *jaccard_sum;  // [U], accumulated
  int *samples;        // [U], accumulated
  int *status;
};

__device__ __forceinline__ uint32_t ordered_bits(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__device__ __forceinline__ int block_sum_int(int v, int *red, int tid) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();  // the previous round's readers are done with red[]
  if ((tid & 31) == 0) red[tid >> 5] = v;
  __syncthreads();
  int t = 0;
#pragma unroll
  for (int w = 0; w < kConsistencyThreads / 32; ++w) t += red[w];
  return t;
}

__global__ void __launch_bounds__(kConsistencyThreads) consistency_kernel(const ConsistencyParams p) {
  extern __shared__ char smem_raw[];
  unsigned long long *keys = (unsigned long long *)smem_align(smem_raw, 16);
  __shared__ int red[kConsistencyThreads / 32];
  const int u = blockIdx.x, tid = threadIdx.x;
  const int live = p.live[u], B = p.kept_live[u];
  if (live < 0 || live > p.Bf || B < 0 || B > p.Bs) {
    if (tid == 0) { atomicOr(p.status, ROCO_DEV_BAD_LIVE); p.overlap[u] = -1; }
    return;
  }
  if (B == 0 || live < B) {  // nothing to compare yet
    if (tid == 0) p.overlap[u] = -1;
    return;
  }
  const size_t base = (size_t)u * p.Bf;
  for (int j = tid; j < live; j += kConsistencyThreads) {
    const float s = p.s[base + j], q = p.q[base + j];
    const int n = p.n[base + j];
    float score;
    if (p.policy == ROCO_POLICY_H2O) score = s;                                                       // AAS
    else if (p.policy == ROCO_POLICY_SCISSORHANDS || p.policy == ROCO_POLICY_TOVA) score = q;          // AQAS, LTAS
    else score = n > 0 ? s / (float)n : 0.f;                                                           // MAS
    keys[j] = ((unsigned long long)ordered_bits(score) << 32) | (uint32_t)p.pos[base + j];
  }
  __syncthreads();
  // T = the B-th largest key: the largest T with #{key >= T} >= B, built from the top bit down
  unsigned long long T = 0;
#pragma unroll 1
  for (int bit = 63; bit >= 0; --bit) {
    const unsigned long long cand = T | (1ull << bit);
    int c = 0;
    for (int j = tid; j < live; j += kConsistencyThreads) c += keys[j] >= cand;
    if (block_sum_int(c, red, tid) >= B) T = cand;
  }
  int ov = 0;
  const size_t kb = (size_t)u * p.Bs;
  for (int i = tid; i < B; i += kConsistencyThreads) {
    const uint32_t kp = (uint32_t)p.kept_pos[kb + i];
    for (int j = 0; j < live; ++j) {
      const unsigned long long k = keys[j];
      if ((uint32_t)k == kp) { ov += k >= T; break; }
    }
  }
  ov = block_sum_int(ov, red, tid);
  if (tid == 0) {
    p.overlap[u] = ov;
    p.jaccard_sum[u] += (float)ov / (float)(2 * B - ov);
    p.samples[u] += 1;
  }
}

roco_status launch_consistency_step(const roco_cache &full, const roco_cache &budgeted, int policy, int32_t *overlap,
                                    float *jaccard_sum, int32_t *samples, cudaStream_t stream) {
  ConsistencyParams p;
  p.s = full.s; p.q = full.q; p.n = full.n; p.pos = full.pos; p.live = full.live;
  p.kept_pos = budgeted.pos; p.kept_live = budgeted.live;
  p.Bf = full.B; p.Bs = budgeted.B; p.policy = policy;
  p.overlap = overlap; p.jaccard_sum = jaccard_sum; p.samples = samples; p.status = budgeted.status;
  const size_t smem = (size_t)full.B * 8 + 16;
  cudaError_t err = cudaFuncSetAttribute(consistency_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return ROCO_ERR_CUDA;
  consistency_kernel<<<full.S * full.G, kConsistencyThreads, smem, stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
