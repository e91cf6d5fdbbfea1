// Prefill-stage eviction to budget (Sec. 4.3 last paragraph, Sec. 5.1 "Other Details") on frozen column
// statistics, then the gather of the survivors into the cache in increasing position order.
//
// Under EXCLUDE_TOP_R, applying the per-step rule L-B times on frozen statistics equals one pass: the r
// tokens last in (variance, position) order are never in scope, so the scope's complement never changes;
// of the other tokens the L-B first in (mean, position) order leave.  Both thresholds come from radix
// selects over the fp64 bit patterns of variance and mean (non-negative doubles order like their bits).
#include "common.cuh"
#include "launch.h"
#include "select.cuh"

namespace roco {

constexpr int kBudgetThreads = 512;
constexpr int kBarAll = 1;

// One CTA per unit.  dst[u][j] = cache slot of token j, or -1 if it is evicted.
// kCached: the fp64 keys are formed once and kept in dynamic shared memory (16 bytes per token); otherwise every
// pass of the selects forms them again (two fp64 divisions per token and pass), which is ~5x slower but has no
// length limit.
template <bool kCached>
__global__ void __launch_bounds__(kBudgetThreads) budget_select_kernel(const float *s_full, const float *q_full,
                                                                       const int *lens, int G, int Lmax, int B, int r,
                                                                       int *dst, int *live, int *t_next) {
  extern __shared__ __align__(16) unsigned char budget_keys_raw[];
  __shared__ SelectScratch sc;
  __shared__ int warp_tot[kBudgetThreads / 32];
  __shared__ int base_sh;
  const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int L = lens[u / G];
  const float *s = s_full + (size_t)u * Lmax, *q = q_full + (size_t)u * Lmax;
  int *du = dst + (size_t)u * Lmax;
  if (tid == 0) { live[u] = L < B ? L : B; t_next[u] = L; }
  if (L <= B) {
    for (int j = tid; j < L; j += kBudgetThreads) du[j] = j;
    return;
  }
  const int E = L - B;  // tokens to evict
  uint64_t *vk = reinterpret_cast<uint64_t *>(budget_keys_raw), *mk = vk + Lmax;
  if (kCached) {
    for (int j = tid; j < L; j += kBudgetThreads) {
      const float sj = s[j], qj = q[j];
      vk[j] = (uint64_t)__double_as_longlong(variance_f64(sj, qj, L - j));
      mk[j] = (uint64_t)__double_as_longlong(mean_f64(sj, L - j));
    }
    __syncthreads();
  }
  auto vkey = [&](int j) {
    return kCached ? vk[j] : (uint64_t)__double_as_longlong(variance_f64(s[j], q[j], L - j));
  };
  auto mkey = [&](int j) { return kCached ? mk[j] : (uint64_t)__double_as_longlong(mean_f64(s[j], L - j)); };
  uint64_t Tv = ~0ull;
  int Pv = 0x7fffffff;
  if (r > 0) {  // the L-r tokens first in (variance, position) order may be evicted
    uint32_t rank, ties;
    Tv = radix_select<uint64_t>(vkey, [&](int) { return true; }, L, (uint32_t)(L - r - 1), sc, tid, kBudgetThreads,
                                kBarAll, &rank, &ties);
    if (ties != rank + 1) {
      uint32_t r2, t2;
      Pv = (int)radix_select<uint32_t>([&](int j) { return (uint32_t)j; }, [&](int j) { return vkey(j) == Tv; }, L,
                                       rank, sc, tid, kBudgetThreads, kBarAll, &r2, &t2);
    }
  }
  auto unprot = [&](int j) {
    if (r == 0) return true;
    const uint64_t k = vkey(j);
    return k < Tv || (k == Tv && j <= Pv);
  };
  uint32_t rank, ties;
  const uint64_t Tm = radix_select<uint64_t>(mkey, unprot, L, (uint32_t)(E - 1), sc, tid, kBudgetThreads, kBarAll,
                                             &rank, &ties);
  int Pm = 0x7fffffff;
  if (ties != rank + 1) {
    uint32_t r2, t2;
    Pm = (int)radix_select<uint32_t>([&](int j) { return (uint32_t)j; },
                                     [&](int j) { return unprot(j) && mkey(j) == Tm; }, L, rank, sc, tid,
                                     kBudgetThreads, kBarAll, &r2, &t2);
  }
  // survivors keep their order: exclusive prefix sum of the keep flags
  if (tid == 0) base_sh = 0;
  __syncthreads();
  for (int j0 = 0; j0 < L; j0 += kBudgetThreads) {
    const int j = j0 + tid;
    bool keep = false;
    if (j < L) {
      const uint64_t k = mkey(j);
      keep = !(unprot(j) && (k < Tm || (k == Tm && j <= Pm)));
    }
    const uint32_t bal = __ballot_sync(0xffffffffu, keep);
    const int before = __popc(bal & ((1u << lane) - 1u));
    if (lane == 0) warp_tot[warp] = __popc(bal);
    __syncthreads();
    int off = base_sh;
    for (int w = 0; w < warp; ++w) off += warp_tot[w];
    if (j < L) du[j] = keep ? off + before : -1;
    __syncthreads();
    if (tid == 0) {
      int t = 0;
      for (int w = 0; w < kBudgetThreads / 32; ++w) t += warp_tot[w];
      base_sh += t;
    }
    __syncthreads();
  }
}

// LOWEST_R has no one-pass form: the scope (the r lowest-variance tokens still alive) gains a member every time
// the victim leaves it.  With frozen statistics the members enter in (variance, position) order, so the kernel
// sorts the tokens once by that order (bitonic sort of 64-bit keys = variance bits : position, in the caller's
// scratch) and then one warp replays the L-B evictions on a scope held in shared memory: pop the lowest
// (mean, position), admit the next token of the sorted order.  One CTA per unit.
constexpr int kLowestMaxR = 2048;

__global__ void __launch_bounds__(kBudgetThreads) budget_lowest_kernel(const float *s_full, const float *q_full,
                                                                       const int *lens, int G, int Lmax, int Lp2max,
                                                                       int B, int r, unsigned long long *sortbuf,
                                                                       int *dst, int *live, int *t_next) {
  __shared__ float sc_mean[kLowestMaxR];
  __shared__ int sc_idx[kLowestMaxR];
  __shared__ int warp_tot[kBudgetThreads / 32];
  __shared__ int base_sh;
  const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int L = lens[u / G];
  const float *s = s_full + (size_t)u * Lmax, *q = q_full + (size_t)u * Lmax;
  int *du = dst + (size_t)u * Lmax;
  unsigned long long *keys = sortbuf + (size_t)u * Lp2max;
  if (tid == 0) { live[u] = L < B ? L : B; t_next[u] = L; }
  if (L <= B) {
    for (int j = tid; j < L; j += kBudgetThreads) du[j] = j;
    return;
  }
  int Lp2 = 1;
  while (Lp2 < L) Lp2 <<= 1;
  for (int j = tid; j < Lp2; j += kBudgetThreads) {
    unsigned long long k = ~0ull;
    if (j < L) {
      k = ((unsigned long long)__float_as_uint((float)variance_f64(s[j], q[j], L - j)) << 32) | (unsigned)j;
      du[j] = 0;  // 0 = alive, -1 = evicted (turned into slots at the end)
    }
    keys[j] = k;
  }
  __syncthreads();
  for (int k = 2; k <= Lp2; k <<= 1) {
    for (int jj = k >> 1; jj > 0; jj >>= 1) {
      for (int i = tid; i < Lp2; i += kBudgetThreads) {
        const int p = i ^ jj;
        if (p > i) {
          const unsigned long long a = keys[i], b = keys[p];
          const bool up = (i & k) == 0;
          if ((a > b) == up) { keys[i] = b; keys[p] = a; }
        }
      }
      __syncthreads();
    }
  }
  if (warp == 0) {
    const int rs = r < L ? r : L;
    for (int k = lane; k < rs; k += 32) {
      const int j = (int)(keys[k] & 0xffffffffu);
      sc_idx[k] = j;
      sc_mean[k] = mean_fast(s[j], L - j);
    }
    __syncwarp();
    int cursor = rs;
    for (int it = 0; it < L - B; ++it) {
      float bm = INFINITY;
      int bi = 0x7fffffff, bk = -1;
      for (int k = lane; k < rs; k += 32) {
        const float m = sc_mean[k];
        const int j = sc_idx[k];
        if (m < bm || (m == bm && j < bi)) { bm = m; bi = j; bk = k; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, bm, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        const int ok = __shfl_xor_sync(0xffffffffu, bk, o);
        if (ok >= 0 && (bk < 0 || om < bm || (om == bm && oi < bi))) { bm = om; bi = oi; bk = ok; }
      }
      if (bk < 0) break;  // NaN statistics everywhere: nothing left to pop
      if (lane == 0) {
        du[bi] = -1;
        if (cursor < L) {
          const int j = (int)(keys[cursor] & 0xffffffffu);
          sc_idx[bk] = j;
          sc_mean[bk] = mean_fast(s[j], L - j);
        } else {
          sc_idx[bk] = 0x7fffffff;
          sc_mean[bk] = INFINITY;
        }
      }
      ++cursor;
      __syncwarp();
    }
  }
  // survivors keep their order: exclusive prefix sum of the keep flags
  if (tid == 0) base_sh = 0;
  __syncthreads();
  for (int j0 = 0; j0 < L; j0 += kBudgetThreads) {
    const int j = j0 + tid;
    const bool keep = j < L && du[j] == 0;
    const uint32_t bal = __ballot_sync(0xffffffffu, keep);
    const int before = __popc(bal & ((1u << lane) - 1u));
    if (lane == 0) warp_tot[warp] = __popc(bal);
    __syncthreads();
    int off = base_sh;
    for (int w = 0; w < warp; ++w) off += warp_tot[w];
    if (j < L) du[j] = keep ? off + before : -1;
    __syncthreads();
    if (tid == 0) {
      int t = 0;
      for (int w = 0; w < kBudgetThreads / 32; ++w) t += warp_tot[w];
      base_sh += t;
    }
    __syncthreads();
  }
}

// grid U * chunks (unit-major); each CTA moves up to 64 tokens.  Also clears the slots past `live`.
template <int ROWB>
__global__ void __launch_bounds__(256) gather_kernel(const char *K, const char *V, const float *s_full,
                                                     const float *q_full, const int *dst, const int *lens, int G,
                                                     int Lmax, int B, int chunks, char *Kc, char *Vc, float *sc,
                                                     float *qc, int *nc, int *posc) {
  constexpr int kChunksPerRow = ROWB / 16;
  const int u = blockIdx.x / chunks, c0 = (int)(blockIdx.x % chunks) * 64;
  const int L = lens[u / G], tid = threadIdx.x;
  const int live = L < B ? L : B;
  const size_t in_off = (size_t)u * Lmax, out_off = (size_t)u * B;
  for (int w = tid; w < 64 * 2 * kChunksPerRow; w += 256) {
    const int k = w / (2 * kChunksPerRow), rem = w % (2 * kChunksPerRow);
    const int j = c0 + k;
    if (j >= L) continue;
    const int slot = dst[in_off + j];
    if (slot < 0) continue;
    const bool isv = rem >= kChunksPerRow;
    const int c = isv ? rem - kChunksPerRow : rem;
    const uint4 val = *((const uint4 *)((isv ? V : K) + (in_off + j) * ROWB) + c);
    *((uint4 *)((isv ? Vc : Kc) + (out_off + slot) * ROWB) + c) = val;
  }
  if (tid < 64) {
    const int j = c0 + tid;
    if (j < L) {
      const int slot = dst[in_off + j];
      if (slot >= 0) {
        sc[out_off + slot] = s_full[in_off + j];
        qc[out_off + slot] = q_full[in_off + j];
        nc[out_off + slot] = L - j;  // Count: queries j..L-1 have attended token j
        posc[out_off + slot] = j;
      }
    }
    if (j >= live && j < B) { sc[out_off + j] = 0.f; qc[out_off + j] = 0.f; nc[out_off + j] = 0; posc[out_off + j] = -1; }
  }
}

int budget_lowest_max_r() { return kLowestMaxR; }

roco_status launch_budget_select_gather(const roco_cache &c, int Lmax, const int *lens_dev, int maxlen, int r,
                                        int scope_mode, const void *K, const void *V, const float *s_full,
                                        const float *q_full, int *dst, unsigned long long *sortbuf, int Lp2max,
                                        cudaStream_t stream) {
  const int U = c.S * c.G;
  if (scope_mode == ROCO_SCOPE_LOWEST_R && maxlen > c.B)
    budget_lowest_kernel<<<U, kBudgetThreads, 0, stream>>>(s_full, q_full, lens_dev, c.G, Lmax, Lp2max, c.B, r,
                                                           sortbuf, dst, c.live, c.t_next);
  else {
    const size_t key_bytes = (size_t)Lmax * 16;
    if (key_bytes <= 200 * 1024 &&
        cudaFuncSetAttribute(budget_select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)key_bytes) == cudaSuccess)
      budget_select_kernel<true><<<U, kBudgetThreads, key_bytes, stream>>>(s_full, q_full, lens_dev, c.G, Lmax, c.B,
                                                                           r, dst, c.live, c.t_next);
    else
      budget_select_kernel<false><<<U, kBudgetThreads, 0, stream>>>(s_full, q_full, lens_dev, c.G, Lmax, c.B, r, dst,
                                                                    c.live, c.t_next);
  }
  const int span = maxlen > c.B ? maxlen : c.B;
  const int chunks = (span + 63) / 64;
  const unsigned grid = (unsigned)U * (unsigned)chunks;
  const int rowb = c.d * (c.kv_dtype == ROCO_BF16 ? 2 : 4);
#define ROCO_GATHER(RB)                                                                                         \
  gather_kernel<RB><<<grid, 256, 0, stream>>>((const char *)K, (const char *)V, s_full, q_full, dst, lens_dev, c.G, \
                                              Lmax, c.B, chunks, (char *)c.K, (char *)c.V, c.s, c.q, c.n, c.pos)
  if (rowb == 128) ROCO_GATHER(128);
  else if (rowb == 256) ROCO_GATHER(256);
  else if (rowb == 512) ROCO_GATHER(512);
  else return ROCO_ERR_UNSUPPORTED;
#undef ROCO_GATHER
  return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
