// Prefill statistics on CUDA cores: row log-sum-exp of the causal score matrix (Eq. 1 with the mask of
// Sec. 2.1) and, from it, the column sums s_j = sum_i P_ij and q_j = sum_i P_ij^2 (Sec. 4.3) without ever
// storing P.  Works for fp32 and bf16 inputs and d in {64, 128}; it is the path for small problems and for
// shapes the tensor-core path does not cover.
#include "common.cuh"
#include "launch.h"

namespace roco {

constexpr int kPT = 64;         // tile edge: 64 query rows x 64 key columns per step
constexpr int kPThreads = 256;  // 16 x 16 threads, 4 x 4 scores each

template <typename T, int D>
__device__ __forceinline__ void load_tile(float *dst /*[64][D+1]*/, const T *src, int row0, int L, int tid) {
  // rows row0..row0+63 of a [L][D] matrix, zero-filled past L
  for (int idx = tid; idx < kPT * D; idx += kPThreads) {
    const int r = idx / D, c = idx % D;
    const int g = row0 + r;
    dst[r * (D + 1) + c] = (g < L) ? Elem<T>::load(src + (size_t)g * D + c) : 0.f;
  }
}

template <int D>
__device__ __forceinline__ void score_tile(const float *Qs, const float *Ks, int ty, int tx, float (&acc)[4][4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 4
  for (int c = 0; c < D; ++c) {
    float a[4], b[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) a[i] = Qs[(ty * 4 + i) * (D + 1) + c];
#pragma unroll
    for (int j = 0; j < 4; ++j) b[j] = Ks[(tx * 4 + j) * (D + 1) + c];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
  }
}

// grid U * tiles, unit-major; heavy (late) row tiles first.  lse[u][i] = log sum_{j<=i} exp(scale * Q_i.K_j)
template <typename T, int D>
__global__ void __launch_bounds__(kPThreads) prefill_lse_kernel(const T *Q, const T *K, const int *lens, int G,
                                                                int Lmax, int tiles, float scale, float *lse) {
  extern __shared__ float psm[];
  float *Qs = psm, *Ks = psm + kPT * (D + 1);
  const int u = blockIdx.x / tiles, L = lens[u / G];
  const int row0 = (tiles - 1 - (int)(blockIdx.x % tiles)) * kPT;
  if (row0 >= L) return;
  const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
  const T *Qu = Q + (size_t)u * Lmax * D, *Ku = K + (size_t)u * Lmax * D;
  const float zscale = scale * kLog2e;
  load_tile<T, D>(Qs, Qu, row0, L, tid);
  float m[4], l[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) { m[i] = -INFINITY; l[i] = 0.f; }
  for (int col0 = 0; col0 <= row0; col0 += kPT) {
    __syncthreads();
    load_tile<T, D>(Ks, Ku, col0, L, tid);
    __syncthreads();
    float acc[4][4];
    score_tile<D>(Qs, Ks, ty, tx, acc);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int gi = row0 + ty * 4 + i;
      float tmax = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int gj = col0 + tx * 4 + j;
        acc[i][j] = (gj <= gi && gi < L) ? acc[i][j] * zscale : -INFINITY;
        tmax = fmaxf(tmax, acc[i][j]);
      }
#pragma unroll
      for (int o = 1; o < 16; o <<= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
      const float mn = fmaxf(m[i], tmax);
      float part = 0.f;
      if (mn > -INFINITY) {
#pragma unroll
        for (int j = 0; j < 4; ++j) part += exp2f(acc[i][j] - mn);
      }
#pragma unroll
      for (int o = 1; o < 16; o <<= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
      l[i] = (mn > -INFINITY) ? l[i] * exp2f(m[i] - mn) + part : 0.f;
      m[i] = mn;
    }
  }
  if (tx == 0) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int gi = row0 + ty * 4 + i;
      if (gi < L) lse[(size_t)u * Lmax + gi] = (m[i] + log2f(l[i])) * kLn2;
    }
  }
}

// grid U * tiles, unit-major; heavy (early) column tiles first.  s[u][j] = sum_{i>=j} P_ij, q[u][j] = sum_{i>=j} P_ij^2 with P_ij = exp(z_ij - lse_i)
template <typename T, int D>
__global__ void __launch_bounds__(kPThreads) prefill_colstats_kernel(const T *Q, const T *K, const int *lens, int G,
                                                                     int Lmax, int tiles, float scale, const float *lse,
                                                                     float *s_full, float *q_full) {
  extern __shared__ float psm[];
  float *Qs = psm, *Ks = psm + kPT * (D + 1), *lse2 = Ks + kPT * (D + 1), *red = lse2 + kPT;
  const int u = blockIdx.x / tiles, L = lens[u / G];
  const int col0 = (int)(blockIdx.x % tiles) * kPT;
  if (col0 >= L) return;
  const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
  const T *Qu = Q + (size_t)u * Lmax * D, *Ku = K + (size_t)u * Lmax * D;
  const float zscale = scale * kLog2e;
  load_tile<T, D>(Ks, Ku, col0, L, tid);
  float cs[4] = {0.f, 0.f, 0.f, 0.f}, cq[4] = {0.f, 0.f, 0.f, 0.f};
  for (int row0 = col0; row0 < L; row0 += kPT) {
    __syncthreads();
    load_tile<T, D>(Qs, Qu, row0, L, tid);
    if (tid < kPT) lse2[tid] = (row0 + tid < L) ? lse[(size_t)u * Lmax + row0 + tid] * kLog2e : 0.f;
    __syncthreads();
    float acc[4][4];
    score_tile<D>(Qs, Ks, ty, tx, acc);
    float ts[4] = {0.f, 0.f, 0.f, 0.f}, tq[4] = {0.f, 0.f, 0.f, 0.f};  // this tile's contribution
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int gi = row0 + ty * 4 + i;
      const float li = lse2[ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int gj = col0 + tx * 4 + j;
        if (gj <= gi && gi < L) {
          const float pij = exp2f(fmaf(acc[i][j], zscale, -li));
          ts[j] += pij;
          tq[j] = fmaf(pij, pij, tq[j]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) { cs[j] += ts[j]; cq[j] += tq[j]; }
  }
  // sum over the 16 row groups (ty) that share a column
  __syncthreads();
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    red[ty * kPT + tx * 4 + j] = cs[j];
    red[16 * kPT + ty * kPT + tx * 4 + j] = cq[j];
  }
  __syncthreads();
  if (tid < kPT) {
    float a = 0.f, b = 0.f;
#pragma unroll
    for (int g = 0; g < 16; ++g) { a += red[g * kPT + tid]; b += red[16 * kPT + g * kPT + tid]; }
    const int gj = col0 + tid;
    if (gj < L) { s_full[(size_t)u * Lmax + gj] = a; q_full[(size_t)u * Lmax + gj] = b; }
  }
}

// grid U * tiles, unit-major; heavy (late) row tiles first.  out[u][i] = sum_{j<=i} exp(scale * Q_i.K_j - lse_i) V_j
// (Eq. 1 with the causal mask of Sec. 2.1) from the row log-sum-exp of prefill_lse_kernel: per key tile the 64 x 64
// block of probabilities goes through shared memory, and each thread keeps 4 rows x D/16 columns of the output.
template <typename T, int D>
__global__ void __launch_bounds__(kPThreads) prefill_attend_simt_kernel(const T *Q, const T *K, const T *V,
                                                                        const int *lens, int G, int Lmax, int tiles,
                                                                        float scale, const float *lse, T *out) {
  extern __shared__ float psm[];
  float *Qs = psm, *Ks = psm + kPT * (D + 1), *Ps = Ks + kPT * (D + 1), *lse2 = Ps + kPT * (kPT + 1);
  const int u = blockIdx.x / tiles, L = lens[u / G];
  const int row0 = (tiles - 1 - (int)(blockIdx.x % tiles)) * kPT;
  if (row0 >= L) return;
  const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
  const T *Qu = Q + (size_t)u * Lmax * D, *Ku = K + (size_t)u * Lmax * D, *Vu = V + (size_t)u * Lmax * D;
  const float zscale = scale * kLog2e;
  load_tile<T, D>(Qs, Qu, row0, L, tid);
  if (tid < kPT) lse2[tid] = (row0 + tid < L) ? lse[(size_t)u * Lmax + row0 + tid] * kLog2e : 0.f;
  float o[4][D / 16];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int c = 0; c < D / 16; ++c) o[i][c] = 0.f;
  for (int col0 = 0; col0 <= row0; col0 += kPT) {
    __syncthreads();  // the previous tile's values (in Ks) and probabilities have been used
    load_tile<T, D>(Ks, Ku, col0, L, tid);
    __syncthreads();
    float acc[4][4];
    score_tile<D>(Qs, Ks, ty, tx, acc);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int gi = row0 + ty * 4 + i;
      const float li = lse2[ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int gj = col0 + tx * 4 + j;
        Ps[(ty * 4 + i) * (kPT + 1) + tx * 4 + j] = (gj <= gi && gi < L) ? exp2f(fmaf(acc[i][j], zscale, -li)) : 0.f;
      }
    }
    __syncthreads();  // scores done with the keys: their place takes the values (rows past L read as zero)
    load_tile<T, D>(Ks, Vu, col0, L, tid);
    __syncthreads();
#pragma unroll 4
    for (int j = 0; j < kPT; ++j) {
      float pr[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) pr[i] = Ps[(ty * 4 + i) * (kPT + 1) + j];
#pragma unroll
      for (int c = 0; c < D / 16; ++c) {
        const float v = Ks[j * (D + 1) + tx + 16 * c];
#pragma unroll
        for (int i = 0; i < 4; ++i) o[i][c] = fmaf(pr[i], v, o[i][c]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gi = row0 + ty * 4 + i;
    if (gi < L) {
#pragma unroll
      for (int c = 0; c < D / 16; ++c) Elem<T>::store(out + ((size_t)u * Lmax + gi) * D + tx + 16 * c, o[i][c]);
    }
  }
}

template <typename T, int D>
static cudaError_t launch_attend_t(int S, int G, int Lmax, const int *lens, int maxlen, const void *Q, const void *K,
                                   const void *V, float scale, const float *lse, void *out, cudaStream_t stream) {
  const size_t smem = (2 * kPT * (D + 1) + kPT * (kPT + 1) + kPT) * sizeof(float);
  cudaError_t err = cudaFuncSetAttribute(prefill_attend_simt_kernel<T, D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  const int tiles = (maxlen + kPT - 1) / kPT;
  const unsigned grid = (unsigned)(S * G) * (unsigned)tiles;
  prefill_attend_simt_kernel<T, D><<<grid, kPThreads, smem, stream>>>((const T *)Q, (const T *)K, (const T *)V, lens, G,
                                                                     Lmax, tiles, scale, lse, (T *)out);
  return cudaGetLastError();
}

roco_status launch_prefill_attend_simt(int kv_dtype, int d, int S, int G, int Lmax, const int *lens_dev, int maxlen,
                                       const void *Q, const void *K, const void *V, float scale, const float *lse,
                                       void *out, cudaStream_t stream) {
  cudaError_t err;
  if (kv_dtype == ROCO_BF16 && d == 128)
    err = launch_attend_t<__nv_bfloat16, 128>(S, G, Lmax, lens_dev, maxlen, Q, K, V, scale, lse, out, stream);
  else if (kv_dtype == ROCO_BF16 && d == 64)
    err = launch_attend_t<__nv_bfloat16, 64>(S, G, Lmax, lens_dev, maxlen, Q, K, V, scale, lse, out, stream);
  else if (kv_dtype == ROCO_F32 && d == 128)
    err = launch_attend_t<float, 128>(S, G, Lmax, lens_dev, maxlen, Q, K, V, scale, lse, out, stream);
  else if (kv_dtype == ROCO_F32 && d == 64)
    err = launch_attend_t<float, 64>(S, G, Lmax, lens_dev, maxlen, Q, K, V, scale, lse, out, stream);
  else
    return ROCO_ERR_UNSUPPORTED;
  return err == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

template <typename T, int D>
static cudaError_t launch_t(int S, int G, int Lmax, const int *lens, int maxlen, const void *Q, const void *K,
                            float scale, float *lse, float *s_full, float *q_full, cudaStream_t stream) {
  const size_t smem1 = 2 * kPT * (D + 1) * sizeof(float);
  const size_t smem2 = smem1 + (kPT + 32 * kPT) * sizeof(float);
  cudaError_t err = cudaFuncSetAttribute(prefill_lse_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem1);
  if (err != cudaSuccess) return err;
  err = cudaFuncSetAttribute(prefill_colstats_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem2);
  if (err != cudaSuccess) return err;
  const int tiles = (maxlen + kPT - 1) / kPT;
  const unsigned grid = (unsigned)(S * G) * (unsigned)tiles;
  prefill_lse_kernel<T, D><<<grid, kPThreads, smem1, stream>>>((const T *)Q, (const T *)K, lens, G, Lmax, tiles, scale,
                                                               lse);
  prefill_colstats_kernel<T, D><<<grid, kPThreads, smem2, stream>>>((const T *)Q, (const T *)K, lens, G, Lmax, tiles,
                                                                    scale, lse, s_full, q_full);
  return cudaGetLastError();
}

roco_status launch_prefill_stats_simt(int kv_dtype, int d, int S, int G, int Lmax, const int *lens_dev, int maxlen,
                                      const void *Q, const void *K, float scale, float *lse, float *s_full,
                                      float *q_full, cudaStream_t stream) {
  cudaError_t err;
  if (kv_dtype == ROCO_BF16 && d == 128)
    err = launch_t<__nv_bfloat16, 128>(S, G, Lmax, lens_dev, maxlen, Q, K, scale, lse, s_full, q_full, stream);
  else if (kv_dtype == ROCO_BF16 && d == 64)
    err = launch_t<__nv_bfloat16, 64>(S, G, Lmax, lens_dev, maxlen, Q, K, scale, lse, s_full, q_full, stream);
  else if (kv_dtype == ROCO_F32 && d == 128)
    err = launch_t<float, 128>(S, G, Lmax, lens_dev, maxlen, Q, K, scale, lse, s_full, q_full, stream);
  else if (kv_dtype == ROCO_F32 && d == 64)
    err = launch_t<float, 64>(S, G, Lmax, lens_dev, maxlen, Q, K, scale, lse, s_full, q_full, stream);
  else
    return ROCO_ERR_UNSUPPORTED;
  return err == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
