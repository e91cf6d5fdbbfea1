// Decode step split over the cache slots, for calls with few units (one layer of a small batch): with one CTA per
// unit such a call cannot fill the GPU, so each unit's slots are divided among `splits` CTAs.  Three launches on
// one stream (in the order of Fig. 1: evict, insert, attend; under ROCO_ATTEND_FIRST launches 2 and 3 come first, over
// the cache as it stands, and launch 1 then selects on the updated statistics and inserts with empty ones):
//   1. split_policy_kernel   one CTA per unit: scope + victim (Sec. 4.3), in-place overwrite with the new K/V;
//   2. split_attend_kernel   one CTA per (unit, slot range): scores, local (max, sum), local sum of p*V; the
//                            log2-domain scores and the partial results go to the caller's workspace;
//   3. split_merge_kernel    one CTA per unit: merges the partial (max, sum, out) triples, writes the output and
//                            the log-sum-exp, then -- the cheap second pass -- turns the saved scores into
//                            probabilities with that log-sum-exp and applies Acc += p, Acc^square += p^2, Count += 1.
// K and V are still read from HBM exactly once; the extra traffic is the 4 bytes per slot of saved scores.
#include "common.cuh"
#include "launch.h"
#include "select.cuh"

namespace roco {

constexpr int kSpConsumerWarps = 8;
constexpr int kSpConsumers = kSpConsumerWarps * 32;
constexpr int kSpThreads = kSpConsumers + 32;
constexpr int kSpTile = 16384;
constexpr int kSpStages = 4;
constexpr int kSpBar = 1;
constexpr int kSpPolicyThreads = 512;  // the selection is the serial part of a call with few units: go wide
constexpr int kSpMergeThreads = 512;

struct SplitParams {
  const char *K, *V;
  float *s, *q;
  int *n, *pos, *live, *t_next, *status;
  const char *qv, *k_new, *v_new;
  char *out;
  float *lse;
  int *ev_slot, *ev_pos;
  int B, r, scope_mode, splits, order;
  float scale;
  // workspace
  float *zbuf;   // [U][B]        log2-domain scores
  float *part;   // [U][splits][2 + d]  local max, local sum, local sum of p*V
  int *slot_new; // [U]           slot that received the new token
};

// ---- 1. policy: one CTA per unit
template <typename T, int D>
__global__ void __launch_bounds__(kSpPolicyThreads) split_policy_kernel(const SplitParams p) {
  constexpr int kRowBytes = D * (int)sizeof(T);
  constexpr int kLanesPerRow = kRowBytes / 16;
  extern __shared__ char sp_smem_raw[];
  uint32_t *vkey = reinterpret_cast<uint32_t *>(sp_smem_raw);
  float *mkey = reinterpret_cast<float *>(vkey + align_up((size_t)p.B, 4));
  __shared__ SelectScratch sel;
  const int u = blockIdx.x, tid = threadIdx.x, B = p.B;
  const size_t unit_st = (size_t)u * B, unit_kv = (size_t)u * B * kRowBytes;
  int live0 = p.live[u];
  if (live0 < 0 || live0 > B) {
    if (tid == 0) atomicOr(p.status, ROCO_DEV_BAD_LIVE);
    live0 = live0 < 0 ? 0 : B;
  }
  const int t_new = p.t_next[u];
  __syncthreads();  // every thread has read live / t_next before thread 0 rewrites them
  int e = live0, ev_slot = -1, ev_pos = -1;
  if (live0 == B) {
    const int m = scope_size(B, p.r, p.scope_mode);
    e = group_select_victim(p.s + unit_st, p.q + unit_st, p.n + unit_st, p.pos + unit_st, B, m, vkey, mkey, sel, tid,
                            kSpPolicyThreads, kSpBar);
    if (e < 0) {
      if (tid == 0) atomicOr(p.status, ROCO_DEV_BAD_VICTIM);
      e = 0;
    }
    ev_slot = e;
    if (tid == 0) ev_pos = p.pos[unit_st + e];
  }
  if (tid == 0) {
    p.slot_new[u] = e;
    p.pos[unit_st + e] = t_new;
    p.ev_slot[u] = ev_slot;
    if (p.ev_pos) p.ev_pos[u] = ev_pos;
    p.live[u] = live0 == B ? B : live0 + 1;
    p.t_next[u] = t_new + 1;
    if (p.order == ROCO_ATTEND_FIRST) {  // the new token was not attended over: its statistics start empty
      p.s[unit_st + e] = 0.f;
      p.q[unit_st + e] = 0.f;
      p.n[unit_st + e] = 0;
    }
  }
  if (tid >= 32 && tid < 32 + 2 * kLanesPerRow) {  // in-place overwrite, 16 bytes per thread
    const int c = tid - 32;
    const bool isv = c >= kLanesPerRow;
    const int cc = isv ? c - kLanesPerRow : c;
    const uint4 val = *((const uint4 *)((isv ? p.v_new : p.k_new) + (size_t)u * kRowBytes) + cc);
    *((uint4 *)(const_cast<char *>(isv ? p.V : p.K) + unit_kv + (size_t)e * kRowBytes) + cc) = val;
  }
}

// ---- 2. attention over one slot range of one unit
template <typename T, int D>
__global__ void __launch_bounds__(kSpThreads) split_attend_kernel(const SplitParams p) {
  constexpr int kRowBytes = D * (int)sizeof(T);
  constexpr int kLanesPerRow = kRowBytes / 16;
  constexpr int kRowsPerLoad = 32 / kLanesPerRow;
  constexpr int kTileRows = kSpTile / kRowBytes;
  constexpr int kRowsPerWarp = kTileRows / kSpConsumerWarps;
  constexpr int kLoads = kRowsPerWarp / kRowsPerLoad;
  constexpr int kEPC = Elem<T>::kPerChunk;

  extern __shared__ char sp_smem_raw[];
  char *ring = smem_align(sp_smem_raw, 128);
  float *z = reinterpret_cast<float *>(ring + (size_t)kSpStages * kSpTile);   // [range rows]
  float *qf = z + align_up((size_t)p.B, 4);
  float *outred = qf + D;                                                     // [8][D]
  float *red = outred + kSpConsumerWarps * D;                                 // [32]
  uint64_t *full = reinterpret_cast<uint64_t *>(red + 32);
  uint64_t *empty = full + kSpStages;
  int *flag = reinterpret_cast<int *>(empty + kSpStages);
  volatile int *abort_flag = flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c = blockIdx.x, u = blockIdx.y, B = p.B, splits = p.splits;
  const size_t unit_kv = (size_t)u * B * kRowBytes;
  const int live = p.live[u];  // slots the query attends over (EVICT_FIRST: the policy kernel has added the new one)
  // slot range of this CTA: whole tiles
  const int tiles_total = (live + kTileRows - 1) / kTileRows;
  const int tiles_per = (tiles_total + splits - 1) / splits;
  const int t0 = c * tiles_per, t1 = min(tiles_total, t0 + tiles_per);
  const int n_tiles = t1 > t0 ? t1 - t0 : 0;
  const int j0 = t0 * kTileRows;
  const int j1 = min(live, t1 * kTileRows);
  float *part = p.part + ((size_t)u * splits + c) * (2 + D);

  if (tid == 0) {
    for (int i = 0; i < kSpStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], kSpConsumerWarps); }
    *flag = 0;
    mbar_init_fence();
  }
  __syncthreads();

  if (warp == kSpConsumerWarps) {
    if (lane == 0) {
      for (int g = 0; g < 2 * n_tiles; ++g) {
        const int st = g % kSpStages;
        if (g >= kSpStages) mbar_wait(&empty[st], ((g / kSpStages) - 1) & 1, abort_flag, p.status);
        const int it = t0 + ((g < n_tiles) ? g : g - n_tiles);
        const char *src = ((g < n_tiles) ? p.K : p.V) + unit_kv + (size_t)it * kSpTile;
        int rows = live - it * kTileRows;
        if (rows > kTileRows) rows = kTileRows;
        const uint32_t bytes = (uint32_t)rows * kRowBytes;
        mbar_expect_tx(&full[st], bytes);
        bulk_g2s(ring + (size_t)st * kSpTile, src, bytes, &full[st]);
      }
    }
    return;
  }

  if (tid < D) qf[tid] = Elem<T>::load((const T *)p.qv + (size_t)u * D + tid);
  named_bar_sync(kSpBar, kSpConsumers);
  const float zscale = p.scale * kLog2e;
  const int lane_chunk = lane % kLanesPerRow, lane_row = lane / kLanesPerRow;
  float qreg[kEPC];
#pragma unroll
  for (int i = 0; i < kEPC; ++i) qreg[i] = qf[lane_chunk * kEPC + i];

  for (int it = 0; it < n_tiles; ++it) {
    const int st = it % kSpStages;
    mbar_wait(&full[st], (it / kSpStages) & 1, abort_flag, p.status);
    const char *tile = ring + (size_t)st * kSpTile;
    // partial dot products of all the rows this lane touches, then one butterfly for all of them
    float acc[kLoads];
#pragma unroll
    for (int l = 0; l < kLoads; ++l) {
      const int row = warp * kRowsPerWarp + l * kRowsPerLoad + lane_row;
      const uint4 ch = *(const uint4 *)(tile + (size_t)row * kRowBytes + lane_chunk * 16);
      float f[kEPC];
      Elem<T>::unpack(ch, f);
      acc[l] = 0.f;
#pragma unroll
      for (int i = 0; i < kEPC; ++i) acc[l] = fmaf(f[i], qreg[i], acc[l]);
    }
#pragma unroll
    for (int o = kLanesPerRow / 2; o > 0; o >>= 1) {
#pragma unroll
      for (int l = 0; l < kLoads; ++l) acc[l] += __shfl_xor_sync(0xffffffffu, acc[l], o);
    }
#pragma unroll
    for (int l = 0; l < kLoads; ++l) {
      const int j = (t0 + it) * kTileRows + warp * kRowsPerWarp + l * kRowsPerLoad + lane_row;
      if (lane_chunk == 0 && j < j1) z[j - j0] = acc[l] * zscale;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty[st]);
  }
  named_bar_sync(kSpBar, kSpConsumers);

  // local max and sum; the scores themselves are saved for the statistics pass of the merge kernel
  const int nloc = j1 - j0;
  float zmax = -INFINITY;
  for (int j = tid; j < nloc; j += kSpConsumers) zmax = fmaxf(zmax, z[j]);
  zmax = warp_max(zmax);
  if (lane == 0) red[warp] = zmax;
  named_bar_sync(kSpBar, kSpConsumers);
  zmax = red[0];
#pragma unroll
  for (int w = 1; w < kSpConsumerWarps; ++w) zmax = fmaxf(zmax, red[w]);
  float zsum = 0.f;
  for (int j = tid; j < nloc; j += kSpConsumers) {
    const float zj = z[j];
    p.zbuf[(size_t)u * B + j0 + j] = zj;
    const float ex = exp2f(zj - zmax);
    z[j] = ex;
    zsum += ex;
  }
  zsum = warp_sum(zsum);
  if (lane == 0) red[16 + warp] = zsum;
  named_bar_sync(kSpBar, kSpConsumers);
  zsum = red[16];
#pragma unroll
  for (int w = 1; w < kSpConsumerWarps; ++w) zsum += red[16 + w];

  // local sum of p*V with the local max as reference
  float acc[kEPC];
#pragma unroll
  for (int i = 0; i < kEPC; ++i) acc[i] = 0.f;
  for (int it = 0; it < n_tiles; ++it) {
    const int g = n_tiles + it;
    const int st = g % kSpStages;
    mbar_wait(&full[st], (g / kSpStages) & 1, abort_flag, p.status);
    const char *tile = ring + (size_t)st * kSpTile;
#pragma unroll
    for (int l = 0; l < kLoads; ++l) {
      const int row = warp * kRowsPerWarp + l * kRowsPerLoad + lane_row;
      const int j = (t0 + it) * kTileRows + row;
      if (j < j1) {
        const uint4 ch = *(const uint4 *)(tile + (size_t)row * kRowBytes + lane_chunk * 16);
        float f[kEPC];
        Elem<T>::unpack(ch, f);
        const float pj = z[j - j0];
#pragma unroll
        for (int i = 0; i < kEPC; ++i) acc[i] = fmaf(pj, f[i], acc[i]);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty[st]);
  }
#pragma unroll
  for (int i = 0; i < kEPC; ++i) {
#pragma unroll
    for (int o = kLanesPerRow; o < 32; o <<= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
  }
  if (lane_row == 0) {
#pragma unroll
    for (int i = 0; i < kEPC; ++i) outred[warp * D + lane_chunk * kEPC + i] = acc[i];
  }
  named_bar_sync(kSpBar, kSpConsumers);
  if (tid < D) {
    float o = 0.f;
#pragma unroll
    for (int w = 0; w < kSpConsumerWarps; ++w) o += outred[w * D + tid];
    part[2 + tid] = o;
  }
  if (tid == 0) { part[0] = zmax; part[1] = zsum; }
}

// ---- 3. merge of the partial results, output, and the statistics pass
template <typename T, int D>
__global__ void __launch_bounds__(kSpMergeThreads) split_merge_kernel(const SplitParams p) {
  __shared__ float w_sh[64];
  __shared__ float ml_sh[2];
  const int u = blockIdx.x, tid = threadIdx.x, B = p.B, splits = p.splits;
  const size_t unit_st = (size_t)u * B;
  const int live = p.live[u];
  const float *part = p.part + (size_t)u * splits * (2 + D);
  if (tid == 0) {
    float M = -INFINITY;
    for (int c = 0; c < splits; ++c) M = fmaxf(M, part[c * (2 + D)]);
    float L = 0.f;
    for (int c = 0; c < splits; ++c) {
      const float m = part[c * (2 + D)];
      const float w = (m > -INFINITY) ? exp2f(m - M) : 0.f;  // an empty range has max -inf and sum 0
      w_sh[c] = w;
      L += w * part[c * (2 + D) + 1];
    }
    ml_sh[0] = M; ml_sh[1] = L;
    if (p.lse) p.lse[u] = live > 0 ? (M + log2f(L)) * kLn2 : -INFINITY;
  }
  __syncthreads();
  const float M = ml_sh[0], L = ml_sh[1];
  const float inv = live > 0 ? 1.f / L : 0.f;
  if (tid < D) {
    float o = 0.f;
    for (int c = 0; c < splits; ++c) o = fmaf(w_sh[c], part[c * (2 + D) + 2 + tid], o);
    Elem<T>::store((T *)p.out + (size_t)u * D + tid, o * inv);
  }
  // statistics of Sec. 4.3 from the saved scores and the merged log-sum-exp
  const int e = p.order == ROCO_EVICT_FIRST ? p.slot_new[u] : -1;  // the slot whose statistics start from zero
#pragma unroll 4
  for (int j = tid; j < live; j += kSpMergeThreads) {
    const float pj = exp2f(p.zbuf[unit_st + j] - M) * inv;
    const bool fresh = (j == e);
    const float s0 = fresh ? 0.f : p.s[unit_st + j], q0 = fresh ? 0.f : p.q[unit_st + j];
    const int n0 = fresh ? 0 : p.n[unit_st + j];
    p.s[unit_st + j] = s0 + pj;
    p.q[unit_st + j] = fmaf(pj, pj, q0);
    p.n[unit_st + j] = n0 + 1;
  }
}

static size_t split_attend_smem(int B, int d) {
  return 128 + (size_t)kSpStages * kSpTile + align_up((size_t)B, 4) * 4 + (size_t)(1 + kSpConsumerWarps) * d * 4 +
         32 * 4 + 2 * kSpStages * 8 + 16;
}

size_t decode_split_workspace_bytes(int U, int B, int d, int splits) {
  return align_up((size_t)U * B * 4, 256) + align_up((size_t)U * splits * (2 + d) * 4, 256) + align_up((size_t)U * 4, 256);
}

template <typename T, int D>
static cudaError_t launch_split_t(SplitParams &p, int U, cudaStream_t stream) {
  const size_t smem1 = align_up((size_t)p.B, 4) * 8;
  const size_t smem2 = split_attend_smem(p.B, D);
  cudaError_t err = cudaFuncSetAttribute(split_policy_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem1);
  if (err == cudaSuccess)
    err = cudaFuncSetAttribute(split_attend_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2);
  if (err != cudaSuccess) return err;
  if (p.order == ROCO_EVICT_FIRST) split_policy_kernel<T, D><<<U, kSpPolicyThreads, smem1, stream>>>(p);
  split_attend_kernel<T, D><<<dim3(p.splits, U), kSpThreads, smem2, stream>>>(p);
  split_merge_kernel<T, D><<<U, kSpMergeThreads, 0, stream>>>(p);
  if (p.order != ROCO_EVICT_FIRST) split_policy_kernel<T, D><<<U, kSpPolicyThreads, smem1, stream>>>(p);
  return cudaGetLastError();
}

roco_status launch_decode_step_split(const roco_cache &c, const void *q, const void *k_new, const void *v_new, int r,
                                     int scope_mode, int step_order, int splits, float scale, void *out, float *lse,
                                     int32_t *ev_slot, int32_t *ev_pos, void *workspace, cudaStream_t stream) {
  SplitParams p;
  const int U = c.S * c.G;
  p.K = (const char *)c.K; p.V = (const char *)c.V;
  p.s = c.s; p.q = c.q; p.n = c.n; p.pos = c.pos; p.live = c.live; p.t_next = c.t_next; p.status = c.status;
  p.qv = (const char *)q; p.k_new = (const char *)k_new; p.v_new = (const char *)v_new;
  p.out = (char *)out; p.lse = lse; p.ev_slot = ev_slot; p.ev_pos = ev_pos;
  p.B = c.B; p.r = r; p.scope_mode = scope_mode; p.splits = splits; p.order = step_order; p.scale = scale;
  char *ws = (char *)workspace;
  p.zbuf = (float *)ws;
  ws += align_up((size_t)U * c.B * 4, 256);
  p.part = (float *)ws;
  ws += align_up((size_t)U * splits * (2 + c.d) * 4, 256);
  p.slot_new = (int *)ws;
  if (U > 65535) return ROCO_ERR_UNSUPPORTED;  // the unit index is the grid's y dimension
  cudaError_t err;
  if (c.kv_dtype == ROCO_BF16 && c.d == 128) err = launch_split_t<__nv_bfloat16, 128>(p, U, stream);
  else if (c.kv_dtype == ROCO_BF16 && c.d == 64) err = launch_split_t<__nv_bfloat16, 64>(p, U, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 128) err = launch_split_t<float, 128>(p, U, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 64) err = launch_split_t<float, 64>(p, U, stream);
  else return ROCO_ERR_UNSUPPORTED;
  return err == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
