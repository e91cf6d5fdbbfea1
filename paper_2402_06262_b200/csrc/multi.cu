// Multi-query steps over the budgeted cache: several queries share one pass over a unit's K and V blocks.
//   - block-wise evict-and-encode (Sec. 5.3 "Overhead", App. B): b new tokens per unit and step; b slots are
//     freed by the rule of Sec. 4.3 applied on frozen statistics, the new tokens take the freed / free slots in
//     increasing slot order, query i attends over the old survivors and the new tokens 0..i, and every attended
//     token gets Count += 1, Acc += p, Acc^square += p^2 per query;
//   - grouped-query attention (Sec. 5.3, App. A): `group` query heads share a key-value head; one new token;
//     the statistics receive the group mean of the probabilities.
// Same organisation as the single-query decode step (producer warp + TMA ring, eight consumer warps, four
// policy warps that select, insert and update the statistics while the consumers stream), with the M x B score
// matrix in shared memory.  Each consumer warp owns four queries and a share of every tile's rows, so the
// per-row arithmetic grows with M while the HBM traffic per unit stays that of one decode step.
#include <cuda.h>

#include "multi.cuh"

namespace roco {

struct MultiSmem {
  char *ring;
  float *z;  // [M][Bp] scores, then probabilities
  uint32_t *vkey;
  float *mkey;
  signed char *newtok;  // [Bp] index of the new token a slot holds, -1 for an old token
  SelectScratch *sel;
  float *qf;      // [M][D]
  float *knew;    // [nb][D]
  float *vnew;    // [nb][D]
  float *zn;      // [M][nb] scores of the queries against the new tokens
  float *outred;  // [8 warps][4][D]
  uint64_t *full, *empty, *p_ready, *policy_done;
  int *ctl;  // [0] abort flag, [1..16] target slots of the new tokens, [17] warp_tot scratch base
};

__host__ __device__ inline size_t multi_smem_bytes(int B, int d, int stages, int M, int nb) {
  const size_t Bp = align_up((size_t)B, 16);
  size_t b = (size_t)stages * kMqTile;
  b += (size_t)M * Bp * 4 + 2 * Bp * 4 + Bp;
  b += sizeof(SelectScratch);
  b += ((size_t)M + 2 * (size_t)nb) * d * 4 + (size_t)M * nb * 4;
  b += (size_t)kMqConsumerWarps * kMqQPW * d * 4;
  b = align_up(b, 8) + (2 * (size_t)stages + 2) * 8 + 64 * 4;
  return b + 128;
}

__device__ inline MultiSmem multi_carve(char *raw, int B, int d, int stages, int M, int nb) {
  MultiSmem m;
  char *p = smem_align(raw, 128);
  const size_t Bp = align_up((size_t)B, 16);
  m.ring = p; p += (size_t)stages * kMqTile;
  m.z = (float *)p; p += (size_t)M * Bp * 4;
  m.vkey = (uint32_t *)p; p += Bp * 4;
  m.mkey = (float *)p; p += Bp * 4;
  m.newtok = (signed char *)p; p += Bp;
  m.sel = (SelectScratch *)p; p += sizeof(SelectScratch);
  m.qf = (float *)p; p += (size_t)M * d * 4;
  m.knew = (float *)p; p += (size_t)nb * d * 4;
  m.vnew = (float *)p; p += (size_t)nb * d * 4;
  m.zn = (float *)p; p += (size_t)M * nb * 4;
  m.outred = (float *)p; p += (size_t)kMqConsumerWarps * kMqQPW * d * 4;
  p = smem_align(p, 8);
  m.full = (uint64_t *)p; p += stages * 8;
  m.empty = (uint64_t *)p; p += stages * 8;
  m.p_ready = (uint64_t *)p; p += 8;
  m.policy_done = (uint64_t *)p; p += 8;
  m.ctl = (int *)p;
  return m;
}

template <typename T, int D>
__global__ void __launch_bounds__(kMqThreads) multi_step_kernel(const MultiParams p) {
  constexpr int kRowBytes = D * (int)sizeof(T);
  constexpr int kLanesPerRow = kRowBytes / 16;
  constexpr int kRowsPerLoad = 32 / kLanesPerRow;
  constexpr int kTileRows = kMqTile / kRowBytes;
  constexpr int kEPC = Elem<T>::kPerChunk;

  extern __shared__ char mq_smem_raw[];
  const int M = p.M, nb = p.nb, B = p.B, stages = p.stages;
  const MultiSmem sm = multi_carve(mq_smem_raw, B, D, stages, M, nb);
  volatile int *abort_flag = sm.ctl;
  const size_t Bp = align_up((size_t)B, 16);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int u = blockIdx.x;
  const size_t unit_kv = (size_t)u * B * kRowBytes;

  if (tid == 0) {
    for (int i = 0; i < stages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], kMqConsumerWarps); }
    mbar_init(sm.p_ready, kMqConsumerWarps);
    mbar_init(sm.policy_done, 1);
    sm.ctl[0] = 0;
    mbar_init_fence();
  }
  int live0 = p.live[u];
  if (live0 < 0 || live0 > B) {
    if (tid == 0) atomicOr(p.status, ROCO_DEV_BAD_LIVE);
    live0 = live0 < 0 ? 0 : B;
  }
  int need = live0 + nb - B;  // tokens that have to leave
  if (need < 0) need = 0;
  const int live1 = live0 - need + nb;  // occupied slots after the insertion = slots every query streams over
  const int n_tiles = (live1 + kTileRows - 1) / kTileRows;
  __syncthreads();

  if (warp == kMqProducerWarp) {
    if (lane == 0) {
      for (int g = 0; g < 2 * n_tiles; ++g) {
        const int st = g % stages;
        if (g >= stages) mbar_wait(&sm.empty[st], ((g / stages) - 1) & 1, abort_flag, p.status);
        const int it = (g < n_tiles) ? g : g - n_tiles;
        const char *src = ((g < n_tiles) ? p.K : p.V) + unit_kv + (size_t)it * kMqTile;
        int rows = live1 - it * kTileRows;
        if (rows > kTileRows) rows = kTileRows;
        const uint32_t bytes = (uint32_t)rows * kRowBytes;
        mbar_expect_tx(&sm.full[st], bytes);
        bulk_g2s(sm.ring + (size_t)st * kMqTile, src, bytes, &sm.full[st]);
      }
    }
    return;
  }

  if (warp >= kMqPolicyWarp0) {
    // ---------------------------------------------------------- policy: free slots, insert, statistics
    PolicyView v;
    v.z = sm.z; v.Bp = Bp; v.vkey = sm.vkey; v.mkey = sm.mkey; v.newtok = sm.newtok; v.sel = sm.sel;
    v.knew = sm.knew; v.vnew = sm.vnew; v.zn = sm.zn; v.qf = nullptr; v.pn = nullptr; v.ctl = sm.ctl;
    v.nbuf = nullptr; v.posbuf = nullptr; v.stats_full = nullptr; v.zn_by_consumers = false;
    v.p_ready = sm.p_ready;
    v.policy_done = sm.policy_done;
    multi_policy<T, D>(p, v, u, tid - kMqPolicyWarp0 * 32, live0, need, live1);
    return;
  }

  // -------------------------------------------------------------- consumers
  const int QG = M <= 4 ? 1 : (M <= 8 ? 2 : 4);  // query groups of four
  const int RG = kMqConsumerWarps / QG;          // row groups
  const int qg = warp % QG, rg = warp / QG;
  const int rows_per_warp = kTileRows / RG;
  const int loads = rows_per_warp / kRowsPerLoad;
  for (int i = tid; i < M * D; i += kMqConsumers)
    sm.qf[i] = Elem<T>::load((const T *)p.Q + (size_t)u * p.q_ustride * D + i);
  named_bar_sync(kMqBarConsumers, kMqConsumers);

  const float zscale = p.scale * kLog2e;
  const int lane_chunk = lane % kLanesPerRow, lane_row = lane / kLanesPerRow;
  float qreg[kMqQPW][kEPC];
#pragma unroll
  for (int i = 0; i < kMqQPW; ++i) {
    const int qi = qg * kMqQPW + i;
#pragma unroll
    for (int e = 0; e < kEPC; ++e) qreg[i][e] = qi < M ? sm.qf[qi * D + lane_chunk * kEPC + e] : 0.f;
  }

  // ---- scores of four queries per warp: z_i[j] = scale * q_i.K[j]  (Eq. 1), log2 domain
  for (int it = 0; it < n_tiles; ++it) {
    const int st = it % stages;
    mbar_wait(&sm.full[st], (it / stages) & 1, abort_flag, p.status);
    const char *tile = sm.ring + (size_t)st * kMqTile;
    for (int l = 0; l < loads; ++l) {
      const int row = rg * rows_per_warp + l * kRowsPerLoad + lane_row;
      const uint4 c = *(const uint4 *)(tile + (size_t)row * kRowBytes + lane_chunk * 16);
      float f[kEPC];
      Elem<T>::unpack(c, f);
      float acc[kMqQPW];
#pragma unroll
      for (int i = 0; i < kMqQPW; ++i) {
        acc[i] = 0.f;
#pragma unroll
        for (int e = 0; e < kEPC; ++e) acc[i] = fmaf(f[e], qreg[i][e], acc[i]);
      }
#pragma unroll
      for (int o = kLanesPerRow / 2; o > 0; o >>= 1) {  // one butterfly for the four queries together
#pragma unroll
        for (int i = 0; i < kMqQPW; ++i) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
      }
      const int j = it * kTileRows + row;
      if (lane_chunk < kMqQPW && j < live1) {
        const int qi = qg * kMqQPW + lane_chunk;
        float v = acc[0];
        if (lane_chunk == 1) v = acc[1];
        if (lane_chunk == 2) v = acc[2];
        if (lane_chunk == 3) v = acc[3];
        if (qi < M) sm.z[(size_t)qi * Bp + j] = v * zscale;
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[st]);
  }

  // the slots the policy warps have filled hold the new tokens: their scores come from k_new, with the causal
  // mask inside a block (query i does not see the tokens after it)
  mbar_wait(sm.policy_done, 0, abort_flag, p.status);
  named_bar_sync(kMqBarConsumers, kMqConsumers);
  for (int w = tid; w < M * nb; w += kMqConsumers) {
    const int i = w / nb, jn = w % nb;
    int slot = sm.ctl[1 + jn];
    if (slot < 0 || slot >= B) slot = 0;
    sm.z[(size_t)i * Bp + slot] = (jn > i / p.group) ? -INFINITY : sm.zn[w];
  }
  named_bar_sync(kMqBarConsumers, kMqConsumers);

  // ---- one softmax per query, each by one warp
  for (int i = warp; i < M; i += kMqConsumerWarps) {
    float *zi = sm.z + (size_t)i * Bp;
    float zmax = -INFINITY;
    for (int j = lane; j < live1; j += 32) zmax = fmaxf(zmax, zi[j]);
    zmax = warp_max(zmax);
    float zsum = 0.f;
    for (int j = lane; j < live1; j += 32) {
      const float ex = exp2f(zi[j] - zmax);
      zi[j] = ex;
      zsum += ex;
    }
    zsum = warp_sum(zsum);
    const float inv = 1.f / zsum;
    for (int j = lane; j < live1; j += 32) zi[j] *= inv;
    if (lane == 0 && p.lse) p.lse[(size_t)u * M + i] = (zmax + log2f(zsum)) * kLn2;
  }
  __syncwarp();
  if (lane == 0) mbar_arrive(sm.p_ready);
  named_bar_sync(kMqBarConsumers, kMqConsumers);

  // ---- out_i = sum_j p_i[j] V[j]; the new tokens' values come from v_new at the end
  float oacc[kMqQPW][kEPC];
#pragma unroll
  for (int i = 0; i < kMqQPW; ++i)
#pragma unroll
    for (int e = 0; e < kEPC; ++e) oacc[i][e] = 0.f;
  for (int it = 0; it < n_tiles; ++it) {
    const int g = n_tiles + it;
    const int st = g % stages;
    mbar_wait(&sm.full[st], (g / stages) & 1, abort_flag, p.status);
    const char *tile = sm.ring + (size_t)st * kMqTile;
    for (int l = 0; l < loads; ++l) {
      const int row = rg * rows_per_warp + l * kRowsPerLoad + lane_row;
      const int j = it * kTileRows + row;
      if (j < live1 && sm.newtok[j] < 0) {
        const uint4 c = *(const uint4 *)(tile + (size_t)row * kRowBytes + lane_chunk * 16);
        float f[kEPC];
        Elem<T>::unpack(c, f);
#pragma unroll
        for (int i = 0; i < kMqQPW; ++i) {
          const int qi = qg * kMqQPW + i;
          const float pj = qi < M ? sm.z[(size_t)qi * Bp + j] : 0.f;
#pragma unroll
          for (int e = 0; e < kEPC; ++e) oacc[i][e] = fmaf(pj, f[e], oacc[i][e]);
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[st]);
  }
#pragma unroll
  for (int i = 0; i < kMqQPW; ++i)
#pragma unroll
    for (int e = 0; e < kEPC; ++e) {
#pragma unroll
      for (int o = kLanesPerRow; o < 32; o <<= 1) oacc[i][e] += __shfl_xor_sync(0xffffffffu, oacc[i][e], o);
    }
  if (lane_row == 0) {
#pragma unroll
    for (int i = 0; i < kMqQPW; ++i)
#pragma unroll
      for (int e = 0; e < kEPC; ++e) sm.outred[((size_t)warp * kMqQPW + i) * D + lane_chunk * kEPC + e] = oacc[i][e];
  }
  named_bar_sync(kMqBarConsumers, kMqConsumers);
  for (int w = tid; w < M * D; w += kMqConsumers) {
    const int qi = w / D, c = w % D;
    float o = 0.f;
    for (int r2 = 0; r2 < RG; ++r2) o += sm.outred[((size_t)(r2 * QG + qi / kMqQPW) * kMqQPW + qi % kMqQPW) * D + c];
    for (int jn = 0; jn < nb; ++jn) {
      int slot = sm.ctl[1 + jn];
      if (slot < 0 || slot >= B) slot = 0;
      o = fmaf(sm.z[(size_t)qi * Bp + slot], sm.vnew[jn * D + c], o);
    }
    Elem<T>::store((T *)p.out + (size_t)u * p.out_ustride * D + w, o);
  }
}

// ------------------------------------------------------------------------------------------------------------
// Tensor-core variant (bf16, d = 128): the M x 64 score block of a tile is one row of warp-level MMAs
// (m16n8k16, queries on the M axis, padded to 16), and so is the 16 x 128 output update, which takes the per-row
// arithmetic off the CUDA cores: the step stays HBM-bound for any M <= 16.  Tiles arrive through TMA tensor maps
// with the 128-byte swizzle so that ldmatrix reads them without bank conflicts.

struct MultiTcSmem {
  char *ring;  // 1024-byte aligned, `stages` tiles of 64 rows x 128 bf16 (two 64-column halves of 8 KiB)
  float *z;    // [M][Bp], Bp = multi_tc_row_stride(B)
  uint32_t *vkey;
  float *mkey;
  signed char *newtok;
  SelectScratch *sel;
  int *nbuf;   // [Bp] Count array of the unit (s and q are staged in vkey and mkey)
  int *posbuf; // [Bp] positions of the unit before the step
  float *vnew, *zn, *pn;
  uint64_t *full, *empty, *p_ready, *policy_done, *stats_full;
  int *ctl;
};

// Row stride of the score matrix: the budget rounded up to a tile, plus 8 floats so that the eight query rows a
// warp touches at once (MMA fragment rows) fall into different shared-memory banks.
__host__ __device__ inline size_t multi_tc_row_stride(int B) { return align_up((size_t)B, 64) + 8; }

__host__ __device__ inline size_t multi_tc_smem_bytes(int B, int stages, int M, int nb) {
  const size_t Bp = multi_tc_row_stride(B);
  size_t b = (size_t)stages * kMqTile;
  b += (size_t)M * Bp * 4 + 4 * Bp * 4 + Bp;
  b += sizeof(SelectScratch);
  b += (size_t)nb * 128 * 4 + 2 * (size_t)M * nb * 4;
  b = align_up(b, 8) + (2 * (size_t)stages + 3) * 8 + 64 * 4;
  return b + 1024;
}

__device__ inline MultiTcSmem multi_tc_carve(char *raw, int B, int stages, int M, int nb) {
  MultiTcSmem m;
  char *p = smem_align(raw, 1024);
  const size_t Bp = multi_tc_row_stride(B);
  m.ring = p; p += (size_t)stages * kMqTile;
  m.z = (float *)p; p += (size_t)M * Bp * 4;
  m.vkey = (uint32_t *)p; p += Bp * 4;
  m.mkey = (float *)p; p += Bp * 4;
  m.nbuf = (int *)p; p += Bp * 4;
  m.posbuf = (int *)p; p += Bp * 4;
  m.newtok = (signed char *)p; p += Bp;
  m.sel = (SelectScratch *)p; p += sizeof(SelectScratch);
  m.vnew = (float *)p; p += (size_t)nb * 128 * 4;
  m.zn = (float *)p; p += (size_t)M * nb * 4;
  m.pn = (float *)p; p += (size_t)M * nb * 4;
  p = smem_align(p, 8);
  m.full = (uint64_t *)p; p += stages * 8;
  m.empty = (uint64_t *)p; p += stages * 8;
  m.p_ready = (uint64_t *)p; p += 8;
  m.policy_done = (uint64_t *)p; p += 8;
  m.stats_full = (uint64_t *)p; p += 8;
  m.ctl = (int *)p;
  return m;
}

__global__ void __launch_bounds__(kMqThreads) multi_step_tc_kernel(const __grid_constant__ CUtensorMap mapK,
                                                                   const __grid_constant__ CUtensorMap mapV,
                                                                   const MultiParams p) {
  using T = __nv_bfloat16;
  constexpr int D = 128, kTileRows = 64;
  extern __shared__ char mq_smem_raw[];
  const int M = p.M, nb = p.nb, B = p.B, stages = p.stages;
  const MultiTcSmem sm = multi_tc_carve(mq_smem_raw, B, stages, M, nb);
  volatile int *abort_flag = sm.ctl;
  const size_t Bp = multi_tc_row_stride(B);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int u = blockIdx.x;

  if (tid == 0) {
    for (int i = 0; i < stages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], kMqConsumerWarps); }
    mbar_init(sm.p_ready, kMqConsumerWarps);
    mbar_init(sm.policy_done, 1);
    mbar_init(sm.stats_full, 1);
    sm.ctl[0] = 0;
    mbar_init_fence();
  }
  int live0 = p.live[u];
  if (live0 < 0 || live0 > B) {
    if (tid == 0) atomicOr(p.status, ROCO_DEV_BAD_LIVE);
    live0 = live0 < 0 ? 0 : B;
  }
  int need = live0 + nb - B;
  if (need < 0) need = 0;
  const int live1 = live0 - need + nb;
  const int n_tiles = (live1 + kTileRows - 1) / kTileRows;
  // The statistics the selection reads come in by bulk copy ahead of the K tiles (plain loads would queue behind
  // the tile stream); needs 16-byte aligned unit offsets, i.e. B a multiple of 4 and aligned arrays.
  const bool stats_by_tma =
      need > 0 && (B & 3) == 0 &&
      ((reinterpret_cast<uintptr_t>(p.s) | reinterpret_cast<uintptr_t>(p.q) | reinterpret_cast<uintptr_t>(p.n) |
        reinterpret_cast<uintptr_t>(p.pos)) & 15) == 0;
  __syncthreads();

  if (warp == kMqProducerWarp) {
    if (lane == 0) {
      if (stats_by_tma) {
        const uint32_t bytes = (uint32_t)align_up((size_t)live0 * 4, 16);  // B % 4 == 0: stays inside the unit
        mbar_expect_tx(sm.stats_full, 4 * bytes);
        bulk_g2s(sm.vkey, p.s + (size_t)u * B, bytes, sm.stats_full);
        bulk_g2s(sm.mkey, p.q + (size_t)u * B, bytes, sm.stats_full);
        bulk_g2s(sm.nbuf, p.n + (size_t)u * B, bytes, sm.stats_full);
        bulk_g2s(sm.posbuf, p.pos + (size_t)u * B, bytes, sm.stats_full);
      }
      for (int g = 0; g < 2 * n_tiles; ++g) {
        const int st = g % stages;
        if (g >= stages) mbar_wait(&sm.empty[st], ((g / stages) - 1) & 1, abort_flag, p.status);
        const int it = (g < n_tiles) ? g : g - n_tiles;
        const CUtensorMap *map = (g < n_tiles) ? &mapK : &mapV;
        char *dst = sm.ring + (size_t)st * kMqTile;
        const int row = u * B + it * kTileRows;
        mbar_expect_tx(&sm.full[st], kMqTile);
        tma_load_2d(dst, map, 0, row, &sm.full[st]);
        tma_load_2d(dst + 8192, map, 64, row, &sm.full[st]);
      }
    }
    return;
  }

  if (warp >= kMqPolicyWarp0) {
    PolicyView v;
    v.z = sm.z; v.Bp = Bp; v.vkey = sm.vkey; v.mkey = sm.mkey; v.newtok = sm.newtok; v.sel = sm.sel;
    v.knew = nullptr; v.vnew = sm.vnew; v.zn = sm.zn; v.qf = nullptr; v.pn = sm.pn; v.ctl = sm.ctl;
    v.nbuf = sm.nbuf; v.posbuf = sm.posbuf; v.stats_full = stats_by_tma ? sm.stats_full : nullptr;
    v.zn_by_consumers = true;
    v.p_ready = sm.p_ready;
    v.policy_done = sm.policy_done;
    multi_policy<T, D>(p, v, u, tid - kMqPolicyWarp0 * 32, live0, need, live1);
    return;
  }

  // -------------------------------------------------------------- consumers
  const float zscale = p.scale * kLog2e;
  const int g = lane >> 2, tq = lane & 3;
  const bool row_lo = g < M, row_hi = g + 8 < M;
  // A fragments of Q (16 x 128, rows >= M are zero): a[s] covers k = 16 s .. 16 s + 15
  uint32_t qa[8][4];
  {
    const T *Qu = (const T *)p.Q + (size_t)u * p.q_ustride * D;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      const int k0 = s * 16 + tq * 2;
      qa[s][0] = row_lo ? *reinterpret_cast<const uint32_t *>(Qu + (size_t)g * D + k0) : 0u;
      qa[s][1] = row_hi ? *reinterpret_cast<const uint32_t *>(Qu + (size_t)(g + 8) * D + k0) : 0u;
      qa[s][2] = row_lo ? *reinterpret_cast<const uint32_t *>(Qu + (size_t)g * D + k0 + 8) : 0u;
      qa[s][3] = row_hi ? *reinterpret_cast<const uint32_t *>(Qu + (size_t)(g + 8) * D + k0 + 8) : 0u;
    }
  }

  // ---- scores: each warp takes 8 keys of every 64-key tile, all queries:  Z[16 x 8] = Q[16 x 128] K^T
  for (int it = 0; it < n_tiles; ++it) {
    const int st = it % stages;
    mbar_wait(&sm.full[st], (it / stages) & 1, abort_flag, p.status);
    const uint32_t tile = smem_u32(sm.ring + (size_t)st * kMqTile);
    float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int sp = 0; sp < 4; ++sp) {
      uint32_t kb[4];
      ldmatrix_x4(tile + tile_chunk_offset(warp * 8 + (lane & 7), sp * 4 + (lane >> 3)), kb);
      mma_bf16_16816(c, qa[2 * sp], kb[0], kb[1]);
      mma_bf16_16816(c, qa[2 * sp + 1], kb[2], kb[3]);
    }
    const int j = it * kTileRows + warp * 8 + tq * 2;
    if (row_lo) {
      if (j < live1) sm.z[(size_t)g * Bp + j] = c[0] * zscale;
      if (j + 1 < live1) sm.z[(size_t)g * Bp + j + 1] = c[1] * zscale;
    }
    if (row_hi) {
      if (j < live1) sm.z[(size_t)(g + 8) * Bp + j] = c[2] * zscale;
      if (j + 1 < live1) sm.z[(size_t)(g + 8) * Bp + j + 1] = c[3] * zscale;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[st]);
  }

  // scores of the queries against the new tokens, from k_new: Zn[16 x 8] per warp, one warp per 8 new tokens
  if (warp * 8 < nb) {
    const T *Kn = (const T *)p.k_new + (size_t)u * p.kv_ustride * D;
    const int jn = warp * 8 + g;  // the new token whose key this thread holds fragments of
    float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      const int k0 = s * 16 + tq * 2;
      const uint32_t b0 = jn < nb ? *reinterpret_cast<const uint32_t *>(Kn + (size_t)jn * D + k0) : 0u;
      const uint32_t b1 = jn < nb ? *reinterpret_cast<const uint32_t *>(Kn + (size_t)jn * D + k0 + 8) : 0u;
      mma_bf16_16816(c, qa[s], b0, b1);
    }
    const int j0 = warp * 8 + tq * 2;
    if (row_lo) {
      if (j0 < nb) sm.zn[g * nb + j0] = c[0] * zscale;
      if (j0 + 1 < nb) sm.zn[g * nb + j0 + 1] = c[1] * zscale;
    }
    if (row_hi) {
      if (j0 < nb) sm.zn[(g + 8) * nb + j0] = c[2] * zscale;
      if (j0 + 1 < nb) sm.zn[(g + 8) * nb + j0 + 1] = c[3] * zscale;
    }
  }
  // ... placed into the score matrix with the causal mask inside a block, once the target slots are known
  mbar_wait(sm.policy_done, 0, abort_flag, p.status);
  named_bar_sync(kMqBarConsumers, kMqConsumers);
  for (int w = tid; w < M * nb; w += kMqConsumers) {
    const int i = w / nb, jn = w % nb;
    int slot = sm.ctl[1 + jn];
    if (slot < 0 || slot >= B) slot = 0;
    sm.z[(size_t)i * Bp + slot] = (jn > i / p.group) ? -INFINITY : sm.zn[w];
  }
  named_bar_sync(kMqBarConsumers, kMqConsumers);

  // ---- one softmax per query, each by one warp; the tail of the last tile is cleared for the MMAs below
  for (int i = warp; i < M; i += kMqConsumerWarps) {
    float *zi = sm.z + (size_t)i * Bp;
    float zmax = -INFINITY;
    for (int j = lane; j < live1; j += 32) zmax = fmaxf(zmax, zi[j]);
    zmax = warp_max(zmax);
    float zsum = 0.f;
    for (int j = lane; j < live1; j += 32) {
      const float ex = exp2f(zi[j] - zmax);
      zi[j] = ex;
      zsum += ex;
    }
    zsum = warp_sum(zsum);
    const float inv = 1.f / zsum;
    for (int j = lane; j < live1; j += 32) zi[j] *= inv;
    for (int j = live1 + lane; j < n_tiles * kTileRows; j += 32) zi[j] = 0.f;
    if (lane == 0 && p.lse) p.lse[(size_t)u * M + i] = (zmax + log2f(zsum)) * kLn2;
  }
  named_bar_sync(kMqBarConsumers, kMqConsumers);
  // the new tokens' values come from v_new: keep their probabilities aside and clear them in z, so that the
  // streamed V rows of those slots (possibly read before the overwrite) contribute nothing
  for (int w = tid; w < M * nb; w += kMqConsumers) {
    const int i = w / nb, jn = w % nb;
    int slot = sm.ctl[1 + jn];
    if (slot < 0 || slot >= B) slot = 0;
    sm.pn[w] = sm.z[(size_t)i * Bp + slot];
    sm.z[(size_t)i * Bp + slot] = 0.f;
  }
  __syncwarp();
  if (lane == 0) mbar_arrive(sm.p_ready);
  named_bar_sync(kMqBarConsumers, kMqConsumers);

  // ---- out[16 x 128] += P[16 x 64] V[64 x 128]: each warp owns 16 output columns
  float o[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
  for (int it = 0; it < n_tiles; ++it) {
    const int gg = n_tiles + it;
    const int st = gg % stages;
    mbar_wait(&sm.full[st], (gg / stages) & 1, abort_flag, p.status);
    const uint32_t tile = smem_u32(sm.ring + (size_t)st * kMqTile);
    // slots >= live0 were free before this step: whatever the stream brought for them (they may hold anything,
    // NaN included, and 0 * NaN would poison the MMA) is cleared in the 16 columns this warp reads
    if ((it + 1) * kTileRows > live0) {
      const int r0 = live0 > it * kTileRows ? live0 - it * kTileRows : 0;
      char *tp = sm.ring + (size_t)st * kMqTile;
      for (int w = lane; w < (kTileRows - r0) * 2; w += 32) {
        const int row = r0 + (w >> 1);
        *reinterpret_cast<uint4 *>(tp + tile_chunk_offset(row, warp * 2 + (w & 1))) = make_uint4(0u, 0u, 0u, 0u);
      }
      __syncwarp();
    }
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      const int j = it * kTileRows + ks * 16 + tq * 2;
      uint32_t pa[4];
      const float *zl = sm.z + (size_t)g * Bp + j, *zh = sm.z + (size_t)(g + 8) * Bp + j;
      pa[0] = row_lo ? pack_bf16x2(zl[0], zl[1]) : 0u;
      pa[1] = row_hi ? pack_bf16x2(zh[0], zh[1]) : 0u;
      pa[2] = row_lo ? pack_bf16x2(zl[8], zl[9]) : 0u;
      pa[3] = row_hi ? pack_bf16x2(zh[8], zh[9]) : 0u;
      uint32_t vb[4];
      const int mi = lane >> 3;
      ldmatrix_x4_trans(tile + tile_chunk_offset(ks * 16 + (mi & 1) * 8 + (lane & 7), warp * 2 + (mi >> 1)), vb);
      mma_bf16_16816(o[0], pa, vb[0], vb[1]);
      mma_bf16_16816(o[1], pa, vb[2], vb[3]);
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[st]);
  }
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    const int dcol = warp * 16 + nt * 8 + tq * 2;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int qi = g + 8 * h;
      if (qi < M) {
        float o0 = o[nt][2 * h], o1 = o[nt][2 * h + 1];
        for (int jn = 0; jn < nb; ++jn) {
          const float pj = sm.pn[qi * nb + jn];
          o0 = fmaf(pj, sm.vnew[jn * D + dcol], o0);
          o1 = fmaf(pj, sm.vnew[jn * D + dcol + 1], o1);
        }
        *reinterpret_cast<uint32_t *>((T *)p.out + ((size_t)u * p.out_ustride + qi) * D + dcol) = pack_bf16x2(o0, o1);
      }
    }
  }
}

static int multi_tc_pick_stages(int B, int M, int nb) {
  const size_t per_sm = 227 * 1024;
  for (int ctas = 2; ctas >= 1; --ctas)
    for (int st = 6; st >= 3; --st)
      if ((multi_tc_smem_bytes(B, st, M, nb) + 1024) * ctas <= per_sm) return st;
  return 0;
}

static int multi_pick_stages(int B, int d, int M, int nb) {
  const size_t per_sm = 227 * 1024;
  for (int ctas = 2; ctas >= 1; --ctas)
    for (int st = 5; st >= 3; --st)
      if ((multi_smem_bytes(B, d, st, M, nb) + 1024) * ctas <= per_sm) return st;
  return 0;
}

template <typename T, int D>
static cudaError_t launch_multi_t(MultiParams &p, int U, cudaStream_t stream) {
  const size_t smem = multi_smem_bytes(p.B, D, p.stages, p.M, p.nb);
  cudaError_t err = cudaFuncSetAttribute(multi_step_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  multi_step_kernel<T, D><<<U, kMqThreads, smem, stream>>>(p);
  return cudaGetLastError();
}

int multi_max_queries() { return kMqMaxQ; }

bool multi_fits(int B, int d, int M, int nb) {
  return multi_pick_stages(B, d, M, nb) > 0 || (d == 128 && multi_tc_pick_stages(B, M, nb) > 0) ||
         (d == 128 && multi_um_rows(M, nb) && multi_um_pick_stages(B, nb) > 0);
}

roco_status launch_multi_step(const roco_cache &c, int M, int nb, const void *Q, const void *k_new,
                              const void *v_new, int r, int scope_mode, float scale, void *out, float *lse,
                              int32_t *ev_slot, int32_t *ev_pos, cudaStream_t stream, long long unit_stride_rows) {
  MultiParams p;
  p.K = (const char *)c.K; p.V = (const char *)c.V;
  p.s = c.s; p.q = c.q; p.n = c.n; p.pos = c.pos; p.live = c.live; p.t_next = c.t_next; p.status = c.status;
  p.Q = (const char *)Q; p.k_new = (const char *)k_new; p.v_new = (const char *)v_new;
  p.out = (char *)out; p.lse = lse; p.ev_slot = ev_slot; p.ev_pos = ev_pos;
  p.B = c.B; p.r = r; p.scope_mode = scope_mode; p.M = M; p.nb = nb; p.scale = scale;
  p.group = M / nb;
  p.q_ustride = unit_stride_rows > 0 ? unit_stride_rows * p.group : M;
  p.kv_ustride = unit_stride_rows > 0 ? unit_stride_rows : nb;
  p.out_ustride = unit_stride_rows > 0 ? unit_stride_rows * p.group : M;
  const int U = c.S * c.G;
  cudaError_t err;
  if (c.kv_dtype == ROCO_BF16 && c.d == 128 && (long long)U * c.B < 0x7fffffffLL) {
    // tensor-core path; falls through to the CUDA-core path if the tensor maps cannot be built
    CUtensorMap mapK, mapV;
    // (the tcgen05 kernel takes its row maxima on the raw scores and masks with -inf before scaling: right only
    // for a positive scale)
    const int um_stages = (multi_um_rows(M, nb) && scale > 0.f) ? multi_um_pick_stages(c.B, nb) : 0;
    // with one CTA per SM either way, the tcgen05 kernel keeps more bytes in flight; with two of the warp-level
    // kernel against one of this, the two win
    const bool tc_two = (multi_tc_smem_bytes(c.B, 3, M, nb) + 1024) * 2 <= (size_t)227 * 1024;
    if (um_stages > 0 && (um_stages == 2 || !tc_two)) {
      p.stages = um_stages;
      const int rc = launch_multi_step_umma(p, c, U, stream);
      if (rc >= 0) return static_cast<roco_status>(rc);
    }
    p.stages = multi_tc_pick_stages(c.B, M, nb);
    if (p.stages > 0 && make_tensor_map_rows128_bf16(&mapK, c.K, (unsigned long long)U * c.B, 64) &&
        make_tensor_map_rows128_bf16(&mapV, c.V, (unsigned long long)U * c.B, 64)) {
      const size_t smem = multi_tc_smem_bytes(c.B, p.stages, M, nb);
      err = cudaFuncSetAttribute(multi_step_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (err != cudaSuccess) return ROCO_ERR_CUDA;
      multi_step_tc_kernel<<<U, kMqThreads, smem, stream>>>(mapK, mapV, p);
      return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
    }
  }
  p.stages = multi_pick_stages(c.B, c.d, M, nb);
  if (p.stages == 0) return ROCO_ERR_UNSUPPORTED;
  if (c.kv_dtype == ROCO_BF16 && c.d == 128) err = launch_multi_t<__nv_bfloat16, 128>(p, U, stream);
  else if (c.kv_dtype == ROCO_BF16 && c.d == 64) err = launch_multi_t<__nv_bfloat16, 64>(p, U, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 128) err = launch_multi_t<float, 128>(p, U, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 64) err = launch_multi_t<float, 64>(p, U, stream);
  else return ROCO_ERR_UNSUPPORTED;
  return err == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
