// Multi-query steps on tcgen05 (see multi.cu for what a step computes and multi.cuh for the policy warps' part).
#include "multi.cuh"

namespace roco {

// tcgen05 variant for up to 16 queries (bf16, d = 128): both contractions of the step run on the fifth-generation
// tensor cores, issued by one thread, with the key index on the accumulator's lanes:
//
//   scores   S^T[128 keys x 16 queries] = K_tile[128 x 128] Q^T        (A: streamed tile, B: the queries, K-major)
//   output   O^T[128 dims x 16 queries] += V_tile^T[128 x 16 keys] P^T (A: streamed tile, B: probabilities, both
//                                                                       with the M / N index contiguous)
//
// A consumer thread then owns one key of a tile with its 16 scores side by side in the columns of its
// tensor-memory lane: the softmax works on them in place (the row maxima and sums are sums over lanes: one
// transposing shuffle reduction per pass), the per-slot sums over the queries of p and p^2 that the statistics
// need (Sec. 4.3) are sums inside a thread, and the 16 probabilities of a key are 32 contiguous bytes of the
// operand P^T.  The consumer warps issue no MMA, no matrix load and no per-tile barrier; what they execute per
// score is one maximum, two fused multiply-adds, two exponentials, the two statistics sums and half a conversion.
// The new tokens' values enter through one more MMA (V_new as a 16-key tile), their scores through a small
// warp-level MMA as before.

constexpr int kUmTile = 128;                    // keys per streamed tile
constexpr int kUmTileBytes = kUmTile * 256;     // two 64-column halves of 16 KiB
constexpr int kUmHalfBytes = kUmTileBytes / 2;
constexpr int kUmMmaWarp = kMqPolicyWarp0 + kMqPolicyThreads / 32;
constexpr int kUmThreads = (kUmMmaWarp + 1) * 32;
constexpr int kUmBarStaged = 3;                 // consumers + MMA warp: the query operand is in shared memory
constexpr int kUmBarDone = 4;                   // consumers + policy warps: nobody reads tensor memory any more
constexpr int kUmMaxTiles = 32;                 // 16 tensor-memory columns each
constexpr int kUmCtlStaleMax = 60;              // ctl word: a replaced slot held a row's maximum
constexpr int kUmPBlock = 16384;                // P^T of four tiles: 128 key rows of 128 bytes (4 x 16 queries)
// kind::f16 instruction descriptors: fp32 accumulator, bf16 operands, M = 128, N = 16
constexpr uint32_t kIdescUmS = (1u << 4) | (1u << 7) | (1u << 10) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescUmO = kIdescUmS | (1u << 15) | (1u << 16);  // A and B with the M / N index contiguous

struct MultiUmSmem {
  char *ring;
  char *pbuf;  // P^T blocks; until the selection is done its first 16 Bp bytes hold vkey | mkey | nbuf | posbuf
  uint32_t *vkey;
  float *mkey;
  int *nbuf, *posbuf;
  char *qv;    // 4 KiB: the queries (B operand of the score MMAs), afterwards V_new (A operand of the last MMA)
  char *pn;    // 2 KiB: P^T of the new tokens, 16 key rows of 128 bytes
  signed char *newtok;
  SelectScratch *sel;
  float *zn;   // [nb][16] raw scores of the queries (second index) against the new tokens
  float *red;  // [2][8 warps][16 queries], then [2][16]: row maxima of zn from the two warps that form it
  uint64_t *full, *empty, *s_full, *p_tile, *p_free, *d_ready, *o_full, *policy_done, *stats_full;
  uint32_t *tmem_base;
  int *ctl;
};

// The P^T buffer holds up to eight tiles' blocks (32 KiB) and is reused as a ring beyond that: a block is free again
// once the output MMAs of its tile have completed.  Until the selection is done the same memory holds the staged
// s, q, n and pos (16 bytes per slot), which sets its size for budgets above 2048.
__host__ __device__ inline size_t multi_um_pbuf_bytes(int B) {
  const size_t tiles = ((size_t)B + kUmTile - 1) / kUmTile;
  const size_t all = (tiles + 3) / 4 * kUmPBlock, ring = all < 2 * (size_t)kUmPBlock ? all : 2 * (size_t)kUmPBlock;
  const size_t stats = align_up(16 * align_up((size_t)B, 64), kUmPBlock);
  return ring > stats ? ring : stats;
}
// tiles of P^T in flight at once: four or eight (a power of two, so that a tile's place is a mask of its index)
__host__ __device__ inline int multi_um_ptiles(int B) { return B <= 4 * kUmTile ? 4 : 8; }

__host__ __device__ inline size_t multi_um_smem_bytes(int B, int stages, int nb) {
  const size_t Bp = align_up((size_t)B, 64);
  size_t b = (size_t)stages * kUmTileBytes + multi_um_pbuf_bytes(B) + 4096 + 2048;
  b += Bp + sizeof(SelectScratch);
  b = align_up(b, 16) + (size_t)16 * nb * 4 + (2 * kMqConsumerWarps + 2) * 16 * 4;
  b = align_up(b, 8) + (2 * (size_t)stages + 6 + 2 * kUmMaxTiles) * 8 + 64 * 4;
  return b + 1024;
}

__device__ inline MultiUmSmem multi_um_carve(char *raw, int B, int stages, int nb) {
  MultiUmSmem m;
  char *p = smem_align(raw, 1024);
  const size_t Bp = align_up((size_t)B, 64);
  m.ring = p; p += (size_t)stages * kUmTileBytes;
  m.pbuf = p;
  m.vkey = (uint32_t *)p;
  m.mkey = (float *)(p + 4 * Bp);
  m.nbuf = (int *)(p + 8 * Bp);
  m.posbuf = (int *)(p + 12 * Bp);
  p += multi_um_pbuf_bytes(B);
  m.qv = p; p += 4096;
  m.pn = p; p += 2048;
  m.newtok = (signed char *)p; p += Bp;
  m.sel = (SelectScratch *)p; p += sizeof(SelectScratch);
  p = smem_align(p, 16);
  m.zn = (float *)p; p += (size_t)16 * nb * 4;
  m.red = (float *)p; p += (2 * kMqConsumerWarps + 2) * 16 * 4;
  p = smem_align(p, 8);
  m.full = (uint64_t *)p; p += stages * 8;
  m.empty = (uint64_t *)p; p += stages * 8;
  m.s_full = (uint64_t *)p; p += 8;
  m.p_tile = (uint64_t *)p; p += kUmMaxTiles * 8;
  m.p_free = (uint64_t *)p; p += kUmMaxTiles * 8;
  m.d_ready = (uint64_t *)p; p += 8;
  m.o_full = (uint64_t *)p; p += 8;
  m.policy_done = (uint64_t *)p; p += 8;
  m.stats_full = (uint64_t *)p; p += 8;
  m.tmem_base = (uint32_t *)p; p += 8;
  m.ctl = (int *)p;
  return m;
}

// Tensor-memory columns of one CTA: 16 per tile of 128 keys and 16 for the output accumulator behind them, a
// power of two of at least 32.  With 16 or 32 tiles the scores alone fill 256 or 512 columns (what two CTAs per SM,
// or one, can have): the output accumulator then takes the columns of tile 0 once that tile's probabilities have
// been formed, and the per-slot sums of tile 0, which would lie there, go to two columns of the last even tile but
// one (by then read for the last time, by the same thread, or not used at all).
__host__ __device__ inline bool multi_um_o_aliases(int B) {
  const int tiles = (B + kUmTile - 1) / kUmTile;
  return tiles == 16 || tiles == 32;
}
__host__ __device__ inline int multi_um_cols(int B) {
  const int tiles = (B + kUmTile - 1) / kUmTile;
  const int need = multi_um_o_aliases(B) ? 16 * tiles : 16 * tiles + 16;
  int c = 32;
  while (c < need) c <<= 1;
  return c;
}
__host__ __device__ inline int multi_um_sums_col_of_tile0(int B) { return 16 * ((B + kUmTile - 1) / kUmTile - 2) + 2; }

// v[i] (i = query, N = 8 or 16 of them) reduced over the 32 lanes; lane l returns the result for query l / (32 / N).
// The exchange halves the number of live values at every step (N shuffles in all instead of 5 N).
template <bool kMax, int N>
__device__ __forceinline__ float lanes_reduce(float (&v)[N], int lane) {
  constexpr int kSteps = N == 16 ? 4 : 3;
#pragma unroll
  for (int step = 0; step < kSteps; ++step) {
    const int w = N >> (step + 1), o = 16 >> step;
    const bool up = (lane & o) != 0;
#pragma unroll
    for (int k = 0; k < w; ++k) {
      const float send = up ? v[k] : v[k + w];
      const float keep = up ? v[k + w] : v[k];
      const float got = __shfl_xor_sync(0xffffffffu, send, o);
      v[k] = kMax ? fmaxf(keep, got) : keep + got;
    }
  }
#pragma unroll
  for (int o = 16 >> kSteps; o >= 1; o >>= 1) {
    const float got = __shfl_xor_sync(0xffffffffu, v[0], o);
    v[0] = kMax ? fmaxf(v[0], got) : v[0] + got;
  }
  return v[0];
}

// kQ consecutive columns of this thread's tensor-memory lane
template <int kQ>
__device__ __forceinline__ void tmem_ldq(uint32_t taddr, uint32_t (&r)[kQ]) {
  if constexpr (kQ == 16) tmem_ld16(taddr, r);
  else tmem_ld8(taddr, r);
}
template <int kQ>
__device__ __forceinline__ void tmem_stq(uint32_t taddr, const uint32_t (&r)[kQ]) {
  if constexpr (kQ == 16) tmem_st16(taddr, r);
  else tmem_st8(taddr, r);
}

// Per token of the block (1 << GS query heads each) the group-wise averaged probability (Sec. 5.3, App. A; one
// head: p itself); ds and dq receive its sum and sum of squares over the tokens.
template <int kQ, int GS>
__device__ __forceinline__ void token_sums(const float (&pr)[kQ], float &ds, float &dq) {
  constexpr int G = 1 << GS;
  if constexpr (G <= kQ) {
#pragma unroll
    for (int t = 0; t < kQ / G; ++t) {
      float m = pr[t * G];
#pragma unroll
      for (int h = 1; h < G; ++h) m += pr[t * G + h];
      m *= 1.f / (float)G;
      ds += m;
      dq = fmaf(m, m, dq);
    }
  }
}

// kQ: query columns the consumer threads work on (8 when the step has at most 8 query rows, else 16; the MMAs
// always carry 16, the rows that do not exist being zero).  kRing: the budget has more tiles than the P^T buffer
// holds, so a tile's block is reused once the output MMAs of the tile that held it have completed.
template <int kQ, bool kRing>
__global__ void __launch_bounds__(kUmThreads, 2) multi_step_umma_kernel(const __grid_constant__ CUtensorMap mapK,
                                                                        const __grid_constant__ CUtensorMap mapV,
                                                                        const MultiParams p, int tmem_cols) {
  using T = __nv_bfloat16;
  constexpr int D = 128;
  extern __shared__ char mq_smem_raw[];
  const int M = p.M, nb = p.nb, B = p.B, stages = p.stages;
  const MultiUmSmem sm = multi_um_carve(mq_smem_raw, B, stages, nb);
  volatile int *abort_flag = sm.ctl;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int u = blockIdx.x;

  if (tid == 0) {
    for (int i = 0; i < stages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], 1); }
    mbar_init(sm.s_full, 1);
    for (int i = 0; i < kUmMaxTiles; ++i) { mbar_init(&sm.p_tile[i], kMqConsumerWarps / 2); mbar_init(&sm.p_free[i], 1); }
    mbar_init(sm.d_ready, kMqConsumerWarps);
    mbar_init(sm.o_full, 1);
    mbar_init(sm.policy_done, 1);
    mbar_init(sm.stats_full, 1);
    sm.ctl[0] = 0;
    sm.ctl[kUmCtlStaleMax] = 0;
    mbar_init_fence();
  }
  if (warp == 0) {
    tmem_alloc(sm.tmem_base, (uint32_t)tmem_cols);
    tmem_relinquish();
  }
  int live0 = p.live[u];
  if (live0 < 0 || live0 > B) {
    if (tid == 0) atomicOr(p.status, ROCO_DEV_BAD_LIVE);
    live0 = live0 < 0 ? 0 : B;
  }
  int need = live0 + nb - B;
  if (need < 0) need = 0;
  const int live1 = live0 - need + nb;
  const int n_tiles = (live1 + kUmTile - 1) / kUmTile;
  const bool stats_by_tma =
      need > 0 && (B & 3) == 0 &&
      ((reinterpret_cast<uintptr_t>(p.s) | reinterpret_cast<uintptr_t>(p.q) | reinterpret_cast<uintptr_t>(p.n) |
        reinterpret_cast<uintptr_t>(p.pos)) & 15) == 0;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *sm.tmem_base;
  const bool o_aliases = multi_um_o_aliases(B);
  const int ptiles = multi_um_ptiles(B), pshift = ptiles == 4 ? 2 : 3;
  const uint32_t tmem_o = o_aliases ? tmem : tmem + (uint32_t)(16 * ((B + kUmTile - 1) / kUmTile));

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
        char *dst = sm.ring + (size_t)st * kUmTileBytes;
        const int row = u * B + it * kUmTile;
        mbar_expect_tx(&sm.full[st], kUmTileBytes);
        tma_load_2d(dst, map, 0, row, &sm.full[st]);
        tma_load_2d(dst + kUmHalfBytes, map, 64, row, &sm.full[st]);
      }
    }
    return;
  }

  if (warp >= kMqPolicyWarp0 && warp < kUmMmaWarp) {
    PolicyView v;
    v.z = nullptr; v.Bp = align_up((size_t)B, 64); v.vkey = sm.vkey; v.mkey = sm.mkey; v.newtok = sm.newtok;
    v.sel = sm.sel; v.knew = nullptr; v.vnew = nullptr; v.zn = sm.zn; v.qf = nullptr; v.pn = nullptr; v.ctl = sm.ctl;
    v.p_ready = nullptr;
    v.policy_done = sm.policy_done;
    v.nbuf = sm.nbuf; v.posbuf = sm.posbuf; v.stats_full = stats_by_tma ? sm.stats_full : nullptr;
    v.zn_by_consumers = true;
    v.stats_by_consumers = true;
    multi_policy<T, D>(p, v, u, tid - kMqPolicyWarp0 * 32, live0, need, live1);
    // The statistics of Sec. 4.3: the consumer that owns a slot leaves the slot's sums over the block's tokens of
    // the (group-wise averaged) probability and of its square in the first two columns of the slot's tile; the
    // four policy warps cover the four lane quarters of tensor memory.  Old values are loaded four tiles at a time.
    // (Following the consumers group by group instead of waiting for all of them cost more in the consumers' pass
    // than it saved here.)
    const int kq = (warp & 3) * 32 + lane;
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const size_t unit_st = (size_t)u * B;
    mbar_wait(sm.d_ready, 0, abort_flag, p.status);
    tc_fence_after();
    for (int it0 = 0; it0 < n_tiles; it0 += 4) {
      float so[4], qo[4];
      int no[4], nt[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int j = (it0 + k) * kUmTile + kq;
        const bool valid = it0 + k < n_tiles && j < live1;
        nt[k] = valid ? (int)sm.newtok[j] : -2;  // -2: nothing to update
        const bool old = nt[k] == -1;
        so[k] = old ? p.s[unit_st + j] : 0.f;
        qo[k] = old ? p.q[unit_st + j] : 0.f;
        no[k] = old ? p.n[unit_st + j] : 0;
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (it0 + k < n_tiles) {  // uniform over the warp
          const int j = (it0 + k) * kUmTile + kq;
          uint32_t d2[2];
          tmem_ld2(tl + (uint32_t)((o_aliases && it0 + k == 0) ? multi_um_sums_col_of_tile0(B) : 16 * (it0 + k)), d2);
          if (nt[k] > -2) {
            p.s[unit_st + j] = so[k] + __uint_as_float(d2[0]);
            p.q[unit_st + j] = qo[k] + __uint_as_float(d2[1]);
            p.n[unit_st + j] = no[k] + (nb == 1 ? 1 : (nt[k] >= 0 ? nb - nt[k] : nb));
          }
        }
      }
    }
    tc_fence_before();
    named_bar_sync(kUmBarDone, kMqConsumers + kMqPolicyThreads);
    return;
  }

  if (warp == kUmMmaWarp) {
    // ---------------------------------------------------------- MMA issue: one thread, the warp helps with zeroing
    named_bar_sync(kUmBarStaged, kMqConsumers + 32);
    for (int it = 0; it < n_tiles; ++it) {
      const int st = it % stages;
      mbar_wait(&sm.full[st], (it / stages) & 1, abort_flag, p.status);
      tc_fence_after();
      if (lane == 0) {
        const char *tile = sm.ring + (size_t)st * kUmTileBytes;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const int off = (kk >> 2) * kUmHalfBytes + (kk & 3) * 32, qoff = (kk >> 2) * 2048 + (kk & 3) * 32;
          umma_bf16(tmem + (uint32_t)(16 * it), smem_desc_sw128(tile + off), smem_desc_sw128(sm.qv + qoff), kIdescUmS,
                    kk > 0 ? 1u : 0u);
        }
        umma_commit(&sm.empty[st]);
        if (it == n_tiles - 1) umma_commit(sm.s_full);
      }
      __syncwarp();
    }
    for (int it = 0; it < n_tiles; ++it) {
      const int g = n_tiles + it;
      const int st = g % stages;
      mbar_wait(&sm.p_tile[it], 0, abort_flag, p.status);  // this tile's P^T block (at it = 0 also: its columns are free)
      mbar_wait(&sm.full[st], (g / stages) & 1, abort_flag, p.status);
      char *tile = sm.ring + (size_t)st * kUmTileBytes;
      if ((it + 1) * kUmTile > live0) {
        // slots that were free before the step may hold anything (their probabilities are zero, but 0 x NaN)
        const int r0 = live0 > it * kUmTile ? live0 - it * kUmTile : 0;
        for (int w = lane; w < (kUmTile - r0) * 8; w += 32) {
          *reinterpret_cast<uint4 *>(tile + (size_t)r0 * 128 + (size_t)w * 16) = make_uint4(0u, 0u, 0u, 0u);
          *reinterpret_cast<uint4 *>(tile + kUmHalfBytes + (size_t)r0 * 128 + (size_t)w * 16) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_async_smem();
        __syncwarp();
      }
      tc_fence_after();
      if (lane == 0) {
        const int ps = kRing ? (it & (ptiles - 1)) : it;  // this tile's place in the P^T buffer
        const char *pb = sm.pbuf + (size_t)(ps >> 2) * kUmPBlock + (ps & 3) * 32;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          umma_bf16(tmem_o, smem_desc_sw128_mn(tile + kk * 2048, kUmHalfBytes), smem_desc_sw128_mn(pb + kk * 2048, 16),
                    kIdescUmO, (it > 0 || kk > 0) ? 1u : 0u);
        umma_commit(&sm.empty[st]);
        if (kRing && it + ptiles < n_tiles) umma_commit(&sm.p_free[ps]);  // a later tile waits for this place
      }
      __syncwarp();
    }
    if (lane == 0) {
      umma_bf16(tmem_o, smem_desc_sw128_mn(sm.qv, 2048), smem_desc_sw128_mn(sm.pn, 16), kIdescUmO, 1u);
      umma_commit(sm.o_full);
    }
    return;
  }

  // -------------------------------------------------------------- consumers
  const float zscale = p.scale * kLog2e;
  const int grp = p.group;
  const T *Qu = (const T *)p.Q + (size_t)u * p.q_ustride * D;
  // the queries as the K-major B operand of the score MMAs: row i = 128 bytes per 64-column half, 128-byte swizzle
  {
    const int i = tid >> 4, chunk = tid & 15;
    uint4 val = make_uint4(0u, 0u, 0u, 0u);
    if (i < M) val = *(reinterpret_cast<const uint4 *>(Qu + (size_t)i * D) + chunk);
    *reinterpret_cast<uint4 *>(sm.qv + (chunk >> 3) * 2048 + i * 128 + (((chunk & 7) ^ (i & 7)) << 4)) = val;
    fence_async_smem();
  }
  named_bar_sync(kUmBarStaged, kMqConsumers + 32);

  // this step's values: each consumer thread fetches one 16-byte piece now and stores it once the score MMAs have
  // finished with the shared memory it goes to
  uint4 vn_piece = make_uint4(0u, 0u, 0u, 0u);
  if ((tid >> 4) < nb)
    vn_piece = *(reinterpret_cast<const uint4 *>((const T *)p.v_new + ((size_t)u * p.kv_ustride + (tid >> 4)) * D) + (tid & 15));
  const int gshift = nb == 1 ? 4 : (grp >= 8 ? 3 : (grp >= 4 ? 2 : (grp >= 2 ? 1 : 0)));  // token of row i: i >> gshift
  // raw scores of the queries against the new tokens, from k_new: Zn[16 x 8] per warp (warps 0 and 1: 8 new
  // tokens each), stored with the query index contiguous, and their row maxima under the causal mask of the block
  if (warp < 2) {
    const int g = lane >> 2, tq = lane & 3;
    const bool row_lo = g < M, row_hi = g + 8 < M;
    const T *Kn = (const T *)p.k_new + (size_t)u * p.kv_ustride * D;
    const int jn = warp * 8 + g;
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    if (warp * 8 < nb) {
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        const int k0 = s * 16 + tq * 2;
        uint32_t qa[4];
        qa[0] = row_lo ? *reinterpret_cast<const uint32_t *>(Qu + (size_t)g * D + k0) : 0u;
        qa[1] = row_hi ? *reinterpret_cast<const uint32_t *>(Qu + (size_t)(g + 8) * D + k0) : 0u;
        qa[2] = row_lo ? *reinterpret_cast<const uint32_t *>(Qu + (size_t)g * D + k0 + 8) : 0u;
        qa[3] = row_hi ? *reinterpret_cast<const uint32_t *>(Qu + (size_t)(g + 8) * D + k0 + 8) : 0u;
        const uint32_t b0 = jn < nb ? *reinterpret_cast<const uint32_t *>(Kn + (size_t)jn * D + k0) : 0u;
        const uint32_t b1 = jn < nb ? *reinterpret_cast<const uint32_t *>(Kn + (size_t)jn * D + k0 + 8) : 0u;
        mma_bf16_16816(c, qa, b0, b1);
      }
    }
    const int j0 = warp * 8 + tq * 2;
    // row i sees new token j iff j < nb and j <= i >> gshift
    const bool s0 = row_lo && j0 < nb && j0 <= (g >> gshift), s1 = row_lo && j0 + 1 < nb && j0 + 1 <= (g >> gshift);
    const bool s2 = row_hi && j0 < nb && j0 <= ((g + 8) >> gshift);
    const bool s3 = row_hi && j0 + 1 < nb && j0 + 1 <= ((g + 8) >> gshift);
    if (j0 < nb) { sm.zn[j0 * 16 + g] = s0 ? c[0] : -INFINITY; sm.zn[j0 * 16 + g + 8] = s2 ? c[2] : -INFINITY; }
    if (j0 + 1 < nb) { sm.zn[(j0 + 1) * 16 + g] = s1 ? c[1] : -INFINITY; sm.zn[(j0 + 1) * 16 + g + 8] = s3 ? c[3] : -INFINITY; }
    float mlo = fmaxf(s0 ? c[0] : -INFINITY, s1 ? c[1] : -INFINITY), mhi = fmaxf(s2 ? c[2] : -INFINITY, s3 ? c[3] : -INFINITY);
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      mlo = fmaxf(mlo, __shfl_xor_sync(0xffffffffu, mlo, o));
      mhi = fmaxf(mhi, __shfl_xor_sync(0xffffffffu, mhi, o));
    }
    if (tq == 0) {
      float *znmax = sm.red + 2 * kMqConsumerWarps * 16 + warp * 16;
      znmax[g] = mlo;
      znmax[g + 8] = mhi;
    }
  }

  // this thread: key kl of the tiles wg, wg + 2, ...; tensor-memory lane kl, columns 16 it .. 16 it + 15
  const int wq = warp & 3, wg = warp >> 2;
  const int kl = wq * 32 + lane;
  const uint32_t tlane = tmem + ((uint32_t)(wq * 32) << 16);
  const uint32_t ninf = 0xff800000u;
  // over the 256 consumer threads; returns the result for query (lane & (kQ - 1)) and leaves in v the maxima of
  // all kQ queries, or the reciprocals of their sums (0 for rows that do not exist)
  auto all_reduce = [&](float (&v)[kQ], bool is_max, float *red) {
    const float x = is_max ? lanes_reduce<true, kQ>(v, lane) : lanes_reduce<false, kQ>(v, lane);
    if ((lane & (32 / kQ - 1)) == 0) red[warp * kQ + lane / (32 / kQ)] = x;
    named_bar_sync(kMqBarConsumers, kMqConsumers);
    float acc = red[lane & (kQ - 1)];
#pragma unroll
    for (int w = 1; w < kMqConsumerWarps; ++w) {
      const float o = red[w * kQ + (lane & (kQ - 1))];
      acc = is_max ? fmaxf(acc, o) : acc + o;
    }
    const float give = is_max ? acc : ((lane & (kQ - 1)) < M ? 1.f / acc : 0.f);
#pragma unroll
    for (int i = 0; i < kQ; ++i) v[i] = __shfl_sync(0xffffffffu, give, i);
    return acc;
  };

  mbar_wait(sm.s_full, 0, abort_flag, p.status);
  tc_fence_after();
  // the score MMAs are done with the query operand: V_new takes its place as a 16-key tile with the dimension
  // index contiguous (rows of new tokens that do not exist are zero), and the new tokens' P^T block is cleared
  {
    const int jn = tid >> 4, chunk = tid & 15;
    *reinterpret_cast<uint4 *>(sm.qv + (chunk >> 3) * 2048 + jn * 128 + (((chunk & 7) ^ (jn & 7)) << 4)) = vn_piece;
    if (tid < 128) *reinterpret_cast<uint4 *>(sm.pn + tid * 16) = make_uint4(0u, 0u, 0u, 0u);
  }

  // ---- pass 1, while the selection may still be running: row maxima over the slots that held a token before
  // the step.  The slots that the new tokens will take still count with the score of the token they held, which
  // only makes the maximum an upper bound (it is the stabiliser of the exponentials, nothing else) -- unless that
  // score was the row's maximum: far above the others it would push every exponential of the row below the
  // smallest float.  Then (rare) a second turn takes the maxima again, over the scores as they stand by then.
  float a[kQ];
  float my_max;
#pragma unroll 1
  for (int turn = 0;; ++turn) {
#pragma unroll
    for (int i = 0; i < kQ; ++i) a[i] = -INFINITY;
    for (int it = wg; it < n_tiles; it += 2) {
      const int j = it * kUmTile + kl;
      uint32_t r[kQ];
      tmem_ldq<kQ>(tlane + (uint32_t)(it * 16), r);
      const bool counts = turn > 0 || j < live0;  // second turn: the masks are in place
#pragma unroll
      for (int i = 0; i < kQ; ++i) a[i] = fmaxf(a[i], counts ? __uint_as_float(r[i]) : -INFINITY);
    }
    my_max = all_reduce(a, true, sm.red);  // its barrier also publishes zn, V_new and the cleared block
    {
      // the new tokens' scores join the maxima
      const float *znmax = sm.red + 2 * kMqConsumerWarps * 16;
      const float zm = fmaxf(znmax[lane & (kQ - 1)], znmax[16 + (lane & (kQ - 1))]);
      my_max = fmaxf(my_max, zm);
#pragma unroll
      for (int k = 0; k < kQ; ++k) a[k] = fmaxf(a[k], __shfl_sync(0xffffffffu, zm, k));
    }
    // a[i] <- -(row maximum in the log2 domain); rows that do not exist hold zeros
#pragma unroll
    for (int i = 0; i < kQ; ++i) a[i] = (a[i] > -INFINITY) ? -a[i] * zscale : 0.f;
    if (turn > 0) break;

    // ---- the selection's result: masks and the new tokens' scores in place
    mbar_wait(sm.policy_done, 0, abort_flag, p.status);
    for (int it = wg; it < n_tiles; it += 2) {
      const int j = it * kUmTile + kl;
      const int nt = j < live1 ? (int)sm.newtok[j] : -1;
      if (__any_sync(0xffffffffu, nt >= 0 || j >= live1)) {
        uint32_t r[kQ];
        tmem_ldq<kQ>(tlane + (uint32_t)(it * 16), r);
        if (j >= live1) {
#pragma unroll
          for (int i = 0; i < kQ; ++i) r[i] = ninf;
        } else if (nt >= 0) {  // the new token's scores, -inf where the block's causal mask hides it
          // (did the score this slot held set a row's maximum?  Within a binary order counts, which also covers
          // the rounding of the comparison.)
          bool held_max = false;
#pragma unroll
          for (int i = 0; i < kQ; ++i) held_max |= i < M && fmaf(__uint_as_float(r[i]), zscale, a[i]) >= -1.f;
          if (held_max && j < live0) sm.ctl[kUmCtlStaleMax] = 1;  // (a slot that was free counted for nothing)
          const uint4 *zr = reinterpret_cast<const uint4 *>(sm.zn + nt * 16);
#pragma unroll
          for (int k = 0; k < kQ / 4; ++k) {
            const uint4 z4 = zr[k];
            r[4 * k] = z4.x; r[4 * k + 1] = z4.y; r[4 * k + 2] = z4.z; r[4 * k + 3] = z4.w;
          }
        }
        tmem_stq<kQ>(tlane + (uint32_t)(it * 16), r);
      }
    }
    tmem_st_wait();
    named_bar_sync(kMqBarConsumers, kMqConsumers);
    if (!sm.ctl[kUmCtlStaleMax]) break;
  }

  // ---- pass 2: e = 2^(z - max) in place, row sums
  float sums[kQ];
#pragma unroll
  for (int i = 0; i < kQ; ++i) sums[i] = 0.f;
  for (int it = wg; it < n_tiles; it += 2) {
    uint32_t r[kQ];
    tmem_ldq<kQ>(tlane + (uint32_t)(it * 16), r);
#pragma unroll
    for (int i = 0; i < kQ; ++i) {
      const float e = ex2_approx(fmaf(__uint_as_float(r[i]), zscale, a[i]));
      sums[i] += e;
      r[i] = __float_as_uint(e);
    }
    tmem_stq<kQ>(tlane + (uint32_t)(it * 16), r);
  }
  tmem_st_wait();
  const float my_sum = all_reduce(sums, false, sm.red + kMqConsumerWarps * 16);
  if (warp == 0 && lane < kQ && lane < M && p.lse) {
    const float mz = (my_max > -INFINITY) ? my_max * zscale : 0.f;
    p.lse[(size_t)u * M + lane] = (mz + log2f(my_sum)) * kLn2;
  }

  float ds_tile0 = 0.f, dq_tile0 = 0.f;
  // ---- pass 3: probabilities; P^T as bf16 operand blocks, tile by tile (the output MMAs of a tile start as soon
  // as its block is complete); the statistics of Sec. 4.3 for this thread's slots
  for (int it = wg; it < n_tiles; it += 2) {
    const int j = it * kUmTile + kl;
    uint32_t r[kQ];
    tmem_ldq<kQ>(tlane + (uint32_t)(it * 16), r);
    float pr[kQ];
#pragma unroll
    for (int i = 0; i < kQ; ++i) pr[i] = __uint_as_float(r[i]) * sums[i];  // sums[] holds the reciprocals by now
    const int nt = j < live1 ? (int)sm.newtok[j] : -1;
    {
      uint4 w0, w1;
      w0.x = pack_bf16x2(pr[0], pr[1]); w0.y = pack_bf16x2(pr[2], pr[3]);
      w0.z = pack_bf16x2(pr[4], pr[5]); w0.w = pack_bf16x2(pr[6], pr[7]);
      if constexpr (kQ == 16) {
        w1.x = pack_bf16x2(pr[8], pr[9]); w1.y = pack_bf16x2(pr[10], pr[11]);
        w1.z = pack_bf16x2(pr[12], pr[13]); w1.w = pack_bf16x2(pr[14], pr[15]);
      } else {
        w1 = make_uint4(0u, 0u, 0u, 0u);  // the operand carries 16 queries: the upper eight do not exist
      }
      if (nt >= 0) {
        // a new token's value comes from V_new: its probabilities go to the new tokens' block, and the streamed
        // row of its slot (possibly read before the overwrite) gets zeros
        char *row = sm.pn + nt * 128;
        *reinterpret_cast<uint4 *>(row + ((0 ^ (nt & 7)) << 4)) = w0;
        *reinterpret_cast<uint4 *>(row + ((1 ^ (nt & 7)) << 4)) = w1;
        w0 = make_uint4(0u, 0u, 0u, 0u);
        w1 = w0;
      }
      const int ps = kRing ? (it & (ptiles - 1)) : it;
      if (kRing && it >= ptiles) mbar_wait(&sm.p_free[ps], ((it >> pshift) - 1) & 1, abort_flag, p.status);
      char *row = sm.pbuf + (size_t)(ps >> 2) * kUmPBlock + kl * 128;
      const int c0 = 2 * (ps & 3);
      *reinterpret_cast<uint4 *>(row + ((c0 ^ (kl & 7)) << 4)) = w0;
      *reinterpret_cast<uint4 *>(row + (((c0 + 1) ^ (kl & 7)) << 4)) = w1;
    }
    fence_async_smem();
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.p_tile[it]);
    // per token of the block the group-wise averaged probability (Sec. 5.3, App. A; one head: p itself), then its
    // sum and sum of squares over the tokens; one token with all rows as its heads when nb = 1
    float ds = 0.f, dq = 0.f;
    if (nb == 1) {  // one token with all rows as its heads
      float t = 0.f;
#pragma unroll
      for (int i = 0; i < kQ; ++i) t += pr[i];
      ds = t / (float)M;
      dq = ds * ds;
    } else if (gshift == 0) {
      token_sums<kQ, 0>(pr, ds, dq);
    } else if (gshift == 1) {
      token_sums<kQ, 1>(pr, ds, dq);
    } else if (gshift == 2) {
      token_sums<kQ, 2>(pr, ds, dq);
    } else {
      token_sums<kQ, 3>(pr, ds, dq);
    }
    // for the policy warps
    if (o_aliases && it == 0) { ds_tile0 = ds; dq_tile0 = dq; }
    else tmem_st2(tlane + (uint32_t)(it * 16), __float_as_uint(ds), __float_as_uint(dq));
  }
  if (o_aliases && wg == 0)
    tmem_st2(tlane + (uint32_t)multi_um_sums_col_of_tile0(B), __float_as_uint(ds_tile0), __float_as_uint(dq_tile0));
  tmem_st_wait();
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(sm.d_ready);

  // ---- output: O^T[dim][query] from tensor memory, this thread's dimension wq * 32 + lane, queries 8 wg .. 8 wg + 7
  mbar_wait(sm.o_full, 0, abort_flag, p.status);
  tc_fence_after();
  {
    uint32_t o[8];
    tmem_ld8(tmem_o + ((uint32_t)(wq * 32) << 16) + (uint32_t)(8 * wg), o);
    T *outp = (T *)p.out + (size_t)u * p.out_ustride * D + kl;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int i = 8 * wg + k;
      if (i < M) outp[(size_t)i * D] = __float2bfloat16(__uint_as_float(o[k]));
    }
  }
  tc_fence_before();
  named_bar_sync(kUmBarDone, kMqConsumers + kMqPolicyThreads);
  if (warp == 0) tmem_dealloc(tmem, (uint32_t)tmem_cols);
}

// Ring stages of the tcgen05 kernel: two (of 32 KiB) where two CTAs then share an SM, which covers a CTA's softmax
// phase with the other's stream; else one CTA per SM with as many stages as fit.  0: the budget does not fit.
int multi_um_pick_stages(int B, int nb) {
  const size_t per_sm = 227 * 1024;
  if (multi_um_cols(B) > 512) return 0;
  if (multi_um_cols(B) <= 256 && (multi_um_smem_bytes(B, 2, nb) + 1024) * 2 <= per_sm) return 2;
  for (int st = 4; st >= 2; --st)
    if (multi_um_smem_bytes(B, st, nb) + 1024 <= per_sm) return st;
  return 0;
}

// Row layouts the tcgen05 kernel takes: the heads of a token are averaged inside a thread -- group sizes that are
// powers of two, or one token with any number of heads.
bool multi_um_rows(int M, int nb) {
  const int grp = M / nb;
  return M >= 1 && (nb == 1 || grp == 1 || grp == 2 || grp == 4 || grp == 8);
}

int launch_multi_step_umma(const MultiParams &p, const roco_cache &c, int U, cudaStream_t stream) {
  CUtensorMap mapK, mapV;
  if (!make_tensor_map_rows128_bf16(&mapK, c.K, (unsigned long long)U * c.B, kUmTile) ||
      !make_tensor_map_rows128_bf16(&mapV, c.V, (unsigned long long)U * c.B, kUmTile))
    return -1;
  const size_t smem = multi_um_smem_bytes(c.B, p.stages, p.nb);
  const bool ring = (c.B + kUmTile - 1) / kUmTile > multi_um_ptiles(c.B);
  auto kernel = p.M <= 8 ? (ring ? multi_step_umma_kernel<8, true> : multi_step_umma_kernel<8, false>)
                         : (ring ? multi_step_umma_kernel<16, true> : multi_step_umma_kernel<16, false>);
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return ROCO_ERR_CUDA;
  kernel<<<U, kUmThreads, smem, stream>>>(mapK, mapV, p, multi_um_cols(c.B));
  return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
