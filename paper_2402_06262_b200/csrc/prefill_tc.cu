// Prefill statistics on the 5th-generation tensor cores (bf16, d = 128): the causal score matrix of Eq. 1 is
// a dense contraction, computed 128 x 128 tiles at a time by tcgen05.mma with fp32 accumulators in tensor
// memory, operands staged in shared memory by TMA (128-byte swizzle, non-multicast).  Two passes, neither
// of which ever stores the L x L matrix:
//   pass 0 (row LSE):      S   = Q_a K_j^T  (a query row per TMEM lane): each thread keeps the running
//                          (max, sum) of one row, lse_i = log sum_{j<=i} exp(scale * Q_i.K_j);
//   pass 1 (column stats): S^T = K_a Q_i^T  (a key per TMEM lane): each thread recomputes
//                          P_ij = exp(z_ij - lse_i) for one key column and keeps running fp32 sums
//                          s_j = sum_i P_ij and q_j = sum_i P_ij^2 (Sec. 4.3) over all query tiles i >= a.
// A CTA owns a pair of stationary tiles (a, T-1-a), so every CTA does the same number of tile products
// under the causal mask.  Warp roles: warps 0-7 read the accumulators (TMEM lane quarter = warp id mod 4) and
// do the softmax arithmetic -- two groups of four warps, each owning one of the two accumulators, so that
// the contraction of one tile overlaps the exponentials of the previous one and the exponential unit always
// has a second group to serve -- warp 8 issues TMA, warp 9 issues the MMAs.  The exponentials, not the
// tensor pipe, are the practical limit of both passes (16384 per tile against 512 MMA cycles).
#include <cuda.h>

#include <type_traits>

#include "common.cuh"
#include "launch.h"
#include "tc.cuh"

namespace roco {

constexpr int kTcStages = 2;                       // streamed-tile ring
constexpr int kTcAccs = 2;                         // accumulators in tensor memory
constexpr int kTcTmemCols = kTcAccs * kTcTile;     // 256 columns
constexpr int kTcComputeWarps = 8;                 // two groups of four, one per accumulator
constexpr int kTcGroupThreads = 128;
constexpr int kTcComputeThreads = kTcComputeWarps * 32;
constexpr int kTcThreads = kTcComputeThreads + 64; // + TMA warp + MMA warp
constexpr int kTcBarGroup0 = 1;                    // named barriers: 1, 2 = the two groups; 3 = both
constexpr int kTcBarBoth = 3;


struct TcSmem {
  char *stat;                 // stationary operand tile
  char *ring;                 // kTcStages streamed operand tiles
  float *lse2;                // [2 groups][2][128] minus the log2-domain row LSE of a group's query tile (pass 1)
  float *merge;               // [2 tasks][2][128] partial running values handed from group 1 to group 0
  uint64_t *stat_full, *stat_empty;
  uint64_t *ring_full, *ring_empty;  // [kTcStages]
  uint64_t *acc_full, *acc_empty;    // [kTcAccs]
  uint32_t *tmem_base;
  int *abort_flag;
};

constexpr size_t kTcSmemBytes = 1024 /*align*/ + (size_t)(1 + kTcStages) * kTcTileBytes + 8 * 128 * 4 +
                                (2 + 2 * kTcStages + 2 * kTcAccs) * 8 + 16;

__device__ inline TcSmem tc_carve(char *raw) {
  TcSmem m;
  char *p = smem_align(raw, 1024);  // swizzle atoms are 1024-byte aligned
  m.stat = p; p += kTcTileBytes;
  m.ring = p; p += (size_t)kTcStages * kTcTileBytes;
  m.lse2 = (float *)p; p += 4 * 128 * 4;
  m.merge = (float *)p; p += 4 * 128 * 4;
  m.stat_full = (uint64_t *)p; p += 8;
  m.stat_empty = (uint64_t *)p; p += 8;
  m.ring_full = (uint64_t *)p; p += 8 * kTcStages;
  m.ring_empty = (uint64_t *)p; p += 8 * kTcStages;
  m.acc_full = (uint64_t *)p; p += 8 * kTcAccs;
  m.acc_empty = (uint64_t *)p; p += 8 * kTcAccs;
  m.tmem_base = (uint32_t *)p; p += 8;
  m.abort_flag = (int *)p;
  return m;
}

// PASS 0: stationary = Q tile a, streamed = K tiles 0..a, output lse.
// PASS 1: stationary = K tile a, streamed = Q tiles a..T-1, input lse, output s_full / q_full.
template <int PASS>
__global__ void __launch_bounds__(kTcThreads, 2) prefill_tc_kernel(const __grid_constant__ CUtensorMap mapQ,
                                                                const __grid_constant__ CUtensorMap mapK,
                                                                const int *lens, int G, int Lmax, int npairs,
                                                                float scale, float *lse, float *s_full, float *q_full,
                                                                int *status) {
  extern __shared__ char tc_smem_raw[];
  const TcSmem sm = tc_carve(tc_smem_raw);
  volatile int *abort_flag = sm.abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int u = blockIdx.x / npairs, pair = blockIdx.x % npairs;
  const int L = lens[u / G];
  const int T = (L + kTcTile - 1) / kTcTile;
  // stationary tiles of this CTA: `pair` and its mirror (same total work for every CTA)
  const int a0 = pair, a1 = T - 1 - pair;
  const int n_tasks = (a0 > a1) ? 0 : (a0 == a1 ? 1 : 2);
  if (n_tasks == 0) return;

  if (tid == 0) {
    mbar_init(sm.stat_full, 1);
    mbar_init(sm.stat_empty, 1);
    for (int i = 0; i < kTcStages; ++i) { mbar_init(&sm.ring_full[i], 1); mbar_init(&sm.ring_empty[i], 1); }
    for (int i = 0; i < kTcAccs; ++i) { mbar_init(&sm.acc_full[i], 1); mbar_init(&sm.acc_empty[i], 4); }
    *sm.abort_flag = 0;
    mbar_init_fence();
  }
  if (warp == 0) {
    tmem_alloc(sm.tmem_base, kTcTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *sm.tmem_base;

  // streamed tiles of task k: first index and count
  auto task_tile = [&](int k) { return k == 0 ? a0 : a1; };
  auto task_first = [&](int a) { return PASS == 0 ? 0 : a; };
  auto task_count = [&](int a) { return PASS == 0 ? a + 1 : T - a; };

  if (warp == kTcComputeWarps) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const CUtensorMap *map_stat = PASS == 0 ? &mapQ : &mapK;
      const CUtensorMap *map_ring = PASS == 0 ? &mapK : &mapQ;
      int g = 0;  // streamed tiles issued so far
      for (int k = 0; k < n_tasks; ++k) {
        const int a = task_tile(k);
        if (k > 0) mbar_wait(sm.stat_empty, (k - 1) & 1, abort_flag, status);
        mbar_expect_tx(sm.stat_full, kTcTileBytes);
        tma_load_3d(sm.stat, map_stat, 0, a * kTcTile, u, sm.stat_full);
        tma_load_3d(sm.stat + kTcHalfBytes, map_stat, 64, a * kTcTile, u, sm.stat_full);
        const int first = task_first(a), cnt = task_count(a);
        for (int t = 0; t < cnt; ++t, ++g) {
          const int st = g % kTcStages;
          if (g >= kTcStages) mbar_wait(&sm.ring_empty[st], ((g / kTcStages) - 1) & 1, abort_flag, status);
          char *dst = sm.ring + (size_t)st * kTcTileBytes;
          mbar_expect_tx(&sm.ring_full[st], kTcTileBytes);
          tma_load_3d(dst, map_ring, 0, (first + t) * kTcTile, u, &sm.ring_full[st]);
          tma_load_3d(dst + kTcHalfBytes, map_ring, 64, (first + t) * kTcTile, u, &sm.ring_full[st]);
        }
      }
    }
  } else if (warp == kTcComputeWarps + 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int g = 0;
      for (int k = 0; k < n_tasks; ++k) {
        const int a = task_tile(k);
        mbar_wait(sm.stat_full, k & 1, abort_flag, status);
        const int cnt = task_count(a);
        for (int t = 0; t < cnt; ++t, ++g) {
          const int st = g % kTcStages, ac = g % kTcAccs;
          mbar_wait(&sm.ring_full[st], (g / kTcStages) & 1, abort_flag, status);
          if (g >= kTcAccs) mbar_wait(&sm.acc_empty[ac], ((g / kTcAccs) - 1) & 1, abort_flag, status);
          tc_fence_after();
          const char *bt = sm.ring + (size_t)st * kTcTileBytes;
#pragma unroll
          for (int kk = 0; kk < kTcD / 16; ++kk) {
            const int off = (kk / 4) * kTcHalfBytes + (kk % 4) * 32;  // 16 bf16 = 32 bytes inside the swizzle row
            umma_bf16(tmem + (uint32_t)(ac * kTcTile), smem_desc_sw128(sm.stat + off), smem_desc_sw128(bt + off),
                      kIdescBf16M128N128, kk > 0 ? 1u : 0u);
          }
          umma_commit(&sm.ring_empty[st]);  // the streamed stage may be refilled once these MMAs are done
          umma_commit(&sm.acc_full[ac]);
        }
        umma_commit(sm.stat_empty);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax / statistics warps
    const float zscale = scale * kLog2e;
    const int group = warp >> 2;                 // which accumulator this warp serves
    const int gtid = tid & (kTcGroupThreads - 1);
    const int row = (warp & 3) * 32 + lane;      // TMEM lane of this thread
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t taddr = tmem + lane_addr + (uint32_t)(group * kTcTile);
    int g0 = 0;     // streamed tiles of earlier tasks
    int mine = 0;   // tiles this group has processed so far (parity of its accumulator barrier, lse2 buffer)
    for (int k = 0; k < n_tasks; ++k) {
      const int a = task_tile(k);
      const int first = task_first(a), cnt = task_count(a);
      const int grow = a * kTcTile + row;  // global index of this thread's row (query in pass 0, key in pass 1)
      float run0 = PASS == 0 ? -INFINITY : 0.f;  // pass 0: running max;  pass 1: running sum of p
      float run1 = 0.f;                          // pass 0: running sum;  pass 1: running sum of p^2
      const int t0 = ((g0 & 1) == group) ? 0 : 1;  // this group's first tile of the task
      float lse_next = 0.f;
      if (PASS == 1 && t0 < cnt) {
        const int qi = (first + t0) * kTcTile + gtid;
        lse_next = (qi < L) ? lse[(size_t)u * Lmax + qi] : 0.f;
      }
      for (int t = t0; t < cnt; t += 2, ++mine) {
        const int j = first + t;  // streamed tile index
        float *l2 = sm.lse2 + (group * 2 + (mine & 1)) * 128;
        if (PASS == 1) {
          l2[gtid] = -lse_next * kLog2e;
          if (group == 0) named_bar_sync(kTcBarGroup0, kTcGroupThreads);
          else named_bar_sync(kTcBarGroup0 + 1, kTcGroupThreads);
          const int qn = (j + 2) * kTcTile + gtid;
          lse_next = (t + 2 < cnt && qn < L) ? lse[(size_t)u * Lmax + qn] : 0.f;
        }
        mbar_wait(&sm.acc_full[group], mine & 1, abort_flag, status);
        tc_fence_after();
        const int col0 = j * kTcTile;  // global index of column 0 (key in pass 0, query in pass 1)
        uint32_t ra[32], rb[32];

        // one 32-column chunk of the accumulator row of this thread
        auto chunk = [&](const uint32_t (&r)[32], int c, auto masked_tag) {
          constexpr bool kMasked = decltype(masked_tag)::value;
          const f32x2 zs2 = pack2(zscale, zscale);
          if (PASS == 0) {
            // online softmax, one rescale per chunk
            float cmax = -INFINITY;
            if (kMasked) {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                cmax = fmaxf(cmax, (col0 + c * 32 + i <= grow) ? __uint_as_float(r[i]) : -INFINITY);
            } else {  // three-input maxima: two elements per instruction
#pragma unroll
              for (int i = 0; i < 32; i += 2) cmax = max3(cmax, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
            }
            const float m_new = fmaxf(run0, cmax * zscale);
            if (m_new > -INFINITY) {
              const f32x2 nm2 = pack2(-m_new, -m_new);
              f32x2 part2 = pack2(0.f, 0.f);
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                f32x2 e2 = exp2_pair(fma2(pack2u(r[i], r[i + 1]), zs2, nm2), i >> 1);
                if (kMasked) {
                  float ea, eb;
                  unpack2(e2, ea, eb);
                  e2 = pack2((col0 + c * 32 + i <= grow) ? ea : 0.f, (col0 + c * 32 + i + 1 <= grow) ? eb : 0.f);
                }
                part2 = add2(part2, e2);
              }
              float pa, pb;
              unpack2(part2, pa, pb);
              run1 = run1 * ex2_approx(run0 - m_new) + (pa + pb);
              run0 = m_new;
            }
          } else {
            f32x2 ts2 = pack2(0.f, 0.f), tq2 = pack2(0.f, 0.f);
            const f32x2 *l2p = reinterpret_cast<const f32x2 *>(l2 + c * 32);  // holds -lse * log2(e)
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              f32x2 p2 = exp2_pair(fma2(pack2u(r[i], r[i + 1]), zs2, l2p[i >> 1]), i >> 1);
              if (kMasked) {
                const int qi = col0 + c * 32 + i;
                float pa, pb;
                unpack2(p2, pa, pb);
                p2 = pack2((qi >= grow && qi < L) ? pa : 0.f, (qi + 1 >= grow && qi + 1 < L) ? pb : 0.f);
              }
              ts2 = add2(ts2, p2);
              tq2 = fma2(p2, p2, tq2);
            }
            float a0, a1, b0, b1;
            unpack2(ts2, a0, a1);
            unpack2(tq2, b0, b1);
            run0 += a0 + a1;
            run1 += b0 + b1;
          }
        };
        auto tile = [&](auto masked_tag) {
          tmem_ld32_issue(taddr, ra);
          tmem_ld_wait(ra);
          tmem_ld32_issue(taddr + 32, rb);
          chunk(ra, 0, masked_tag);
          tmem_ld_wait(rb);
          tmem_ld32_issue(taddr + 64, ra);
          chunk(rb, 1, masked_tag);
          tmem_ld_wait(ra);
          tmem_ld32_issue(taddr + 96, rb);
          chunk(ra, 2, masked_tag);
          tmem_ld_wait(rb);
          // the accumulator has been read completely: hand it back before the last chunk's arithmetic
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.acc_empty[group]);
          chunk(rb, 3, masked_tag);
        };
        const bool edge = PASS == 0 ? (j == a) : ((j == a) || ((j + 1) * kTcTile > L));
        if (edge) tile(std::true_type{}); else tile(std::false_type{});
      }
      g0 += cnt;
      // group 1 hands its partial running values to group 0, which merges and stores
      float *mg = sm.merge + k * 256;
      if (group == 1) { mg[row] = run0; mg[128 + row] = run1; }
      named_bar_sync(kTcBarBoth, kTcComputeThreads);
      if (group == 0 && grow < L) {
        const float o0 = mg[row], o1 = mg[128 + row];
        if (PASS == 0) {
          const float m = fmaxf(run0, o0);
          const float l = run1 * ex2_approx(run0 - m) + o1 * ex2_approx(o0 - m);
          lse[(size_t)u * Lmax + grow] = (m + log2f(l)) * kLn2;
        } else {
          s_full[(size_t)u * Lmax + grow] = run0 + o0;
          q_full[(size_t)u * Lmax + grow] = run1 + o1;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTcTmemCols);
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// [U][Lmax][128] bf16 as a 3-D tensor; box = 64 columns x 128 rows x 1 unit, 128-byte swizzle, zero fill
bool make_tensor_map_prompt_bf16(void *map_out, const void *base, int U, int Lmax) {
  CUtensorMap *map = static_cast<CUtensorMap *>(map_out);
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)kTcD, (cuuint64_t)Lmax, (cuuint64_t)U};
  const cuuint64_t strides[2] = {(cuuint64_t)kTcD * 2, (cuuint64_t)Lmax * kTcD * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)kTcTile, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [rows][128] bf16 as a 2-D tensor; box = 64 columns x box_rows rows, 128-byte swizzle, zero fill
bool make_tensor_map_rows128_bf16(void *map, const void *base, unsigned long long rows, unsigned box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)kTcD, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)kTcD * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(static_cast<CUtensorMap *>(map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool prefill_tc_supported(int kv_dtype, int d) { return kv_dtype == ROCO_BF16 && d == kTcD && encode_fn() != nullptr; }

roco_status launch_prefill_stats_tc(int S, int G, int Lmax, const int *lens_dev, int maxlen, const void *Q,
                                    const void *K, float scale, float *lse, float *s_full, float *q_full, int *status,
                                    cudaStream_t stream, bool lse_ready) {
  CUtensorMap mapQ, mapK;
  const int U = S * G;
  if (!make_tensor_map_prompt_bf16(&mapQ, Q, U, Lmax) || !make_tensor_map_prompt_bf16(&mapK, K, U, Lmax))
    return ROCO_ERR_CUDA;
  const int T = (maxlen + kTcTile - 1) / kTcTile;
  const int npairs = (T + 1) / 2;
  const unsigned grid = (unsigned)U * (unsigned)npairs;
  cudaError_t err = cudaFuncSetAttribute(prefill_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kTcSmemBytes);
  if (err == cudaSuccess)
    err = cudaFuncSetAttribute(prefill_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemBytes);
  if (err != cudaSuccess) return ROCO_ERR_CUDA;
  if (!lse_ready)
    prefill_tc_kernel<0><<<grid, kTcThreads, kTcSmemBytes, stream>>>(mapQ, mapK, lens_dev, G, Lmax, npairs, scale, lse,
                                                                    s_full, q_full, status);
  prefill_tc_kernel<1><<<grid, kTcThreads, kTcSmemBytes, stream>>>(mapQ, mapK, lens_dev, G, Lmax, npairs, scale, lse,
                                                                  s_full, q_full, status);
  return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
