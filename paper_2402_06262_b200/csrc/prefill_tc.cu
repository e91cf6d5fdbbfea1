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

namespace roco {

constexpr int kTcTile = 128;                       // rows of a stationary / streamed tile
constexpr int kTcD = 128;                          // head dimension
constexpr int kTcTileBytes = kTcTile * kTcD * 2;   // 32 KiB: two 64-column halves of 16 KiB
constexpr int kTcHalfBytes = kTcTileBytes / 2;
constexpr int kTcStages = 2;                       // streamed-tile ring
constexpr int kTcAccs = 2;                         // accumulators in tensor memory
constexpr int kTcTmemCols = kTcAccs * kTcTile;     // 256 columns
constexpr int kTcComputeWarps = 8;                 // two groups of four, one per accumulator
constexpr int kTcGroupThreads = 128;
constexpr int kTcComputeThreads = kTcComputeWarps * 32;
constexpr int kTcThreads = kTcComputeThreads + 64; // + TMA warp + MMA warp
constexpr int kTcBarGroup0 = 1;                    // named barriers: 1, 2 = the two groups; 3 = both
constexpr int kTcBarBoth = 3;

// ------------------------------------------------------------------ PTX wrappers (tcgen05, TMA tensor)

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int c0, int c1, int c2, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, M = 128, N = 128, K = 16.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// mbarrier arrives once all MMAs issued so far by this thread have completed
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread t of the warp gets lane (base + t).  The load is
// asynchronous: the registers are valid only after tmem_ld_wait on the same array.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}

// Waits for this thread's outstanding tensor-memory loads.  The array is an in/out operand so that no use
// of its registers can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                 "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]),
                 "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]),
                 "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- packed fp32x2 arithmetic (two lanes per instruction) and exp2 on the FMA pipe
typedef unsigned long long f32x2;

__device__ __forceinline__ f32x2 pack2(float a, float b) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ f32x2 pack2u(uint32_t a, uint32_t b) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float &a, float &b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// 2^x for a pair of x <= 0 without the exponential unit: x = n + f with n the nearest integer (magic-number
// rounding) and f in [-1/2, 1/2]; 2^f by a degree-4 polynomial (max relative error 2.7e-6, mean error 4e-8);
// the integer n is then added to the exponent field.  x is clamped at -125 (results below 2^-125 are noise
// for the sums they enter).
__device__ __forceinline__ f32x2 exp2_poly2(f32x2 x2) {
  float xa, xb;
  unpack2(x2, xa, xb);
  x2 = pack2(fmaxf(xa, -125.f), fmaxf(xb, -125.f));
  const f32x2 magic = pack2(12582912.f, 12582912.f);  // 1.5 * 2^23: the low mantissa bits hold n
  const f32x2 t2 = add2(x2, magic);
  const f32x2 n2 = add2(t2, pack2(-12582912.f, -12582912.f));
  const f32x2 f2 = fma2(n2, pack2(-1.f, -1.f), x2);
  f32x2 p2 = fma2(f2, pack2(0.009570101276040077f, 0.009570101276040077f),
                  pack2(0.05591785907745361f, 0.05591785907745361f));
  p2 = fma2(p2, f2, pack2(0.240247443318367f, 0.240247443318367f));
  p2 = fma2(p2, f2, pack2(0.6931217908859253f, 0.6931217908859253f));
  p2 = fma2(p2, f2, pack2(0.9999992847442627f, 0.9999992847442627f));
  float ta, tb, pa, pb;
  unpack2(t2, ta, tb);
  unpack2(p2, pa, pb);
  const uint32_t ra = __float_as_uint(pa) + (__float_as_uint(ta) << 23);
  const uint32_t rb = __float_as_uint(pb) + (__float_as_uint(tb) << 23);
  return pack2u(ra, rb);
}

__device__ __forceinline__ f32x2 exp2_mufu2(f32x2 x2) {
  float xa, xb;
  unpack2(x2, xa, xb);
  return pack2(ex2_approx(xa), ex2_approx(xb));
}

// Of every 8 pairs, how many take the polynomial instead of the exponential unit (which is the bottleneck
// of both passes: 16 results per cycle per SM against 128 FMA lanes).
#ifndef ROCO_POLY_PAIRS_PER_8
#define ROCO_POLY_PAIRS_PER_8 2
#endif
constexpr int kPolyPairsPer8 = ROCO_POLY_PAIRS_PER_8;

__device__ __forceinline__ f32x2 exp2_pair(f32x2 x2, int pair_index) {
  return ((pair_index & 7) < kPolyPairsPer8) ? exp2_poly2(x2) : exp2_mufu2(x2);
}

// Shared-memory matrix descriptor of a K-major bf16 operand tile stored as rows of 128 bytes with the
// 128-byte swizzle (what TMA writes for a 64-column box): 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(const void *p) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_u32(p) >> 4) & 0x3fffu);  // start address, 16-byte units
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                         // 128-byte swizzle
  return d;
}

// kind::f16 instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = 128
constexpr uint32_t kIdescBf16M128N128 = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

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
  char *p = (char *)align_up((size_t)raw, 1024);  // swizzle atoms are 1024-byte aligned
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
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const bool ok = !kMasked || (col0 + c * 32 + i <= grow);
              cmax = fmaxf(cmax, ok ? __uint_as_float(r[i]) : -INFINITY);
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
static bool make_map(CUtensorMap *map, const void *base, int U, int Lmax) {
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
                                    cudaStream_t stream) {
  CUtensorMap mapQ, mapK;
  const int U = S * G;
  if (!make_map(&mapQ, Q, U, Lmax) || !make_map(&mapK, K, U, Lmax)) return ROCO_ERR_CUDA;
  const int T = (maxlen + kTcTile - 1) / kTcTile;
  const int npairs = (T + 1) / 2;
  const unsigned grid = (unsigned)U * (unsigned)npairs;
  cudaError_t err = cudaFuncSetAttribute(prefill_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kTcSmemBytes);
  if (err == cudaSuccess)
    err = cudaFuncSetAttribute(prefill_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemBytes);
  if (err != cudaSuccess) return ROCO_ERR_CUDA;
  prefill_tc_kernel<0><<<grid, kTcThreads, kTcSmemBytes, stream>>>(mapQ, mapK, lens_dev, G, Lmax, npairs, scale, lse,
                                                                  s_full, q_full, status);
  prefill_tc_kernel<1><<<grid, kTcThreads, kTcSmemBytes, stream>>>(mapQ, mapK, lens_dev, G, Lmax, npairs, scale, lse,
                                                                  s_full, q_full, status);
  return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
