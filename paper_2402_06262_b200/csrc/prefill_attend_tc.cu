// Causal attention output of the prompt pass (Eq. 1 with the mask of Sec. 2.1) on the 5th-generation tensor
// cores, bf16, d = 128:   out_i = sum_{j<=i} P_ij V_j,   P_ij = exp(scale Q_i.K_j - lse_i),
// with the row log-sum-exp lse that the statistics pass produced, so that no running maximum and no rescaling
// of the output accumulator is needed.
//
// A CTA works on 256 query rows at a time (two 128-row query tiles h = 0, 1 that share every key/value tile it
// streams, which halves the L2 traffic per product) and owns the 256-row blocks (a, T2-1-a), so that every CTA
// does about the same number of tile products under the causal mask.  Per query tile and 128-key tile j:
//   S_h  = Q_h K_j^T    operands in shared memory as TMA wrote them (K-major)       -> tensor memory, fp32
//   P_h  = exp(...)     softmax group h (four warps, one query row per thread) reads S_h and writes P_h as
//                       bf16 over the columns S_h occupied
//   O_h += P_h V_j      A operand from tensor memory, V_j from shared memory as an MN-major operand
// Tensor memory holds S_0 | S_1 | O_0 | O_1 (4 x 128 columns).  Warp 8 issues TMA (K ring and V ring), warp 9
// issues the contractions in the order PV_0(j-1), S_0(j), PV_1(j-1), S_1(j): the products of one query tile
// run while the other tile's exponentials are computed.  S_h(j) follows PV_h(j-1) in the issue order of one
// thread, and the tensor pipe executes one thread's contractions in that order, so P_h(j-1) is read before S_h(j)
// overwrites it.
#include <cuda.h>
#include <cuda_bf16.h>

#include <type_traits>

#include "common.cuh"
#include "launch.h"
#include "tc.cuh"

namespace roco {

constexpr int kAtKStages = 2;                       // ring of K tiles
constexpr int kAtVStages = 3;                       // ring of V tiles
constexpr int kAtTmemCols = 512;                    // S0 | S1 | O0 | O1
constexpr int kAtColO = 2 * kTcTile;
constexpr int kAtComputeWarps = 8;
constexpr int kAtThreads = kAtComputeWarps * 32 + 64;
// Of every 8 pairs of exponentials, how many run on the FMA pipe (polynomial) instead of the exponential unit.
// Here two contractions stand against each tile's exponentials, so the exponential unit is not the limit and
// the cheaper instruction sequence wins (measured: 0 -> 1043, 1 -> 1009, 2 -> 997 TFLOP/s executed).
#ifndef ROCO_ATTEND_POLY_PAIRS_PER_8
#define ROCO_ATTEND_POLY_PAIRS_PER_8 0
#endif
constexpr int kAtPolyPairsPer8 = ROCO_ATTEND_POLY_PAIRS_PER_8;

// V_j as the B operand of O += P V_j: B[n][k] = V[key k][dim n] with the dimension index contiguous
// (MN-major).  The tile sits as two halves of 64 dims, each 128 rows (keys) of 128 bytes, 128-byte swizzle:
// 8-key groups are 1024 bytes apart (stride offset), the second 64-dim block is one half further (leading
// offset).
constexpr uint32_t kIdescPV = kIdescBf16M128N128 | (1u << 16);  // B operand MN-major

// D[tmem] (+)= A[tmem] * B[smem]: A is 128 lanes (rows) x 8 columns of packed bf16 pairs (K = 16)
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}



struct AtSmem {
  char *qt;     // two query tiles
  char *kt;     // kAtKStages key tiles
  char *vt;     // kAtVStages value tiles
  uint64_t *q_full, *q_empty;
  uint64_t *k_full, *k_empty;  // [kAtKStages]
  uint64_t *v_full, *v_empty;  // [kAtVStages]
  uint64_t *s_full, *p_full;   // [2] per query tile
  uint64_t *o_full, *o_empty;  // [2]
  uint32_t *tmem_base;
  int *abort_flag;
};

constexpr int kAtBarriers = 2 + 2 * kAtKStages + 2 * kAtVStages + 8;
constexpr size_t kAtSmemBytes = 1024 + (size_t)kTcTileBytes * (2 + kAtKStages + kAtVStages) + kAtBarriers * 8 + 16;

__device__ inline AtSmem at_carve(char *raw) {
  AtSmem m;
  char *p = smem_align(raw, 1024);
  m.qt = p; p += 2 * kTcTileBytes;
  m.kt = p; p += (size_t)kAtKStages * kTcTileBytes;
  m.vt = p; p += (size_t)kAtVStages * kTcTileBytes;
  m.q_full = (uint64_t *)p; p += 8;
  m.q_empty = (uint64_t *)p; p += 8;
  m.k_full = (uint64_t *)p; p += 8 * kAtKStages;
  m.k_empty = (uint64_t *)p; p += 8 * kAtKStages;
  m.v_full = (uint64_t *)p; p += 8 * kAtVStages;
  m.v_empty = (uint64_t *)p; p += 8 * kAtVStages;
  m.s_full = (uint64_t *)p; p += 16;
  m.p_full = (uint64_t *)p; p += 16;
  m.o_full = (uint64_t *)p; p += 16;
  m.o_empty = (uint64_t *)p; p += 16;
  m.tmem_base = (uint32_t *)p; p += 8;
  m.abort_flag = (int *)p;
  return m;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

// kOnline: a row is moved to a new reference when the sum of one 32-column chunk of its unnormalised
// probabilities 2^(z - reference) reaches 2^60 (or is not finite).  Up to there bf16 and fp32 hold the values with
// their full relative precision, and whatever an fp32 sum drops beside such a term is below its last bit anyway.
constexpr float kAtRescaleLimit = 1152921504606846976.f;  // 2^60

// kOnline = false: the row log-sum-exp comes from `lse_in` (computed earlier for the same Q, K).
// kOnline = true:  one sweep yields both: every softmax thread keeps a reference maximum m and the running sum
//   l = sum_j 2^(z_j - m) of its query row (m = the maximum over the row's first key tile, to begin with); P =
//   2^(z - m) goes to the output contraction unnormalised; when a chunk of P grows past kAtRescaleLimit, m moves to
//   that chunk's maximum and the row of the output accumulator, l and the part of the current P tile already
//   written are scaled by 2^(m_old - m_new) (the accumulator is idle at
//   that point: S_h(j) complete implies PV_h(j-1) complete, and PV_h(j) is issued only after this thread's
//   arrival).  At the end out = O / l and lse = (m + log2 l) ln 2 is written to `lse_out`.  Needs scale > 0.
template <bool kOnline>
__global__ void __launch_bounds__(kAtThreads, 1)
    prefill_attend_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                             const __grid_constant__ CUtensorMap mapV, const int *lens, int G, int Lmax, int npairs,
                             float scale, const float *lse_in, float *lse_out, __nv_bfloat16 *out, int *status) {
  extern __shared__ char at_smem_raw[];
  const AtSmem sm = at_carve(at_smem_raw);
  volatile int *abort_flag = sm.abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int u = blockIdx.x / npairs, pair = blockIdx.x % npairs;
  const int L = lens[u / G];
  const int T = (L + kTcTile - 1) / kTcTile;  // 128-row tiles
  const int T2 = (T + 1) / 2;                 // 256-row blocks
  const int a0 = pair, a1 = T2 - 1 - pair;
  const int n_tasks = (a0 > a1) ? 0 : (a0 == a1 ? 1 : 2);
  if (n_tasks == 0) return;

  if (tid == 0) {
    mbar_init(sm.q_full, 1);
    mbar_init(sm.q_empty, 1);
    for (int i = 0; i < kAtKStages; ++i) { mbar_init(&sm.k_full[i], 1); mbar_init(&sm.k_empty[i], 1); }
    for (int i = 0; i < kAtVStages; ++i) { mbar_init(&sm.v_full[i], 1); mbar_init(&sm.v_empty[i], 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sm.s_full[i], 1);
      mbar_init(&sm.p_full[i], 4);
      mbar_init(&sm.o_full[i], 1);
      mbar_init(&sm.o_empty[i], 4);
    }
    *sm.abort_flag = 0;
    mbar_init_fence();
  }
  if (warp == 0) {
    tmem_alloc(sm.tmem_base, kAtTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *sm.tmem_base;

  // Task k works on the 256-row block A: query tiles 2A (h = 0) and 2A+1 (h = 1, if it exists); key tiles
  // 0 .. 2A + nq - 1; query tile h takes part in key tile j while j <= 2A + h.
  auto task_block = [&](int k) { return k == 0 ? a0 : a1; };
  auto task_nq = [&](int A) { return (2 * A + 1 < T) ? 2 : 1; };

  if (warp == kAtComputeWarps) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int gj = 0;  // key/value tiles issued so far
      for (int k = 0; k < n_tasks; ++k) {
        const int A = task_block(k), nq = task_nq(A), nj = 2 * A + nq;
        if (k > 0) mbar_wait(sm.q_empty, (k - 1) & 1, abort_flag, status);
        mbar_expect_tx(sm.q_full, nq * kTcTileBytes);
        for (int h = 0; h < nq; ++h) {
          tma_load_3d(sm.qt + h * kTcTileBytes, &mapQ, 0, (2 * A + h) * kTcTile, u, sm.q_full);
          tma_load_3d(sm.qt + h * kTcTileBytes + kTcHalfBytes, &mapQ, 64, (2 * A + h) * kTcTile, u, sm.q_full);
        }
        for (int j = 0; j < nj; ++j, ++gj) {
          const int ks = gj % kAtKStages, vs = gj % kAtVStages;
          if (gj >= kAtKStages) mbar_wait(&sm.k_empty[ks], ((gj / kAtKStages) - 1) & 1, abort_flag, status);
          char *kd = sm.kt + (size_t)ks * kTcTileBytes;
          mbar_expect_tx(&sm.k_full[ks], kTcTileBytes);
          tma_load_3d(kd, &mapK, 0, j * kTcTile, u, &sm.k_full[ks]);
          tma_load_3d(kd + kTcHalfBytes, &mapK, 64, j * kTcTile, u, &sm.k_full[ks]);
          if (gj >= kAtVStages) mbar_wait(&sm.v_empty[vs], ((gj / kAtVStages) - 1) & 1, abort_flag, status);
          char *vd = sm.vt + (size_t)vs * kTcTileBytes;
          mbar_expect_tx(&sm.v_full[vs], kTcTileBytes);
          tma_load_3d(vd, &mapV, 0, j * kTcTile, u, &sm.v_full[vs]);
          tma_load_3d(vd + kTcHalfBytes, &mapV, 64, j * kTcTile, u, &sm.v_full[vs]);
        }
      }
    }
  } else if (warp == kAtComputeWarps + 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int gj0 = 0;                 // key tiles of earlier tasks
      int ns[2] = {0, 0};          // S products issued per query tile (= P tiles expected)
      for (int k = 0; k < n_tasks; ++k) {
        const int A = task_block(k), nq = task_nq(A), nj = 2 * A + nq;
        auto active = [&](int h, int j) { return h < nq && j >= 0 && j < nj && j <= 2 * A + h; };
        auto last_user = [&](int h, int j) { return !active(h + 1, j); };  // h is the last query tile using tile j
        int np[2] = {ns[0], ns[1]};  // P tiles consumed per query tile
        mbar_wait(sm.q_full, k & 1, abort_flag, status);
        for (int j = 0; j <= nj; ++j) {
          for (int h = 0; h < 2; ++h) {
            if (active(h, j - 1)) {  // O_h += P_h V_{j-1}
              const int gj = gj0 + j - 1, vs = gj % kAtVStages;
              if (h == 0 || !active(0, j - 1)) mbar_wait(&sm.v_full[vs], (gj / kAtVStages) & 1, abort_flag, status);
              mbar_wait(&sm.p_full[h], np[h] & 1, abort_flag, status);
              ++np[h];
              if (j - 1 == 0 && k > 0) mbar_wait(&sm.o_empty[h], (k - 1) & 1, abort_flag, status);
              tc_fence_after();
              const char *vt = sm.vt + (size_t)vs * kTcTileBytes;
#pragma unroll
              for (int kk = 0; kk < kTcTile / 16; ++kk)  // 16 keys per instruction
                umma_bf16_ts(tmem + (uint32_t)(kAtColO + h * kTcTile), tmem + (uint32_t)(h * kTcTile + kk * 8),
                             smem_desc_sw128_mn(vt + kk * 2048, kTcHalfBytes), kIdescPV, (kk > 0 || j - 1 > 0) ? 1u : 0u);
              if (last_user(h, j - 1)) umma_commit(&sm.v_empty[vs]);
              if (!active(h, j)) umma_commit(&sm.o_full[h]);  // that was this query tile's last key tile
            }
            if (active(h, j)) {  // S_h = Q_h K_j^T
              const int gj = gj0 + j, ks = gj % kAtKStages;
              if (h == 0 || !active(0, j)) mbar_wait(&sm.k_full[ks], (gj / kAtKStages) & 1, abort_flag, status);
              tc_fence_after();
              const char *kt = sm.kt + (size_t)ks * kTcTileBytes;
              const char *qt = sm.qt + h * kTcTileBytes;
#pragma unroll
              for (int kk = 0; kk < kTcD / 16; ++kk) {
                const int off = (kk / 4) * kTcHalfBytes + (kk % 4) * 32;
                umma_bf16(tmem + (uint32_t)(h * kTcTile), smem_desc_sw128(qt + off), smem_desc_sw128(kt + off),
                          kIdescBf16M128N128, kk > 0 ? 1u : 0u);
              }
              umma_commit(&sm.s_full[h]);
              ++ns[h];
              if (last_user(h, j)) umma_commit(&sm.k_empty[ks]);
              if (j == nj - 1 && last_user(h, j)) umma_commit(sm.q_empty);  // the task's last S product
            }
          }
        }
        gj0 += nj;
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps
    const float zscale = scale * kLog2e;
    const int h = warp >> 2;                 // the query tile this group serves
    const int row = (warp & 3) * 32 + lane;  // TMEM lane = query row inside the tile
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t taddr = tmem + lane_addr + (uint32_t)(h * kTcTile);
    int gj0 = 0, mine = 0;
    for (int k = 0; k < n_tasks; ++k) {
      const int A = task_block(k), nq = task_nq(A), nj = 2 * A + nq;
      if (h < nq) {
        const int a = 2 * A + h;  // this group's 128-row query tile; its diagonal key tile
        const int grow = a * kTcTile + row;
        float nl2 = 0.f, m_ref = -INFINITY, lsum = 0.f;
        if constexpr (!kOnline) nl2 = (grow < L) ? -lse_in[(size_t)u * Lmax + grow] * kLog2e : 0.f;
        f32x2 nl22 = pack2(nl2, nl2);
        const f32x2 zs2 = pack2(zscale, zscale);
        const uint32_t oaddr = tmem + lane_addr + (uint32_t)(kAtColO + h * kTcTile);
        for (int j = 0; j <= a; ++j, ++mine) {
          mbar_wait(&sm.s_full[h], mine & 1, abort_flag, status);
          tc_fence_after();
          const int col0 = j * kTcTile;
          uint32_t ra[32], rb[32];
          if constexpr (kOnline) {
            if (j == 0) {  // the row's reference maximum starts as the maximum over its first key tile
              float mx = -INFINITY;
#pragma unroll 1
              for (int c = 0; c < 4; ++c) {
                tmem_ld32_issue(taddr + c * 32, ra);
                tmem_ld_wait(ra);
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  mx = fmaxf(mx, (a > 0 || c * 32 + i <= grow) ? __uint_as_float(ra[i]) : -INFINITY);
              }
              m_ref = mx * zscale;
              nl22 = pack2(-m_ref, -m_ref);
            }
          }
          // kOnline: move the row's reference maximum up to `cz` (where `need`) before chunk c of this tile
          auto rescale_row = [&](int c, bool need, float cz) {
            const float m_new = need ? cz : m_ref;
            const float f = need ? exp2f(m_ref - m_new) : 1.f;
            lsum *= f;
            uint32_t t16[16];
#pragma unroll 1
            for (int cc = 0; cc < kTcD / 16; ++cc) {  // the output accumulator's row (j > 0 here: it is valid)
              tmem_ld16(oaddr + cc * 16, t16);
#pragma unroll
              for (int i = 0; i < 16; ++i) t16[i] = __float_as_uint(__uint_as_float(t16[i]) * f);
              tmem_st16(oaddr + cc * 16, t16);
            }
#pragma unroll 1
            for (int c2 = 0; c2 < c; ++c2) {  // the chunks of this tile's P written so far (packed bf16 pairs)
              tmem_ld16(taddr + c2 * 16, t16);
#pragma unroll
              for (int i = 0; i < 16; ++i)
                t16[i] = pack_bf16x2(__uint_as_float(t16[i] << 16) * f, __uint_as_float(t16[i] & 0xffff0000u) * f);
              tmem_st16(taddr + c2 * 16, t16);
            }
            tmem_st_wait();
            m_ref = m_new;
            nl22 = pack2(-m_ref, -m_ref);
          };

          auto chunk = [&](const uint32_t (&r)[32], int c, auto masked_tag) {
            constexpr bool kMasked = decltype(masked_tag)::value;
            uint32_t pk[16];
            float ls = 0.f;
            // P of the chunk against the current reference (packed bf16 pairs in pk, their fp32 sum in ls)
            auto exponentials = [&]() {
              ls = 0.f;
              [[maybe_unused]] f32x2 ls2 = pack2(0.f, 0.f);
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                f32x2 p2 = ((i >> 1) & 7) < kAtPolyPairsPer8 ? exp2_poly2(fma2(pack2u(r[i], r[i + 1]), zs2, nl22))
                                                           : exp2_mufu2(fma2(pack2u(r[i], r[i + 1]), zs2, nl22));
                float pa, pb;
                unpack2(p2, pa, pb);
                if (kMasked) {
                  const int kj = col0 + c * 32 + i;
                  pa = (kj <= grow) ? pa : 0.f;
                  pb = (kj + 1 <= grow) ? pb : 0.f;
                }
                if constexpr (kOnline) {
                  if constexpr (kMasked) ls += pa + pb; else ls2 = add2(ls2, p2);
                }
                pk[i >> 1] = pack_bf16x2(pa, pb);
              }
              if constexpr (kOnline) {
                float la, lb;
                unpack2(ls2, la, lb);
                ls += la + lb;
              }
            };
            if constexpr (!kOnline) {
              exponentials();
            } else {
              // No maximum is formed ahead of the exponentials: a score far above the row's reference shows in
              // the chunk's sum (beyond 2^kAtRescaleLog2, or not finite).  Only then is the chunk's maximum
              // taken, the row moved to it, and the chunk done again -- once, since its maximum is then the
              // reference.
#pragma unroll 1
              for (int pass = 0; pass < 2; ++pass) {
                exponentials();
                const bool need = !(ls < kAtRescaleLimit);
                if (pass == 1 || j == 0 || !__any_sync(0xffffffffu, need)) break;
                float cm = -INFINITY;
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  cm = fmaxf(cm, (!kMasked || col0 + c * 32 + i <= grow) ? __uint_as_float(r[i]) : -INFINITY);
                rescale_row(c, need, cm * zscale);
              }
              lsum += ls;
            }
            tmem_st16(taddr + c * 16, pk);  // behind the columns already read
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
            chunk(rb, 3, masked_tag);
          };
          if (j == a) tile(std::true_type{}); else tile(std::false_type{});
          // value rows past the prompt may hold anything (0 x NaN would poison every query): clear them.
          // Only the last key tile of the prompt has such rows, and only one query tile ever reaches it.
          if (j == T - 1 && col0 + row >= L) {
            const int gj = gj0 + j, vs = gj % kAtVStages;
            mbar_wait(&sm.v_full[vs], (gj / kAtVStages) & 1, abort_flag, status);
            char *vrow = sm.vt + (size_t)vs * kTcTileBytes + row * 128;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              *reinterpret_cast<uint4 *>(vrow + i * 16) = make_uint4(0, 0, 0, 0);
              *reinterpret_cast<uint4 *>(vrow + kTcHalfBytes + i * 16) = make_uint4(0, 0, 0, 0);
            }
            fence_async_smem();  // generic-proxy writes -> visible to the tensor core's reads
          }
          tmem_st_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.p_full[h]);
        }
        // the finished output accumulator of this query tile: one row per thread
        mbar_wait(&sm.o_full[h], k & 1, abort_flag, status);
        tc_fence_after();
        uint32_t r[32];
        float inv = 1.f;
        if constexpr (kOnline) {
          inv = 1.f / lsum;
          if (grow < L) lse_out[(size_t)u * Lmax + grow] = (m_ref + log2f(lsum)) * kLn2;
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          tmem_ld32_issue(oaddr + c * 32, r);
          tmem_ld_wait(r);
          if constexpr (kOnline) {
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * inv);
          }
          if (grow < L) {
            uint4 *dst = reinterpret_cast<uint4 *>(out + ((size_t)u * Lmax + grow) * kTcD + c * 32);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              dst[i] = make_uint4(pack_bf16x2(__uint_as_float(r[8 * i]), __uint_as_float(r[8 * i + 1])),
                                  pack_bf16x2(__uint_as_float(r[8 * i + 2]), __uint_as_float(r[8 * i + 3])),
                                  pack_bf16x2(__uint_as_float(r[8 * i + 4]), __uint_as_float(r[8 * i + 5])),
                                  pack_bf16x2(__uint_as_float(r[8 * i + 6]), __uint_as_float(r[8 * i + 7])));
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.o_empty[h]);
      }
      gj0 += nj;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kAtTmemCols);
}

roco_status launch_prefill_attend_tc(int S, int G, int Lmax, const int *lens_dev, int maxlen, const void *Q,
                                     const void *K, const void *V, float scale, const float *lse_in, float *lse_out,
                                     void *out, int *status, cudaStream_t stream) {
  CUtensorMap mapQ, mapK, mapV;
  const int U = S * G;
  if (!make_tensor_map_prompt_bf16(&mapQ, Q, U, Lmax) || !make_tensor_map_prompt_bf16(&mapK, K, U, Lmax) ||
      !make_tensor_map_prompt_bf16(&mapV, V, U, Lmax))
    return ROCO_ERR_CUDA;
  const int T = (maxlen + kTcTile - 1) / kTcTile;
  const int T2 = (T + 1) / 2;
  const int npairs = (T2 + 1) / 2;
  const unsigned grid = (unsigned)U * (unsigned)npairs;
  auto launch = [&](auto kernel) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAtSmemBytes) != cudaSuccess)
      return ROCO_ERR_CUDA;
    kernel<<<grid, kAtThreads, kAtSmemBytes, stream>>>(mapQ, mapK, mapV, lens_dev, G, Lmax, npairs, scale, lse_in,
                                                      lse_out, static_cast<__nv_bfloat16 *>(out), status);
    return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
  };
  // lse_in given: the output alone from a known row log-sum-exp; else one sweep that also produces lse_out
  return lse_in ? launch(prefill_attend_tc_kernel<false>) : launch(prefill_attend_tc_kernel<true>);
}

}  // namespace roco
