// Causal attention output of the prompt pass (Eq. 1 with the mask of Sec. 2.1) on the 5th-generation tensor
// cores, bf16, d = 128:   out_i = sum_{j<=i} P_ij V_j,   P_ij = exp(scale Q_i.K_j - lse_i),
// with the row log-sum-exp lse that the statistics pass produced, so that no running maximum and no rescaling
// of the output accumulator is needed.  Per 128 x 128 tile two contractions:
//   S = Q_a K_j^T       (both operands K-major, as TMA wrote them)           -> tensor memory, fp32
//   O += P V_j          (P: bf16, written by the softmax warps into a swizzled K-major tile;
//                        V_j: the TMA tile as it is, read as an MN-major operand) -> tensor memory, fp32
// A CTA owns the query tiles (a, T-1-a) like the statistics passes.  Warps 0-7 turn S into P (two groups of four,
// one per S accumulator), warp 8 issues TMA, warp 9 issues both contractions; the S product of tile j+1 is
// issued before the P V product of tile j so that the tensor pipe works while the exponentials run.
#include <cuda.h>
#include <cuda_bf16.h>

#include <type_traits>

#include "common.cuh"
#include "launch.h"
#include "tc.cuh"

namespace roco {

constexpr int kAtStages = 2;                        // ring of (K_j, V_j) tile pairs
constexpr int kAtStageBytes = 2 * kTcTileBytes;     // 64 KiB
constexpr int kAtTmemCols = 512;                    // S0 | S1 | O | unused (allocations are powers of two)
constexpr int kAtColO = 2 * kTcTile;
constexpr int kAtComputeWarps = 8;
constexpr int kAtThreads = kAtComputeWarps * 32 + 64;

// V_j as the B operand of O += P V_j: B[n][k] = V[key k][dim n] with the dimension index contiguous
// (MN-major).  The tile sits as two halves of 64 dims, each 128 rows (keys) of 128 bytes, 128-byte swizzle:
// 8-key groups are 1024 bytes apart (stride offset), the second 64-dim block is one half further (leading
// offset).
__device__ __forceinline__ uint64_t smem_desc_sw128_mn(const void *p) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_u32(p) >> 4) & 0x3fffu);
  d |= (uint64_t)(kTcHalfBytes >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

constexpr uint32_t kIdescPV = kIdescBf16M128N128 | (1u << 16);  // B operand MN-major

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

struct AtSmem {
  char *qt;     // query tile
  char *ring;   // kAtStages x (K tile, V tile)
  char *pt;     // probability tile, bf16, K-major, swizzled like a TMA tile
  uint64_t *q_full, *q_empty;
  uint64_t *ring_full, *ring_empty;  // [kAtStages]
  uint64_t *acc_full, *acc_empty;    // [2]
  uint64_t *p_full, *p_empty, *o_full, *o_empty;
  uint32_t *tmem_base;
  int *abort_flag;
};

constexpr size_t kAtSmemBytes = 1024 + (size_t)kTcTileBytes * 2 + (size_t)kAtStages * kAtStageBytes + 16 * 8 + 16;

__device__ inline AtSmem at_carve(char *raw) {
  AtSmem m;
  char *p = (char *)align_up((size_t)raw, 1024);
  m.qt = p; p += kTcTileBytes;
  m.ring = p; p += (size_t)kAtStages * kAtStageBytes;
  m.pt = p; p += kTcTileBytes;
  m.q_full = (uint64_t *)p; p += 8;
  m.q_empty = (uint64_t *)p; p += 8;
  m.ring_full = (uint64_t *)p; p += 8 * kAtStages;
  m.ring_empty = (uint64_t *)p; p += 8 * kAtStages;
  m.acc_full = (uint64_t *)p; p += 16;
  m.acc_empty = (uint64_t *)p; p += 16;
  m.p_full = (uint64_t *)p; p += 8;
  m.p_empty = (uint64_t *)p; p += 8;
  m.o_full = (uint64_t *)p; p += 8;
  m.o_empty = (uint64_t *)p; p += 8;
  m.tmem_base = (uint32_t *)p; p += 8;
  m.abort_flag = (int *)p;
  return m;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

__global__ void __launch_bounds__(kAtThreads, 1)
    prefill_attend_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                             const __grid_constant__ CUtensorMap mapV, const int *lens, int G, int Lmax, int npairs,
                             float scale, const float *lse, __nv_bfloat16 *out, int *status) {
  extern __shared__ char at_smem_raw[];
  const AtSmem sm = at_carve(at_smem_raw);
  volatile int *abort_flag = sm.abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int u = blockIdx.x / npairs, pair = blockIdx.x % npairs;
  const int L = lens[u / G];
  const int T = (L + kTcTile - 1) / kTcTile;
  const int a0 = pair, a1 = T - 1 - pair;
  const int n_tasks = (a0 > a1) ? 0 : (a0 == a1 ? 1 : 2);
  if (n_tasks == 0) return;

  if (tid == 0) {
    mbar_init(sm.q_full, 1);
    mbar_init(sm.q_empty, 1);
    for (int i = 0; i < kAtStages; ++i) { mbar_init(&sm.ring_full[i], 1); mbar_init(&sm.ring_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sm.acc_full[i], 1); mbar_init(&sm.acc_empty[i], 4); }
    mbar_init(sm.p_full, 4);
    mbar_init(sm.p_empty, 1);
    mbar_init(sm.o_full, 1);
    mbar_init(sm.o_empty, 4);
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

  auto task_tile = [&](int k) { return k == 0 ? a0 : a1; };  // query tile a streams key tiles 0..a
  const int n_tiles = (a0 + 1) + (n_tasks == 2 ? a1 + 1 : 0);

  if (warp == kAtComputeWarps) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int g = 0;
      for (int k = 0; k < n_tasks; ++k) {
        const int a = task_tile(k);
        if (k > 0) mbar_wait(sm.q_empty, (k - 1) & 1, abort_flag, status);
        mbar_expect_tx(sm.q_full, kTcTileBytes);
        tma_load_3d(sm.qt, &mapQ, 0, a * kTcTile, u, sm.q_full);
        tma_load_3d(sm.qt + kTcHalfBytes, &mapQ, 64, a * kTcTile, u, sm.q_full);
        for (int j = 0; j <= a; ++j, ++g) {
          const int st = g % kAtStages;
          if (g >= kAtStages) mbar_wait(&sm.ring_empty[st], ((g / kAtStages) - 1) & 1, abort_flag, status);
          char *kd = sm.ring + (size_t)st * kAtStageBytes, *vd = kd + kTcTileBytes;
          mbar_expect_tx(&sm.ring_full[st], kAtStageBytes);
          tma_load_3d(kd, &mapK, 0, j * kTcTile, u, &sm.ring_full[st]);
          tma_load_3d(kd + kTcHalfBytes, &mapK, 64, j * kTcTile, u, &sm.ring_full[st]);
          tma_load_3d(vd, &mapV, 0, j * kTcTile, u, &sm.ring_full[st]);
          tma_load_3d(vd + kTcHalfBytes, &mapV, 64, j * kTcTile, u, &sm.ring_full[st]);
        }
      }
    }
  } else if (warp == kAtComputeWarps + 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // tile g of the CTA: its task and whether it opens / closes the task
      auto first_of = [&](int g) { return g == 0 || g == a0 + 1; };
      auto last_of = [&](int g) { return g == a0 || g == n_tiles - 1; };
      auto task_of = [&](int g) { return g <= a0 ? 0 : 1; };
      auto issue_s = [&](int g) {  // S = Q K_j^T into accumulator g & 1
        const int st = g % kAtStages, ac = g & 1;
        if (first_of(g)) mbar_wait(sm.q_full, task_of(g) & 1, abort_flag, status);
        mbar_wait(&sm.ring_full[st], (g / kAtStages) & 1, abort_flag, status);
        if (g >= 2) mbar_wait(&sm.acc_empty[ac], ((g >> 1) - 1) & 1, abort_flag, status);
        tc_fence_after();
        const char *kt = sm.ring + (size_t)st * kAtStageBytes;
#pragma unroll
        for (int kk = 0; kk < kTcD / 16; ++kk) {
          const int off = (kk / 4) * kTcHalfBytes + (kk % 4) * 32;
          umma_bf16(tmem + (uint32_t)(ac * kTcTile), smem_desc_sw128(sm.qt + off), smem_desc_sw128(kt + off),
                    kIdescBf16M128N128, kk > 0 ? 1u : 0u);
        }
        umma_commit(&sm.acc_full[ac]);
        if (last_of(g)) umma_commit(sm.q_empty);
      };
      auto issue_pv = [&](int g) {  // O += P V_j
        const int st = g % kAtStages;
        mbar_wait(sm.p_full, g & 1, abort_flag, status);
        if (first_of(g) && task_of(g) > 0) mbar_wait(sm.o_empty, (task_of(g) - 1) & 1, abort_flag, status);
        tc_fence_after();
        const char *vt = sm.ring + (size_t)st * kAtStageBytes + kTcTileBytes;
#pragma unroll
        for (int kk = 0; kk < kTcTile / 16; ++kk) {  // 16 keys per instruction
          const int poff = (kk / 4) * kTcHalfBytes + (kk % 4) * 32;
          umma_bf16(tmem + (uint32_t)kAtColO, smem_desc_sw128(sm.pt + poff), smem_desc_sw128_mn(vt + kk * 2048),
                    kIdescPV, (kk > 0 || !first_of(g)) ? 1u : 0u);
        }
        umma_commit(&sm.ring_empty[st]);
        umma_commit(sm.p_empty);
        if (last_of(g)) umma_commit(sm.o_full);
      };
      issue_s(0);
      for (int g = 0; g < n_tiles; ++g) {
        if (g + 1 < n_tiles) issue_s(g + 1);
        issue_pv(g);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps
    const float zscale = scale * kLog2e;
    const int group = warp >> 2;
    const int row = (warp & 3) * 32 + lane;  // TMEM lane = query row inside the tile
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t taddr = tmem + lane_addr + (uint32_t)(group * kTcTile);
    char *prow = sm.pt + row * 128;
    const int sw = row & 7;
    int g0 = 0, mine = 0;
    for (int k = 0; k < n_tasks; ++k) {
      const int a = task_tile(k);
      const int grow = a * kTcTile + row;
      const float nl2 = (grow < L) ? -lse[(size_t)u * Lmax + grow] * kLog2e : 0.f;
      const f32x2 nl22 = pack2(nl2, nl2), zs2 = pack2(zscale, zscale);
      const int t0 = ((g0 & 1) == group) ? 0 : 1;
      for (int j = t0; j <= a; j += 2, ++mine) {
        const int g = g0 + j;
        mbar_wait(&sm.acc_full[group], mine & 1, abort_flag, status);
        tc_fence_after();
        const int col0 = j * kTcTile;
        uint32_t ra[32], rb[32];
        bool p_free = (g == 0);

        auto chunk = [&](const uint32_t (&r)[32], int c, auto masked_tag) {
          constexpr bool kMasked = decltype(masked_tag)::value;
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            f32x2 p2 = exp2_pair(fma2(pack2u(r[i], r[i + 1]), zs2, nl22), i >> 1);
            float pa, pb;
            unpack2(p2, pa, pb);
            if (kMasked) {
              const int kj = col0 + c * 32 + i;
              pa = (kj <= grow) ? pa : 0.f;
              pb = (kj + 1 <= grow) ? pb : 0.f;
            }
            pk[i >> 1] = pack_bf16x2(pa, pb);
          }
          if (!p_free) {  // the previous tile's P V product must have read the probability tile
            mbar_wait(sm.p_empty, (g - 1) & 1, abort_flag, status);
            p_free = true;
          }
          char *half = prow + (c >> 1) * kTcHalfBytes;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int cc = (c & 1) * 4 + i;
            *reinterpret_cast<uint4 *>(half + ((cc ^ sw) << 4)) =
                make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
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
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.acc_empty[group]);
          chunk(rb, 3, masked_tag);
        };
        if (j == a) tile(std::true_type{}); else tile(std::false_type{});
        // value rows past the prompt may hold anything (0 x NaN would poison every query): clear them
        if (j == T - 1 && col0 + row >= L) {
          char *vrow = sm.ring + (size_t)(g % kAtStages) * kAtStageBytes + kTcTileBytes + row * 128;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            *reinterpret_cast<uint4 *>(vrow + i * 16) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4 *>(vrow + kTcHalfBytes + i * 16) = make_uint4(0, 0, 0, 0);
          }
        }
        fence_async_smem();  // generic-proxy writes -> visible to the tensor core's reads
        __syncwarp();
        if (lane == 0) mbar_arrive(sm.p_full);
      }
      g0 += a + 1;
      if (group == 0) {  // read the finished output accumulator: one query row per thread
        mbar_wait(sm.o_full, k & 1, abort_flag, status);
        tc_fence_after();
        const uint32_t oaddr = tmem + lane_addr + (uint32_t)kAtColO;
        uint32_t r[32];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          tmem_ld32_issue(oaddr + c * 32, r);
          tmem_ld_wait(r);
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
        if (lane == 0) mbar_arrive(sm.o_empty);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kAtTmemCols);
}

roco_status launch_prefill_attend_tc(int S, int G, int Lmax, const int *lens_dev, int maxlen, const void *Q,
                                     const void *K, const void *V, float scale, const float *lse, void *out,
                                     int *status, cudaStream_t stream) {
  CUtensorMap mapQ, mapK, mapV;
  const int U = S * G;
  if (!make_tensor_map_prompt_bf16(&mapQ, Q, U, Lmax) || !make_tensor_map_prompt_bf16(&mapK, K, U, Lmax) ||
      !make_tensor_map_prompt_bf16(&mapV, V, U, Lmax))
    return ROCO_ERR_CUDA;
  const int T = (maxlen + kTcTile - 1) / kTcTile;
  const int npairs = (T + 1) / 2;
  const unsigned grid = (unsigned)U * (unsigned)npairs;
  if (cudaFuncSetAttribute(prefill_attend_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)kAtSmemBytes) != cudaSuccess)
    return ROCO_ERR_CUDA;
  prefill_attend_tc_kernel<<<grid, kAtThreads, kAtSmemBytes, stream>>>(
      mapQ, mapK, mapV, lens_dev, G, Lmax, npairs, scale, lse, static_cast<__nv_bfloat16 *>(out), status);
  return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
