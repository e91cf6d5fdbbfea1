// Per-unit eviction-scope construction and victim choice (Sec. 4.3), done by one thread group on
// statistics that already sit in shared memory.
//
//   scope   = the m cached tokens first in (variance asc, position asc)
//   victim  = the in-scope token first in (mean asc, position asc)
//
// The rank-m threshold comes from a most-significant-digit radix select over unsigned keys (the bit
// pattern of a non-negative float or double orders like its value); ties on the threshold variance are
// resolved by a second radix select over the tied tokens' positions, only when not all of them fit in the
// scope.
#pragma once

#include "common.cuh"

namespace roco {

struct SelectScratch {
  uint32_t hist[256];
  uint32_t digit, rank, count, pad;
  float red_mean[32];
  int red_pos[32];
  int red_slot[32];
};

// Shared-memory reduction with the state space spelled out: the scratch is reached through pointers whose
// provenance the compiler cannot see, and a generic-address atomic on shared memory is far slower.
__device__ __forceinline__ void smem_red_add(uint32_t *addr, uint32_t v) {
  asm volatile("red.shared::cta.add.u32 [%0], %1;" ::"r"(smem_u32(addr)), "r"(v) : "memory");
}

// k-th smallest (0-based) of key(j) over the j in [0, n) with pred(j); keys are unsigned integers of type
// KeyT (32 or 64 bits).  Called by all `nthreads` threads that synchronise on named barrier `bar_id`.
// *rank_in_ties: how many elements equal to the result precede the k-th in a stable order (so
// rank_in_ties + 1 of them are among the k+1 smallest); *n_ties: how many elements equal the result.
// `common` (optional): bits on which all selected keys are known to agree, as (AND of the keys, OR of the keys);
// the digits above the first disagreeing one are then skipped.
template <typename KeyT, typename KeyF, typename PredF>
__device__ __forceinline__ KeyT radix_select(KeyF key, PredF pred, int n, uint32_t k, SelectScratch &sc, int tid,
                                             int nthreads, int bar_id, uint32_t *rank_in_ties, uint32_t *n_ties,
                                             KeyT all_and = 0, KeyT all_or = ~(KeyT)0) {
  KeyT prefix = 0, mask = 0;
  uint32_t kk = k;
  const int lane = tid & 31;
  int shift0 = (int)sizeof(KeyT) * 8 - 8;
  {
    const KeyT diff = all_and ^ all_or;  // a set bit: the keys may differ there
    while (shift0 > 0 && (diff >> shift0) == 0) shift0 -= 8;
    if (shift0 < (int)sizeof(KeyT) * 8 - 8) {
      mask = ~(KeyT)0 << (shift0 + 8);
      prefix = all_and & mask;
    }
  }
#pragma unroll 1
  for (int shift = shift0; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += nthreads) sc.hist[i] = 0;
    named_bar_sync(bar_id, nthreads);
#pragma unroll 4
    for (int j = tid; j < n; j += nthreads) {
      if (pred(j)) {
        const KeyT x = key(j);
        if ((x & mask) == prefix) smem_red_add(&sc.hist[(uint32_t)(x >> shift) & 255u], 1u);
      }
    }
    named_bar_sync(bar_id, nthreads);
    if (tid < 32) {
      uint32_t c[8], total = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { c[i] = sc.hist[lane * 8 + i]; total += c[i]; }
      uint32_t incl = total;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      uint32_t excl = incl - total;
      if (kk >= excl && kk < incl) {
        uint32_t rem = kk - excl;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (rem < c[i]) { sc.digit = lane * 8 + i; sc.rank = rem; sc.count = c[i]; break; }
          rem -= c[i];
        }
      }
    }
    named_bar_sync(bar_id, nthreads);
    prefix |= (KeyT)sc.digit << shift;
    mask |= (KeyT)255u << shift;
    kk = sc.rank;
  }
  *rank_in_ties = kk;
  *n_ties = sc.count;
  named_bar_sync(bar_id, nthreads);  // sc.* may be reused by the caller right away
  return prefix;
}

__device__ __forceinline__ double mean_f64(float s, int n) { return (double)s / (double)n; }

__device__ __forceinline__ double variance_f64(float s, float q, int n) {
  double mean = (double)s / (double)n;
  double var = (double)q / (double)n - mean * mean;
  return fmax(var, 0.0);  // also maps NaN to 0
}

// Decode-step keys avoid fp64 division: the variance numerator q*n - s*s is formed in fp64 (both products
// of fp32 values are exact there, so the cancellation costs nothing), then rounded to fp32 and divided by
// n*n; the mean is the fp32 quotient s/n.  Both carry a relative error of a few 1e-7 of the value itself,
// far inside the 1e-5 decision margin; equal (s, q, n) always give equal keys, so exact ties still fall to
// the position rule.
__device__ __forceinline__ uint32_t variance_key_fast(float s, float q, int n) {
  const double num = fmax((double)q * (double)n - (double)s * (double)s, 0.0);  // NaN -> 0
  const float nf = (float)n;
  return __float_as_uint(__fdiv_rn((float)num, nf * nf));
}

__device__ __forceinline__ float mean_fast(float s, int n) { return __fdiv_rn(s, (float)n); }

// AND and OR of a per-thread pair over the whole group (in place); every thread gets the group's values.
__device__ __forceinline__ void group_and_or(uint32_t &k_and, uint32_t &k_or, SelectScratch &sc, int tid, int nthreads,
                                             int bar_id) {
  k_and = __reduce_and_sync(0xffffffffu, k_and);
  k_or = __reduce_or_sync(0xffffffffu, k_or);
  const int warp = tid >> 5, nwarps = nthreads >> 5;
  if ((tid & 31) == 0) { sc.red_pos[warp] = (int)k_and; sc.red_slot[warp] = (int)k_or; }
  named_bar_sync(bar_id, nthreads);
  for (int w = 0; w < nwarps; ++w) { k_and &= (uint32_t)sc.red_pos[w]; k_or |= (uint32_t)sc.red_slot[w]; }
  named_bar_sync(bar_id, nthreads);  // the scratch may be reused right away
}

// Victim slot among slots [0, live) given scope size m (1 <= m <= live), from the keys in shared memory:
// vkey[j] = variance key, mkey[j] = mean of slot j; (k_and, k_or) = each thread's AND / OR over the variance keys it
// wrote (combined over the group here, which also publishes the keys).  pos: the unit's positions, read only
// where a tie has to be broken.  Returns -1 if no slot qualifies (NaN statistics).  Called by the `nthreads`
// threads (a multiple of 32) that synchronise on named barrier `bar_id`; every one of them gets the same value.
__device__ __forceinline__ int group_select_from_keys(const int *pos, int live, int m, const uint32_t *vkey,
                                                      const float *mkey, uint32_t k_and, uint32_t k_or,
                                                      SelectScratch &sc, int tid, int nthreads, int bar_id) {
  const int warp = tid >> 5, nwarps = nthreads >> 5;
  // (mean, position, slot) of the group's best candidate from each thread's own; every thread gets it
  auto reduce_best = [&](float &bm, int &bp, int &bs) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, bm, o);
      const int op = __shfl_xor_sync(0xffffffffu, bp, o);
      const int os = __shfl_xor_sync(0xffffffffu, bs, o);
      if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
    }
    if ((tid & 31) == 0) { sc.red_mean[warp] = bm; sc.red_pos[warp] = bp; sc.red_slot[warp] = bs; }
    named_bar_sync(bar_id, nthreads);
    bm = sc.red_mean[0]; bp = sc.red_pos[0]; bs = sc.red_slot[0];
    for (int w = 1; w < nwarps; ++w) {
      const float om = sc.red_mean[w];
      const int op = sc.red_pos[w], os = sc.red_slot[w];
      if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
    }
    named_bar_sync(bar_id, nthreads);  // the scratch may be reused right away
  };
  named_bar_sync(bar_id, nthreads);  // publishes the keys
  // A scope that leaves out only a few tokens almost always contains the token of lowest mean.  So: take the
  // tokens in (mean, position) order and test each for membership -- it is in scope iff fewer than m tokens come
  // before it in (variance, position) order -- which costs two passes over the keys per candidate where the radix
  // select below costs two per digit.  After three candidates outside the scope the radix select takes over.
  if (2 * m >= live) {
    int excl0 = -1, excl1 = -1, excl2 = -1;
#pragma unroll 1
    for (int attempt = 0; attempt < 3; ++attempt) {
      float bm = INFINITY;
      int bs = -1;
#pragma unroll 4
      for (int j = tid; j < live; j += nthreads) {
        if (j == excl0 || j == excl1 || j == excl2) continue;
        const float mean = mkey[j];
        if (mean < bm) { bm = mean; bs = j; }
        else if (mean == bm && bs >= 0 && pos[j] < pos[bs]) bs = j;
      }
      int bp = (bs >= 0) ? pos[bs] : 0x7fffffff;
      reduce_best(bm, bp, bs);
      if (bs < 0) return -1;  // no candidate left (NaN statistics)
      const uint32_t cv = vkey[bs];
      uint32_t cnt = 0;
#pragma unroll 4
      for (int j = tid; j < live; j += nthreads) {
        const uint32_t k = vkey[j];
        cnt += (k < cv || (k == cv && pos[j] < bp)) ? 1u : 0u;
      }
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      if ((tid & 31) == 0) sc.red_slot[warp] = (int)cnt;
      named_bar_sync(bar_id, nthreads);
      cnt = 0;
      for (int w = 0; w < nwarps; ++w) cnt += (uint32_t)sc.red_slot[w];
      named_bar_sync(bar_id, nthreads);
      if (cnt < (uint32_t)m) return bs;
      if (attempt == 0) excl0 = bs; else if (attempt == 1) excl1 = bs; else excl2 = bs;
    }
  }
  group_and_or(k_and, k_or, sc, tid, nthreads, bar_id);
  uint32_t T = 0xffffffffu;
  int P = 0x7fffffff;
  if (m < live) {
    uint32_t rank, ties;
    T = radix_select<uint32_t>([&](int j) { return vkey[j]; }, [&](int) { return true; }, live, (uint32_t)(m - 1),
                               sc, tid, nthreads, bar_id, &rank, &ties, k_and, k_or);
    if (ties != rank + 1) {  // only some of the tokens tied at the threshold are in scope: lowest positions
      uint32_t r2, t2;
      P = (int)radix_select<uint32_t>([&](int j) { return (uint32_t)pos[j]; }, [&](int j) { return vkey[j] == T; },
                                      live, rank, sc, tid, nthreads, bar_id, &r2, &t2);
    }
  }
  float bm = INFINITY;
  int bs = -1;
#pragma unroll 4
  for (int j = tid; j < live; j += nthreads) {
    const uint32_t k = vkey[j];
    if (k > T) continue;
    if (k == T && P != 0x7fffffff && pos[j] > P) continue;
    const float mean = mkey[j];
    if (mean < bm) { bm = mean; bs = j; }
    else if (mean == bm && bs >= 0 && pos[j] < pos[bs]) bs = j;
  }
  int bp = (bs >= 0) ? pos[bs] : 0x7fffffff;
  reduce_best(bm, bp, bs);
  return bs;
}

// The same with the keys formed here from the unit's statistics s, q, n (any memory; each read once, coalesced).
// vkey[live] and mkey[live] are shared-memory scratch.
__device__ __forceinline__ int group_select_victim(const float *s, const float *q, const int *n, const int *pos,
                                                   int live, int m, uint32_t *vkey, float *mkey, SelectScratch &sc,
                                                   int tid, int nthreads, int bar_id) {
  uint32_t k_and = 0xffffffffu, k_or = 0u;
#pragma unroll 4
  for (int j = tid; j < live; j += nthreads) {
    const float sj = s[j], qj = q[j];
    const int nj = n[j];
    const uint32_t vk = variance_key_fast(sj, qj, nj);
    vkey[j] = vk;
    mkey[j] = mean_fast(sj, nj);
    k_and &= vk;
    k_or |= vk;
  }
  return group_select_from_keys(pos, live, m, vkey, mkey, k_and, k_or, sc, tid, nthreads, bar_id);
}

// Slot first in (score asc, position asc) order among the slots [0, live) with eligible(j); -1 if there is none.
// Same calling convention as group_select_victim.  Used by the policies of Table 1 other than RoCo.
template <typename ScoreF, typename EligF>
__device__ __forceinline__ int group_argmin(ScoreF score, EligF eligible, const int *pos, int live, SelectScratch &sc,
                                            int tid, int nthreads, int bar_id) {
  float bm = INFINITY;
  int bs = -1;
  for (int j = tid; j < live; j += nthreads) {
    if (!eligible(j)) continue;
    const float v = score(j);
    if (bs < 0 || v < bm) { bm = v; bs = j; }
    else if (v == bm && pos[j] < pos[bs]) bs = j;
  }
  int bp = (bs >= 0) ? pos[bs] : 0x7fffffff;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, bm, o);
    const int op = __shfl_xor_sync(0xffffffffu, bp, o);
    const int os = __shfl_xor_sync(0xffffffffu, bs, o);
    if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
  }
  const int warp = tid >> 5, nwarps = nthreads >> 5;
  if ((tid & 31) == 0) { sc.red_mean[warp] = bm; sc.red_pos[warp] = bp; sc.red_slot[warp] = bs; }
  named_bar_sync(bar_id, nthreads);
  bm = sc.red_mean[0]; bp = sc.red_pos[0]; bs = sc.red_slot[0];
  for (int w = 1; w < nwarps; ++w) {
    const float om = sc.red_mean[w];
    const int op = sc.red_pos[w], os = sc.red_slot[w];
    if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
  }
  named_bar_sync(bar_id, nthreads);
  return bs;
}

// Scope size for `live` cached tokens (Sec. 4.3 / Sec. 1 readings), clipped to [1, live].
__device__ __host__ __forceinline__ int scope_size(int live, int r, int scope_mode) {
  int m = (scope_mode == ROCO_SCOPE_EXCLUDE_TOP_R) ? live - r : r;
  if (m < 1) m = 1;
  if (m > live) m = live;
  return m;
}

}  // namespace roco
