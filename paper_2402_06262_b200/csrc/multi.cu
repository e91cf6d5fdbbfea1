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

#include "common.cuh"
#include "launch.h"
#include "select.cuh"
#include "tc.cuh"

namespace roco {

constexpr int kMqConsumerWarps = 8;
constexpr int kMqConsumers = kMqConsumerWarps * 32;
constexpr int kMqProducerWarp = kMqConsumerWarps;
constexpr int kMqPolicyWarp0 = kMqConsumerWarps + 1;
constexpr int kMqPolicyThreads = 128;
constexpr int kMqThreads = kMqConsumers + 32 + kMqPolicyThreads;
constexpr int kMqBarConsumers = 1;
constexpr int kMqBarPolicy = 2;
constexpr int kMqTile = 16384;
constexpr int kMqMaxQ = 16;  // queries per step
constexpr int kMqQPW = 4;    // queries per consumer warp

struct MultiParams {
  const char *K, *V;
  float *s, *q;
  int *n, *pos, *live, *t_next, *status;
  const char *Q, *k_new, *v_new;
  char *out;
  float *lse;
  int *ev_slot, *ev_pos;
  int B, r, scope_mode, stages, M, nb;
  int group;  // query heads per new token: M = nb * group, query row i belongs to token i / group of the block
  float scale;
  long long q_ustride, kv_ustride, out_ustride;  // rows (tokens) between consecutive units in Q, K_new/V_new, out
};

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

// What the policy warps of a multi-query step see of the CTA's shared memory.
struct PolicyView {
  float *z;  // [M][Bp] probabilities once p_ready has completed
  size_t Bp;
  uint32_t *vkey;
  float *mkey;
  signed char *newtok;
  SelectScratch *sel;
  float *knew, *vnew, *zn;
  float *qf;  // [M][D] queries as fp32, filled by the policy warps themselves (nullptr: read Q from global)
  float *pn;  // [M][nb] probabilities of the new tokens when the consumers have zeroed them in z, else nullptr
  int *ctl;
  uint64_t *p_ready, *policy_done;
  // Tensor-core kernel only (else nullptr / false): the producer copies the unit's s, q, n arrays into vkey, mkey,
  // nbuf with bulk copies that complete on stats_full (the keys are then formed in place), and the consumer warps
  // compute the new tokens' scores themselves, so the policy warps stage only the new values.
  int *nbuf;
  int *posbuf;  // the unit's positions as they were before the step (with stats_full)
  uint64_t *stats_full;
  bool zn_by_consumers;
  // tcgen05 kernel only: the kernel applies the statistics update itself (from sums its consumer threads form)
  bool stats_by_consumers = false;
};

// The policy warps' part of a multi-query step: free `need` slots (Sec. 4.3 rule on frozen statistics), insert
// the new tokens in increasing slot order, score the queries against the new keys, and -- once the consumers
// have normalised -- apply the statistics update.  Called by the kMqPolicyThreads policy threads.
template <typename T, int D>
__device__ __forceinline__ void multi_policy(const MultiParams &p, const PolicyView &v, int u, int ptid, int live0,
                                             int need, int live1) {
  constexpr int kRowBytes = D * (int)sizeof(T);
  constexpr int kLanesPerRow = kRowBytes / 16;
  const int M = p.M, nb = p.nb, B = p.B;
  const size_t Bp = v.Bp;
  const size_t unit_kv = (size_t)u * B * kRowBytes, unit_st = (size_t)u * B;
  volatile int *abort_flag = v.ctl;
  const int plane = ptid & 31, pwarp = ptid >> 5;
  const int t_new = p.t_next[u];
  const float *gs = p.s + unit_st, *gq = p.q + unit_st;
  const int *gn = p.n + unit_st;
  int *gpos = p.pos + unit_st;
  const int *opos = v.stats_full ? v.posbuf : gpos;  // positions before the step (shared-memory copy if staged)
  for (int j = ptid; j < live1; j += kMqPolicyThreads) v.newtok[j] = -1;
  {  // new keys / values (and the queries) as fp32 in shared memory, 16-byte loads issued back to back
    constexpr int kEPC = Elem<T>::kPerChunk;
    const uint4 *gk = reinterpret_cast<const uint4 *>(p.k_new + (size_t)u * p.kv_ustride * kRowBytes);
    const uint4 *gv = reinterpret_cast<const uint4 *>(p.v_new + (size_t)u * p.kv_ustride * kRowBytes);
    const uint4 *gqr = reinterpret_cast<const uint4 *>(p.Q + (size_t)u * p.q_ustride * kRowBytes);
    const int nkv = nb * D / kEPC, nq = v.qf ? M * D / kEPC : 0;
    if (v.zn_by_consumers && !v.vnew) {
      // the consumers read the new values from global memory themselves
    } else if (v.zn_by_consumers) {
#pragma unroll 4
      for (int i = ptid; i < nkv; i += kMqPolicyThreads) {
        float f[kEPC];
        Elem<T>::unpack(gv[i], f);
#pragma unroll
        for (int e = 0; e < kEPC; ++e) v.vnew[i * kEPC + e] = f[e];
      }
    } else {
#pragma unroll 4
      for (int i = ptid; i < 2 * nkv + nq; i += kMqPolicyThreads) {
        const uint4 c = i < nkv ? gk[i] : (i < 2 * nkv ? gv[i - nkv] : gqr[i - 2 * nkv]);
        float *dst =
            i < nkv ? v.knew + i * kEPC : (i < 2 * nkv ? v.vnew + (i - nkv) * kEPC : v.qf + (i - 2 * nkv) * kEPC);
        float f[kEPC];
        Elem<T>::unpack(c, f);
#pragma unroll
        for (int e = 0; e < kEPC; ++e) dst[e] = f[e];
      }
    }
  }
  named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
  int *tgt = v.ctl + 1;  // [nb] target slots, ascending
  if (need > 0) {
    // the rule of Sec. 4.3 applied `need` times on frozen statistics = one pass: the tokens outside the scope
    // (the live0 - m last in (variance, position) order) never enter it, so the `need` first of the scope in
    // (mean, position) order leave
    uint32_t k_and = 0xffffffffu, k_or = 0u;
    if (v.stats_full) {  // s, q, n sit in vkey, mkey, nbuf: form the keys in place
      mbar_wait(v.stats_full, 0, abort_flag, p.status);
#pragma unroll 8
      for (int j = ptid; j < live0; j += kMqPolicyThreads) {
        const float sj = __uint_as_float(v.vkey[j]), qj = v.mkey[j];
        const int nj = v.nbuf[j];
        const uint32_t vk = variance_key_fast(sj, qj, nj);
        v.vkey[j] = vk;
        v.mkey[j] = mean_fast(sj, nj);
        k_and &= vk;
        k_or |= vk;
      }
    } else {
#pragma unroll 8
      for (int j = ptid; j < live0; j += kMqPolicyThreads) {
        const float sj = gs[j], qj = gq[j];
        const int nj = gn[j];
        const uint32_t vk = variance_key_fast(sj, qj, nj);
        v.vkey[j] = vk;
        v.mkey[j] = mean_fast(sj, nj);
        k_and &= vk;
        k_or |= vk;
      }
    }
    group_and_or(k_and, k_or, *v.sel, ptid, kMqPolicyThreads, kMqBarPolicy);  // publishes vkey / mkey too
    const int m = scope_size(live0, p.r, p.scope_mode);
    int *list = v.ctl + 24;  // freed slots, in the order they were chosen
    int *cnt = v.ctl + 20;
    uint32_t rank, ties;
    // `rounds` times the token first in (mean, position) order over mkey; a chosen token is masked by the thread
    // that scans it, which keeps the mean it had in keep[] (about 2 000 cycles a round)
    float keep[4] = {0.f, 0.f, 0.f, 0.f};
    auto argmin_rounds = [&](int rounds) {
      bool ok = true;
#pragma unroll 1
      for (int e = 0; e < rounds; ++e) {
        float bm = INFINITY;
        int bs = -1;
#pragma unroll 4
        for (int j = ptid; j < live0; j += kMqPolicyThreads) {
          const float mean = v.mkey[j];
          if (mean < bm) { bm = mean; bs = j; }
          else if (mean == bm && bs >= 0 && opos[j] < opos[bs]) bs = j;
        }
        // a thread's candidates come in increasing slot order but ties go to the lower *position*
        int bp = bs >= 0 ? opos[bs] : 0x7fffffff;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float om = __shfl_xor_sync(0xffffffffu, bm, o);
          const int op = __shfl_xor_sync(0xffffffffu, bp, o);
          const int os = __shfl_xor_sync(0xffffffffu, bs, o);
          if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
        }
        float *rm = v.sel->red_mean + (e & 1) * 4;  // double-buffered: one barrier per round
        int *rp = v.sel->red_pos + (e & 1) * 4, *rs = v.sel->red_slot + (e & 1) * 4;
        if (plane == 0) { rm[pwarp] = bm; rp[pwarp] = bp; rs[pwarp] = bs; }
        named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
        bm = rm[0]; bp = rp[0]; bs = rs[0];
#pragma unroll
        for (int w = 1; w < kMqPolicyThreads / 32; ++w) {
          const float om = rm[w];
          const int op = rp[w], os = rs[w];
          if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
        }
        if (bs < 0) {
          ok = false;
          bs = e;  // keeps the slots distinct
        }
        if (ptid == 0) list[e] = bs;
        if (ok && (bs % kMqPolicyThreads) == ptid) {  // only this thread ever scans slot bs
          if (e < 4) keep[e] = v.mkey[bs];
          v.mkey[bs] = INFINITY;
        }
      }
      return ok;
    };
    // the `need` smallest of mkey by radix select on the need-th, then one pass that collects everything up to it
    auto collect_lowest = [&](uint32_t m_and, uint32_t m_or) {
      const uint32_t Tm = radix_select<uint32_t>([&](int j) { return __float_as_uint(v.mkey[j]); },
                                                 [&](int) { return true; }, live0, (uint32_t)(need - 1), *v.sel, ptid,
                                                 kMqPolicyThreads, kMqBarPolicy, &rank, &ties, m_and, m_or);
      int Pm = 0x7fffffff;
      if (ties != rank + 1) {
        uint32_t r2, t2;
        Pm = (int)radix_select<uint32_t>([&](int j) { return (uint32_t)opos[j]; },
                                         [&](int j) { return __float_as_uint(v.mkey[j]) == Tm; }, live0, rank,
                                         *v.sel, ptid, kMqPolicyThreads, kMqBarPolicy, &r2, &t2);
      }
      if (ptid == 0) *cnt = 0;
      named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
      for (int j = ptid; j < live0; j += kMqPolicyThreads) {
        const uint32_t k = __float_as_uint(v.mkey[j]);
        if (k < 0x7f800000u && (k < Tm || (k == Tm && (Pm == 0x7fffffff || opos[j] <= Pm)))) {
          const int at = atomicAdd(cnt, 1);
          if (at < kMqMaxQ) list[at] = j;
        }
      }
      named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
      return *cnt == need;
    };

    // A scope that leaves out only a few tokens almost always contains the `need` tokens of lowest mean.  So
    // those are picked first, over all cached tokens, and then tested: the one of them that comes last in
    // (variance, position) order is in scope iff fewer than m tokens come before it, and then so are the others
    // (they come before it too) -- one counting pass in place of the radix select for the scope threshold.
    bool done = false;
    if (need > 1 && p.scope_mode == ROCO_SCOPE_LOWEST_R && m < live0) {
      // The scope is the r lowest-variance tokens still cached (Sec. 1 reading), so it refills after every
      // eviction: one radix select gives the scope of the first eviction, and each later one admits the token
      // next in (variance, position) order before the in-scope token of lowest mean leaves.  The state of a
      // token is kept in newtok for the duration: -1 outside the scope, -2 in scope, -3 evicted.
      uint32_t Tv = radix_select<uint32_t>([&](int j) { return v.vkey[j]; }, [&](int) { return true; }, live0,
                                           (uint32_t)(m - 1), *v.sel, ptid, kMqPolicyThreads, kMqBarPolicy, &rank, &ties,
                                           k_and, k_or);
      int Pv = 0x7fffffff;
      if (ties != rank + 1) {
        uint32_t r2, t2;
        Pv = (int)radix_select<uint32_t>([&](int j) { return (uint32_t)opos[j]; },
                                         [&](int j) { return v.vkey[j] == Tv; }, live0, rank, *v.sel, ptid,
                                         kMqPolicyThreads, kMqBarPolicy, &r2, &t2);
      }
      for (int j = ptid; j < live0; j += kMqPolicyThreads) {
        const uint32_t k = v.vkey[j];
        if (k < Tv || (k == Tv && (Pv == 0x7fffffff || opos[j] <= Pv))) v.newtok[j] = -2;
      }
      named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
      bool ok = true;
#pragma unroll 1
      for (int it = 0; it < need; ++it) {
        if (it > 0 && p.r <= live0 - it) {  // the scope has lost a token and the cache still holds one to admit
          uint32_t bk = 0xffffffffu;
          int bs = -1, bp = 0x7fffffff;
          for (int j = ptid; j < live0; j += kMqPolicyThreads) {
            if (v.newtok[j] != -1) continue;
            const uint32_t k = v.vkey[j];
            const int pj = opos[j];
            if (bs < 0 || k < bk || (k == bk && pj < bp)) { bk = k; bs = j; bp = pj; }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const uint32_t ok2 = __shfl_xor_sync(0xffffffffu, bk, o);
            const int op = __shfl_xor_sync(0xffffffffu, bp, o);
            const int os = __shfl_xor_sync(0xffffffffu, bs, o);
            if (os >= 0 && (bs < 0 || ok2 < bk || (ok2 == bk && op < bp))) { bk = ok2; bp = op; bs = os; }
          }
          if (plane == 0) { v.sel->hist[pwarp] = bk; v.sel->red_pos[pwarp] = bp; v.sel->red_slot[pwarp] = bs; }
          named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
          bk = v.sel->hist[0]; bp = v.sel->red_pos[0]; bs = v.sel->red_slot[0];
#pragma unroll
          for (int w = 1; w < kMqPolicyThreads / 32; ++w) {
            const uint32_t ok2 = v.sel->hist[w];
            const int op = v.sel->red_pos[w], os = v.sel->red_slot[w];
            if (os >= 0 && (bs < 0 || ok2 < bk || (ok2 == bk && op < bp))) { bk = ok2; bp = op; bs = os; }
          }
          named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
          if (bs >= 0 && ptid == 0) v.newtok[bs] = -2;
          named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
        }
        float bm = INFINITY;
        int bs = -1, bp = 0x7fffffff;
        for (int j = ptid; j < live0; j += kMqPolicyThreads) {
          if (v.newtok[j] != -2) continue;
          const float mean = v.mkey[j];
          const int pj = opos[j];
          if (mean < bm || (mean == bm && pj < bp)) { bm = mean; bs = j; bp = pj; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float om = __shfl_xor_sync(0xffffffffu, bm, o);
          const int op = __shfl_xor_sync(0xffffffffu, bp, o);
          const int os = __shfl_xor_sync(0xffffffffu, bs, o);
          if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
        }
        if (plane == 0) { v.sel->red_mean[pwarp] = bm; v.sel->red_pos[pwarp] = bp; v.sel->red_slot[pwarp] = bs; }
        named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
        bm = v.sel->red_mean[0]; bp = v.sel->red_pos[0]; bs = v.sel->red_slot[0];
#pragma unroll
        for (int w = 1; w < kMqPolicyThreads / 32; ++w) {
          const float om = v.sel->red_mean[w];
          const int op = v.sel->red_pos[w], os = v.sel->red_slot[w];
          if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
        }
        named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
        if (bs < 0) { ok = false; bs = it; }  // only after corrupt statistics; keeps the slots distinct
        if (ptid == 0) { list[it] = bs; v.newtok[bs] = -3; }
        named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
      }
      for (int j = ptid; j < live0; j += kMqPolicyThreads) v.newtok[j] = -1;
      if (!ok && ptid == 0) atomicOr(p.status, ROCO_DEV_BAD_VICTIM);
      named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
      done = true;
    } else if (2 * m >= live0) {
      bool ok;
      if (need <= 4) {
        ok = argmin_rounds(need);
      } else {
        uint32_t m_and = 0xffffffffu, m_or = 0u;
#pragma unroll 8
        for (int j = ptid; j < live0; j += kMqPolicyThreads) {
          const uint32_t k = __float_as_uint(v.mkey[j]);
          m_and &= k;
          m_or |= k;
        }
        group_and_or(m_and, m_or, *v.sel, ptid, kMqPolicyThreads, kMqBarPolicy);
        ok = collect_lowest(m_and, m_or);
      }
      named_bar_sync(kMqBarPolicy, kMqPolicyThreads);  // list[] is complete
      // the candidate last in (variance, position) order
      uint32_t cv = 0u;
      int cp = -1;
      if (ptid < need) {
        const int c = list[ptid];
        cv = v.vkey[c];
        cp = opos[c];
      }
      if (pwarp == 0) {  // need <= 16: the first warp holds all candidates
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const uint32_t ov = __shfl_xor_sync(0xffffffffu, cv, o);
          const int op = __shfl_xor_sync(0xffffffffu, cp, o);
          if (ov > cv || (ov == cv && op > cp)) { cv = ov; cp = op; }
        }
        if (plane == 0) { v.sel->digit = cv; v.sel->rank = (uint32_t)cp; }
      }
      named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
      cv = v.sel->digit;
      cp = (int)v.sel->rank;
      uint32_t before = 0;
#pragma unroll 8
      for (int j = ptid; j < live0; j += kMqPolicyThreads) {
        const uint32_t k = v.vkey[j];
        before += (k < cv || (k == cv && opos[j] < cp)) ? 1u : 0u;
      }
      before = __reduce_add_sync(0xffffffffu, before);
      if (plane == 0) v.sel->hist[pwarp] = before;
      named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
      before = 0;
#pragma unroll
      for (int w = 0; w < kMqPolicyThreads / 32; ++w) before += v.sel->hist[w];
      done = ok && before < (uint32_t)m;
      if (done) {
        if (need == 1 && ptid == 0) tgt[0] = list[0];
      } else if (need <= 4) {  // the general rule below needs the means as they were
        for (int e = 0; e < need; ++e) {
          const int c = list[e];
          if (c >= 0 && c < live0 && (c % kMqPolicyThreads) == ptid && v.mkey[c] == INFINITY) v.mkey[c] = keep[e];
        }
      }
      named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
    }
    if (!done) {
      uint32_t Tv = 0xffffffffu;
      int Pv = 0x7fffffff;
      if (m < live0) {
        Tv = radix_select<uint32_t>([&](int j) { return v.vkey[j]; }, [&](int) { return true; }, live0,
                                    (uint32_t)(m - 1), *v.sel, ptid, kMqPolicyThreads, kMqBarPolicy, &rank, &ties,
                                    k_and, k_or);
        if (ties != rank + 1) {
          uint32_t r2, t2;
          Pv = (int)radix_select<uint32_t>([&](int j) { return (uint32_t)opos[j]; },
                                           [&](int j) { return v.vkey[j] == Tv; }, live0, rank, *v.sel, ptid,
                                           kMqPolicyThreads, kMqBarPolicy, &r2, &t2);
        }
      }
      auto in_scope = [&](int j) {
        const uint32_t k = v.vkey[j];
        return k < Tv || (k == Tv && (Pv == 0x7fffffff || opos[j] <= Pv));
      };
      // the `need` (at most 16) in-scope tokens first in (mean, position) order; out-of-scope tokens are masked
      // once, which leaves a plain selection over mkey
      for (int j = ptid; j < live0; j += kMqPolicyThreads)
        if (!in_scope(j)) v.mkey[j] = INFINITY;
      named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
      bool ok;
      if (need <= 4) ok = argmin_rounds(need);  // few victims: one argmin after the other
      else ok = collect_lowest(0u, 0xffffffffu);
      named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
      if (!ok && ptid == 0) {  // only after corrupt statistics; the step's results are void
        atomicOr(p.status, ROCO_DEV_BAD_VICTIM);
        if (need > 4)
          for (int x = *cnt < 0 ? 0 : (*cnt > need ? need : *cnt); x < need; ++x) list[x] = x;
      }
      if (need == 1 && ptid == 0) tgt[0] = list[0];
      named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
    }
    if (need > 1 && ptid < need) {  // order the freed slots by slot index
      int rk = 0;
      for (int x = 0; x < need; ++x) rk += list[x] < list[ptid];
      if (rk < nb) tgt[rk] = list[ptid];
    }
  }
  if (ptid < nb - need) tgt[need + ptid] = live0 + ptid;  // free slots behind the occupied ones
  named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
  // the new tokens take the target slots: evicted positions out, new K/V and positions in
  if (ptid < nb) {
    int slot = tgt[ptid];
    if (slot < 0 || slot >= B) slot = 0;  // only after corrupt statistics (status bit set above)
    p.ev_slot[(size_t)u * nb + ptid] = ptid < need ? slot : -1;
    if (p.ev_pos) p.ev_pos[(size_t)u * nb + ptid] = ptid < need ? opos[slot] : -1;
    v.newtok[slot] = (signed char)ptid;
    gpos[slot] = t_new + ptid;
  }
  // scores of every query against every new token, from k_new directly (log2 domain)
  const float zscale = p.scale * kLog2e;
  if (v.zn_by_consumers) {
    // the consumer warps form these scores on the tensor cores
  } else if (v.qf) {
    // one dot product per thread and turn, operands in shared memory; the element order is rotated by the lane
    // so that the 32 lanes of a warp (different keys, same offset) hit different banks
    for (int w = ptid; w < M * nb; w += kMqPolicyThreads) {
      const int i = w / nb, jn = w % nb;
      const float *qr = v.qf + i * D, *kr = v.knew + jn * D;
      float acc = 0.f;
#pragma unroll 8
      for (int c = 0; c < D; ++c) {
        const int cc = (c + plane) & (D - 1);
        acc = fmaf(qr[cc], kr[cc], acc);
      }
      v.zn[w] = acc * zscale;
    }
  } else {
    for (int w = pwarp; w < M * nb; w += kMqPolicyThreads / 32) {  // one dot product per warp and turn
      const int i = w / nb, jn = w % nb;
      const T *qrow = (const T *)p.Q + ((size_t)u * p.q_ustride + i) * D;
      float acc = 0.f;
      for (int c = plane; c < D; c += 32) acc = fmaf(Elem<T>::load(qrow + c), v.knew[jn * D + c], acc);
      acc = warp_sum(acc);
      if (plane == 0) v.zn[w] = acc * zscale;
    }
  }
  if (ptid == 0) { p.live[u] = live1; p.t_next[u] = t_new + nb; }
  named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
  if (ptid == 0) mbar_arrive(v.policy_done);
  // In-place overwrite, 16 bytes per thread and turn.  Nothing in this step reads these rows from the cache (the
  // scores and values of new tokens come from K_new / V_new), so it is done after the consumers were released.
#pragma unroll 4
  for (int w = ptid; w < nb * 2 * kLanesPerRow; w += kMqPolicyThreads) {
    const int i = w / (2 * kLanesPerRow), c = w % (2 * kLanesPerRow);
    const bool isv = c >= kLanesPerRow;
    const int cc = isv ? c - kLanesPerRow : c;
    int slot = tgt[i];
    if (slot < 0 || slot >= B) slot = 0;
    const uint4 val = *((const uint4 *)((isv ? p.v_new : p.k_new) + ((size_t)u * p.kv_ustride + i) * kRowBytes) + cc);
    *((uint4 *)(const_cast<char *>(isv ? p.V : p.K) + unit_kv + (size_t)slot * kRowBytes) + cc) = val;
  }

  if (v.stats_by_consumers) return;
  // statistics of Sec. 4.3 once the probabilities are in shared memory
  mbar_wait(v.p_ready, 0, abort_flag, p.status);
  // four slots per turn, their old statistics loaded before the first store (the arrays are updated in place,
  // so the compiler keeps loads behind earlier stores)
  constexpr int kBatch = 4;
  for (int j0 = ptid; j0 < live1; j0 += kBatch * kMqPolicyThreads) {
    float s0v[kBatch], q0v[kBatch];
    int n0v[kBatch];
#pragma unroll
    for (int k = 0; k < kBatch; ++k) {
      const int j = j0 + k * kMqPolicyThreads;
      const bool old = j < live1 && v.newtok[j] < 0;
      s0v[k] = old ? gs[j] : 0.f;
      q0v[k] = old ? gq[j] : 0.f;
      n0v[k] = old ? gn[j] : 0;
    }
#pragma unroll
    for (int k = 0; k < kBatch; ++k) {
      const int j = j0 + k * kMqPolicyThreads;
      if (j >= live1) break;
      const int jn = v.newtok[j];
      const bool fresh = jn >= 0;
      float ds = 0.f, dq = 0.f;
      int dn;
      {
        // token t of the block (its `group` query heads) sees new token jn only if t >= jn; the statistics take
        // the group-wise averaged probability once per token (Sec. 5.3, App. A), which for one head is p itself
        const int t0 = fresh ? jn : 0, group = p.group;
        for (int t = t0; t < nb; ++t) {
          float pb = 0.f;
          for (int g = 0; g < group; ++g) {
            const int i = t * group + g;
            pb += (fresh && v.pn) ? v.pn[i * nb + jn] : v.z[(size_t)i * Bp + j];
          }
          if (group > 1) pb = pb / (float)group;
          ds += pb;
          dq = fmaf(pb, pb, dq);
        }
        dn = nb - t0;
      }
      p.s[unit_st + j] = s0v[k] + ds;
      p.q[unit_st + j] = q0v[k] + dq;
      p.n[unit_st + j] = n0v[k] + dn;
    }
  }
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

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16 x 8, fp32) += A (16 x 16, bf16, row-major) * B (16 x 8, bf16, column-major)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
// byte offset of the 16-byte chunk `chunk` (0..15 over the 128 columns) of row `row` inside a swizzled tile
__device__ __forceinline__ uint32_t tile_chunk_offset(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * 8192 + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
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

// ------------------------------------------------------------------------------------------------------------
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
constexpr int kUmMaxTiles = 31;                 // 16 tensor-memory columns each, and 16 for the output
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
  uint64_t *full, *empty, *s_full, *p_tile, *d_ready, *o_full, *policy_done, *stats_full;
  uint32_t *tmem_base;
  int *ctl;
};

__host__ __device__ inline size_t multi_um_pbuf_bytes(int B) {
  const size_t tiles = ((size_t)B + kUmTile - 1) / kUmTile;
  return (tiles + 3) / 4 * kUmPBlock;
}

__host__ __device__ inline size_t multi_um_smem_bytes(int B, int stages, int nb) {
  const size_t Bp = align_up((size_t)B, 64);
  size_t b = (size_t)stages * kUmTileBytes + multi_um_pbuf_bytes(B) + 4096 + 2048;
  b += Bp + sizeof(SelectScratch);
  b = align_up(b, 16) + (size_t)16 * nb * 4 + (2 * kMqConsumerWarps + 2) * 16 * 4;
  b = align_up(b, 8) + (2 * (size_t)stages + 6 + kUmMaxTiles) * 8 + 64 * 4;
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
  m.d_ready = (uint64_t *)p; p += 8;
  m.o_full = (uint64_t *)p; p += 8;
  m.policy_done = (uint64_t *)p; p += 8;
  m.stats_full = (uint64_t *)p; p += 8;
  m.tmem_base = (uint32_t *)p; p += 8;
  m.ctl = (int *)p;
  return m;
}

// Tensor-memory columns of one CTA: 16 per tile of 128 keys and 16 for the output accumulator behind them, a
// power of two of at least 32.
__host__ __device__ inline int multi_um_cols(int B) {
  const int tiles = (B + kUmTile - 1) / kUmTile;
  int c = 32;
  while (c < 16 * tiles + 16) c <<= 1;
  return c;
}

// v[i] (i = query) reduced over the 32 lanes; lane l returns the result for query l >> 1.  The exchange halves
// the number of live values at every step (16 shuffles in all instead of 80).
template <bool kMax>
__device__ __forceinline__ float lanes_reduce16(float (&v)[16], int lane) {
#pragma unroll
  for (int step = 0; step < 4; ++step) {
    const int w = 8 >> step, o = 16 >> step;
    const bool up = (lane & o) != 0;
#pragma unroll
    for (int k = 0; k < w; ++k) {
      const float send = up ? v[k] : v[k + w];
      const float keep = up ? v[k + w] : v[k];
      const float got = __shfl_xor_sync(0xffffffffu, send, o);
      v[k] = kMax ? fmaxf(keep, got) : keep + got;
    }
  }
  const float got = __shfl_xor_sync(0xffffffffu, v[0], 1);
  return kMax ? fmaxf(v[0], got) : v[0] + got;
}

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
    for (int i = 0; i < kUmMaxTiles; ++i) mbar_init(&sm.p_tile[i], kMqConsumerWarps / 2);
    mbar_init(sm.d_ready, kMqConsumerWarps);
    mbar_init(sm.o_full, 1);
    mbar_init(sm.policy_done, 1);
    mbar_init(sm.stats_full, 1);
    sm.ctl[0] = 0;
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
  const uint32_t tmem_o = tmem + (uint32_t)(16 * ((B + kUmTile - 1) / kUmTile));

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
          tmem_ld2(tl + (uint32_t)(16 * (it0 + k)), d2);
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
      mbar_wait(&sm.p_tile[it], 0, abort_flag, p.status);  // this tile's P^T block
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
        const char *pb = sm.pbuf + (size_t)(it >> 2) * kUmPBlock + (it & 3) * 32;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          umma_bf16(tmem_o, smem_desc_sw128_mn(tile + kk * 2048, kUmHalfBytes), smem_desc_sw128_mn(pb + kk * 2048, 16),
                    kIdescUmO, (it > 0 || kk > 0) ? 1u : 0u);
        umma_commit(&sm.empty[st]);
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
  // over the 256 consumer threads; returns the result for query (lane & 15) and leaves in v the maxima of all 16
  // queries, or the reciprocals of their sums (0 for rows that do not exist)
  auto all_reduce16 = [&](float (&v)[16], bool is_max, float *red) {
    const float x = is_max ? lanes_reduce16<true>(v, lane) : lanes_reduce16<false>(v, lane);
    if (!(lane & 1)) red[warp * 16 + (lane >> 1)] = x;
    named_bar_sync(kMqBarConsumers, kMqConsumers);
    float acc = red[lane & 15];
#pragma unroll
    for (int w = 1; w < kMqConsumerWarps; ++w) {
      const float o = red[w * 16 + (lane & 15)];
      acc = is_max ? fmaxf(acc, o) : acc + o;
    }
    const float give = is_max ? acc : ((lane & 15) < M ? 1.f / acc : 0.f);
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __shfl_sync(0xffffffffu, give, i);
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
  // only makes the maximum an upper bound (it is the stabiliser of the exponentials, nothing else).
  float a[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) a[i] = -INFINITY;
  for (int it = wg; it < n_tiles; it += 2) {
    const int j = it * kUmTile + kl;
    uint32_t r[16];
    tmem_ld16(tlane + (uint32_t)(it * 16), r);
    const bool held = j < live0;
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = fmaxf(a[i], held ? __uint_as_float(r[i]) : -INFINITY);
  }
  float my_max = all_reduce16(a, true, sm.red);  // its barrier also publishes zn, V_new and the cleared block
  {
    // the new tokens' scores join the maxima
    const float *znmax = sm.red + 2 * kMqConsumerWarps * 16;
    const float zm = fmaxf(znmax[lane & 15], znmax[16 + (lane & 15)]);
    my_max = fmaxf(my_max, zm);
#pragma unroll
    for (int k = 0; k < 16; ++k) a[k] = fmaxf(a[k], __shfl_sync(0xffffffffu, zm, k));
  }
  // a[i] <- -(row maximum in the log2 domain); rows that do not exist hold zeros
#pragma unroll
  for (int i = 0; i < 16; ++i) a[i] = (a[i] > -INFINITY) ? -a[i] * zscale : 0.f;

  // ---- the selection's result: masks and the new tokens' scores in place
  mbar_wait(sm.policy_done, 0, abort_flag, p.status);
  for (int it = wg; it < n_tiles; it += 2) {
    const int j = it * kUmTile + kl;
    const int nt = j < live1 ? (int)sm.newtok[j] : -1;
    if (__any_sync(0xffffffffu, nt >= 0 || j >= live1)) {
      uint32_t r[16];
      tmem_ld16(tlane + (uint32_t)(it * 16), r);
      if (j >= live1) {
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = ninf;
      } else if (nt >= 0) {  // the new token's scores, -inf where the block's causal mask hides it
        const uint4 *zr = reinterpret_cast<const uint4 *>(sm.zn + nt * 16);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint4 z4 = zr[k];
          r[4 * k] = z4.x; r[4 * k + 1] = z4.y; r[4 * k + 2] = z4.z; r[4 * k + 3] = z4.w;
        }
      }
      tmem_st16(tlane + (uint32_t)(it * 16), r);
    }
  }
  tmem_st_wait();

  // ---- pass 2: e = 2^(z - max) in place, row sums
  float sums[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) sums[i] = 0.f;
  for (int it = wg; it < n_tiles; it += 2) {
    uint32_t r[16];
    tmem_ld16(tlane + (uint32_t)(it * 16), r);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float e = ex2_approx(fmaf(__uint_as_float(r[i]), zscale, a[i]));
      sums[i] += e;
      r[i] = __float_as_uint(e);
    }
    tmem_st16(tlane + (uint32_t)(it * 16), r);
  }
  tmem_st_wait();
  const float my_sum = all_reduce16(sums, false, sm.red + kMqConsumerWarps * 16);
  if (warp == 0 && lane < M && p.lse) {
    const float mz = (my_max > -INFINITY) ? my_max * zscale : 0.f;
    p.lse[(size_t)u * M + lane] = (mz + log2f(my_sum)) * kLn2;
  }

  // ---- pass 3: probabilities; P^T as bf16 operand blocks, tile by tile (the output MMAs of a tile start as soon
  // as its block is complete); the statistics of Sec. 4.3 for this thread's slots
  for (int it = wg; it < n_tiles; it += 2) {
    const int j = it * kUmTile + kl;
    uint32_t r[16];
    tmem_ld16(tlane + (uint32_t)(it * 16), r);
    float pr[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) pr[i] = __uint_as_float(r[i]) * sums[i];  // sums[] holds the reciprocals by now
    const int nt = j < live1 ? (int)sm.newtok[j] : -1;
    {
      uint4 w0, w1;
      w0.x = pack_bf16x2(pr[0], pr[1]); w0.y = pack_bf16x2(pr[2], pr[3]);
      w0.z = pack_bf16x2(pr[4], pr[5]); w0.w = pack_bf16x2(pr[6], pr[7]);
      w1.x = pack_bf16x2(pr[8], pr[9]); w1.y = pack_bf16x2(pr[10], pr[11]);
      w1.z = pack_bf16x2(pr[12], pr[13]); w1.w = pack_bf16x2(pr[14], pr[15]);
      if (nt >= 0) {
        // a new token's value comes from V_new: its probabilities go to the new tokens' block, and the streamed
        // row of its slot (possibly read before the overwrite) gets zeros
        char *row = sm.pn + nt * 128;
        *reinterpret_cast<uint4 *>(row + ((0 ^ (nt & 7)) << 4)) = w0;
        *reinterpret_cast<uint4 *>(row + ((1 ^ (nt & 7)) << 4)) = w1;
        w0 = make_uint4(0u, 0u, 0u, 0u);
        w1 = w0;
      }
      char *row = sm.pbuf + (size_t)(it >> 2) * kUmPBlock + kl * 128;
      const int c0 = 2 * (it & 3);
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
    if (nb == 1) {
      float t = 0.f;
#pragma unroll
      for (int i = 0; i < 16; ++i) t += pr[i];
      ds = t / (float)M;
      dq = ds * ds;
    } else if (gshift == 0) {
#pragma unroll
      for (int i = 0; i < 16; ++i) { ds += pr[i]; dq = fmaf(pr[i], pr[i], dq); }
    } else if (gshift == 1) {
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const float m2 = (pr[2 * t] + pr[2 * t + 1]) * 0.5f;
        ds += m2; dq = fmaf(m2, m2, dq);
      }
    } else if (gshift == 2) {
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float m4 = ((pr[4 * t] + pr[4 * t + 1]) + (pr[4 * t + 2] + pr[4 * t + 3])) * 0.25f;
        ds += m4; dq = fmaf(m4, m4, dq);
      }
    } else {
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        float m8 = 0.f;
#pragma unroll
        for (int h = 0; h < 8; ++h) m8 += pr[8 * t + h];
        m8 *= 0.125f;
        ds += m8; dq = fmaf(m8, m8, dq);
      }
    }
    tmem_st2(tlane + (uint32_t)(it * 16), __float_as_uint(ds), __float_as_uint(dq));  // for the policy warps
  }
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

static int multi_tc_pick_stages(int B, int M, int nb) {
  const size_t per_sm = 227 * 1024;
  for (int ctas = 2; ctas >= 1; --ctas)
    for (int st = 6; st >= 3; --st)
      if ((multi_tc_smem_bytes(B, st, M, nb) + 1024) * ctas <= per_sm) return st;
  return 0;
}

// Ring stages of the tcgen05 kernel: two (of 32 KiB) where two CTAs then share an SM, which covers a CTA's softmax
// phase with the other's stream; else one CTA per SM with as many stages as fit.  0: the budget does not fit.
static int multi_um_pick_stages(int B, int nb) {
  const size_t per_sm = 227 * 1024;
  if (multi_um_cols(B) > 512) return 0;
  if (multi_um_cols(B) <= 256 && (multi_um_smem_bytes(B, 2, nb) + 1024) * 2 <= per_sm) return 2;
  for (int st = 4; st >= 2; --st)
    if (multi_um_smem_bytes(B, st, nb) + 1024 <= per_sm) return st;
  return 0;
}

// Row layouts the tcgen05 kernel takes: from 4 rows up (below that the warp-level kernel is as fast), the heads of
// a token averaged inside a thread -- group sizes that are powers of two, or one token with any number of heads.
static bool multi_um_rows(int M, int nb) {
  const int grp = M / nb;
  return M >= 4 && (nb == 1 || grp == 1 || grp == 2 || grp == 4 || grp == 8);
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
    const int um_stages = multi_um_rows(M, nb) ? multi_um_pick_stages(c.B, nb) : 0;
    // with one CTA per SM either way, the tcgen05 kernel keeps more bytes in flight; with two of the warp-level
    // kernel against one of this, the two win
    const bool tc_two = (multi_tc_smem_bytes(c.B, 3, M, nb) + 1024) * 2 <= (size_t)227 * 1024;
    if (um_stages > 0 && (um_stages == 2 || !tc_two) &&
        make_tensor_map_rows128_bf16(&mapK, c.K, (unsigned long long)U * c.B, kUmTile) &&
        make_tensor_map_rows128_bf16(&mapV, c.V, (unsigned long long)U * c.B, kUmTile)) {
      const size_t smem = multi_um_smem_bytes(c.B, um_stages, nb);
      err = cudaFuncSetAttribute(multi_step_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (err != cudaSuccess) return ROCO_ERR_CUDA;
      p.stages = um_stages;
      multi_step_umma_kernel<<<U, kUmThreads, smem, stream>>>(mapK, mapV, p, multi_um_cols(c.B));
      return cudaGetLastError() == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
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
