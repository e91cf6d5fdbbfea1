// Shared by the multi-query step kernels (block-wise evict-and-encode, grouped-query decode): launch parameters,
// warp roles, the policy warps' part of a step, and the small PTX helpers of the tensor-core variants.
#pragma once

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

// Victims of a block step under ROCO_SCOPE_LOWEST_R when more than one token leaves.  The scope is the r
// lowest-variance tokens still cached (Sec. 1 reading), so it refills after every eviction: before each eviction but
// the first the token next in (variance, position) order is admitted, then the in-scope token of lowest mean
// leaves.  Everything that can take part is known up front: the first scope S (rank m - 1 in variance order), the
// at most need - 1 tokens that follow it in that order (the admits), and -- since a victim from S is always the
// lowest-mean token left in S -- the `need` lowest means of S.  Three threshold searches find them; one warp then
// plays the evictions on those at most 31 tokens.  The freed slots go to ctl[24 ..] in the order they were chosen;
// mkey is left masked.  Called by the kMqPolicyThreads policy threads.  (Not inlined: it is the rarer reading, and
// inlined its registers weigh on every kernel that contains the policy warps' code.)
static __device__ __noinline__ void lowest_r_block_victims(const uint32_t *vkey, float *mkey, SelectScratch *sel, int *ctl,
                                                    const int *opos, int *status, int r, int live0, int need, int m,
                                                    uint32_t k_and, uint32_t k_or, int ptid) {
  const int plane = ptid & 31, pwarp = ptid >> 5;
  int *list = ctl + 24, *cnt = ctl + 20;
  uint32_t rank, ties;
  auto variance_threshold = [&](int rk, uint32_t &T, int &P) {
    T = radix_select<uint32_t>([&](int j) { return vkey[j]; }, [&](int) { return true; }, live0, (uint32_t)rk, *sel,
                               ptid, kMqPolicyThreads, kMqBarPolicy, &rank, &ties, k_and, k_or);
    P = 0x7fffffff;
    if (ties != rank + 1) {
      uint32_t r2, t2;
      P = (int)radix_select<uint32_t>([&](int j) { return (uint32_t)opos[j]; }, [&](int j) { return vkey[j] == T; },
                                      live0, rank, *sel, ptid, kMqPolicyThreads, kMqBarPolicy, &r2, &t2);
    }
  };
  auto up_to = [&](int j, uint32_t T, int P) {
    const uint32_t k = vkey[j];
    return k < T || (k == T && (P == 0x7fffffff || opos[j] <= P));
  };
  uint32_t Tv, Tw;
  int Pv, Pw;
  variance_threshold(m - 1, Tv, Pv);
  const int wsize = live0 < m + need - 1 ? live0 : m + need - 1;  // first scope and admits together
  Tw = Tv; Pw = Pv;
  if (wsize > m) variance_threshold(wsize - 1, Tw, Pw);
  int *adm_slot = sel->red_slot;  // the admits (unordered), with the means they had
  float *adm_mean = sel->red_mean;
  if (ptid == 0) *cnt = 0;
  named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
  for (int j = ptid; j < live0; j += kMqPolicyThreads) {
    if (up_to(j, Tv, Pv)) continue;
    if (wsize > m && up_to(j, Tw, Pw)) {
      const int at = atomicAdd(cnt, 1);
      if (at < kMqMaxQ) { adm_slot[at] = j; adm_mean[at] = mkey[j]; }
    }
    mkey[j] = INFINITY;  // outside the first scope: no candidate below
  }
  named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
  int n_adm = *cnt;
  if (n_adm > kMqMaxQ - 1) n_adm = kMqMaxQ - 1;
  named_bar_sync(kMqBarPolicy, kMqPolicyThreads);  // cnt is reused below
  // the n_cand lowest means of the first scope: threshold search on the n_cand-th, then everything up to it
  const int n_cand = need < m ? need : m;
  const uint32_t Tm = radix_select<uint32_t>([&](int j) { return __float_as_uint(mkey[j]); }, [&](int) { return true; },
                                             live0, (uint32_t)(n_cand - 1), *sel, ptid, kMqPolicyThreads, kMqBarPolicy,
                                             &rank, &ties);
  int Pm = 0x7fffffff;
  if (ties != rank + 1) {
    uint32_t r2, t2;
    Pm = (int)radix_select<uint32_t>([&](int j) { return (uint32_t)opos[j]; },
                                     [&](int j) { return __float_as_uint(mkey[j]) == Tm; }, live0, rank, *sel, ptid,
                                     kMqPolicyThreads, kMqBarPolicy, &r2, &t2);
  }
  if (ptid == 0) *cnt = 0;
  named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
  for (int j = ptid; j < live0; j += kMqPolicyThreads) {
    const uint32_t k = __float_as_uint(mkey[j]);
    if (k < 0x7f800000u && (k < Tm || (k == Tm && (Pm == 0x7fffffff || opos[j] <= Pm)))) {
      const int at = atomicAdd(cnt, 1);
      if (at < kMqMaxQ) list[at] = j;
    }
  }
  named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
  bool ok = *cnt == n_cand;
  if (pwarp == 0) {
    // lanes 0-15: the candidates of the first scope; lanes 16-31: the admits, ranked in (variance, position) order
    const bool is_adm = plane >= 16;
    const int idx = is_adm ? plane - 16 : plane;
    const bool has = is_adm ? idx < n_adm : idx < n_cand;
    int slot = -1, pj = 0x7fffffff;
    float mean = INFINITY;
    uint32_t vk = 0xffffffffu;
    if (has) {
      slot = is_adm ? adm_slot[idx] : list[idx];
      if (slot < 0 || slot >= live0) slot = 0;  // only after corrupt statistics
      mean = is_adm ? adm_mean[idx] : mkey[slot];
      pj = opos[slot];
      vk = vkey[slot];
    }
    int ord = 0;
#pragma unroll
    for (int i = 16; i < 32; ++i) {
      const uint32_t ovk = __shfl_sync(0xffffffffu, vk, i);
      const int op = __shfl_sync(0xffffffffu, pj, i);
      const bool oh = __shfl_sync(0xffffffffu, (int)has, i) != 0;
      if (oh && (ovk < vk || (ovk == vk && op < pj))) ++ord;
    }
    bool in_scope = has && !is_adm, gone = false;
    int n_admitted = 0;
#pragma unroll 1
    for (int it = 0; it < need; ++it) {
      if (it > 0 && r <= live0 - it && n_admitted < n_adm) {  // the scope has lost a token: the next one enters
        if (has && is_adm && ord == n_admitted) in_scope = true;
        ++n_admitted;
      }
      float bm = (in_scope && !gone) ? mean : INFINITY;
      int bp = pj, bs = (in_scope && !gone) ? slot : -1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, bm, o);
        const int op = __shfl_xor_sync(0xffffffffu, bp, o);
        const int os = __shfl_xor_sync(0xffffffffu, bs, o);
        if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
      }
      if (bs < 0) { ok = false; bs = it; }  // only after corrupt statistics; keeps the slots distinct
      else if (in_scope && !gone && slot == bs) gone = true;
      if (plane == 0) list[it] = bs;
    }
    if (!ok && plane == 0) atomicOr(status, ROCO_DEV_BAD_VICTIM);
  }
  named_bar_sync(kMqBarPolicy, kMqPolicyThreads);
}

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
    // the kn smallest of mkey by radix select on the kn-th, then one pass that collects everything up to it
    auto collect_lowest = [&](int kn, uint32_t m_and, uint32_t m_or) {
      const uint32_t Tm = radix_select<uint32_t>([&](int j) { return __float_as_uint(v.mkey[j]); },
                                                 [&](int) { return true; }, live0, (uint32_t)(kn - 1), *v.sel, ptid,
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
      return *cnt == kn;
    };

    // A scope that leaves out only a few tokens almost always contains the `need` tokens of lowest mean.  So
    // those are picked first, over all cached tokens, and then tested: the one of them that comes last in
    // (variance, position) order is in scope iff fewer than m tokens come before it, and then so are the others
    // (they come before it too) -- one counting pass in place of the radix select for the scope threshold.
    bool done = false;
    if (need > 1 && p.scope_mode == ROCO_SCOPE_LOWEST_R && m < live0) {
      lowest_r_block_victims(v.vkey, v.mkey, v.sel, v.ctl, opos, p.status, p.r, live0, need, m, k_and, k_or, ptid);
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
        ok = collect_lowest(need, m_and, m_or);
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
      else ok = collect_lowest(need, 0u, 0xffffffffu);
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

// ---- the tcgen05 kernel (multi_umma.cu)
// Ring stages it would run with at budget B (two: two CTAs per SM; more: one CTA per SM), 0 if it does not fit.
int multi_um_pick_stages(int B, int nb);
// Whether it takes M query rows that belong to nb new tokens.
bool multi_um_rows(int M, int nb);
// Launches it with p.stages ring stages; -1 if the tensor maps could not be built (nothing was launched).
int launch_multi_step_umma(const MultiParams &p, const roco_cache &c, int U, cudaStream_t stream);

}  // namespace roco
