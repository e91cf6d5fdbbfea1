// One decode step of KV-constrained inference with RoCo eviction (Sec. 3, Sec. 4.3, Fig. 1) for calls with few
// units -- one layer of a small batch, or a few long sequences -- where one CTA per unit leaves most SMs idle.
// Here a thread-block CLUSTER of k CTAs (k = 2, 4 or 8) shares a unit: rank c streams the tiles of its own slot
// range and keeps that range's scores, probabilities and statistics to itself, and what the ranks have to agree
// on travels through distributed shared memory -- never through global memory, whose round trips queue behind
// the streamed tiles for microseconds:
//   - every rank is organised like the one-CTA-per-unit kernel: a producer warp (bulk asynchronous copies of the
//     rank's K tiles, then its V tiles, non-multicast, through a ring), eight consumer warps, four policy warps;
//   - softmax: each rank reduces its own scores to (max, sum of exp2(z - max)); the pairs are pushed into every
//     rank's shared memory, and all ranks derive the same merged maximum and denominator of Eq. 1;
//   - output: each rank's partial sum of p*V is pushed to rank 0, which adds them up and stores the result;
//   - eviction scope and victim (Sec. 4.3): a most-significant-digit radix select that runs on all ranks in
//     lockstep -- local digit histograms are pushed to every rank and added up there, so every rank takes the
//     same decisions -- then the argmin of the mean among the in-scope tokens, again by exchanging one candidate
//     per rank.  The rank that owns the victim's slot overwrites it in place;
//   - statistics (Acc, Acc^square, Count): each rank updates its own slots.
// Two groups exchange independently (the consumers, the policy warps).  A push is an asynchronous store into the
// peer's shared memory that completes bytes on the peer's transaction barrier (st.async ... complete_tx), so the
// data and its arrival signal travel together, one way: whatever enters an SM queues behind the tiles that SM
// has requested, and a push, a fence that waits for its acknowledgement and a separate arrive would pay that
// queue three times.  The receiver's leader thread posts the bytes it expects and the group waits on its own
// barrier.  Barriers and buffers are double-buffered by phase parity (a peer can be at most one phase ahead).
// All waits are bounded.  The cluster's CTAs are co-scheduled by the hardware, so waiting on a peer is legitimate.
#include "common.cuh"
#include "launch.h"
#include "select.cuh"

namespace roco {

constexpr int kClConsumerWarps = 8;
constexpr int kClConsumers = kClConsumerWarps * 32;
constexpr int kClProducerWarp = kClConsumerWarps;
constexpr int kClPolicyWarp0 = kClConsumerWarps + 1;
constexpr int kClPolicyWarps = 4;
constexpr int kClPolicyThreads = kClPolicyWarps * 32;
constexpr int kClThreads = kClConsumers + 32 + kClPolicyThreads;
constexpr int kClTile = 16384;
constexpr int kClBarConsumers = 1;  // named barrier ids
constexpr int kClBarPolicy = 2;
constexpr int kClMaxRanks = 8;

struct ClusterParams {
  const char *K, *V;
  float *s, *q;
  int *n, *pos, *live, *t_next, *status;
  const char *qv, *k_new, *v_new;
  char *out;
  float *lse;
  int *ev_slot, *ev_pos;
  int B, r, scope_mode, order, stages;
  int k;    // CTAs per unit (cluster size)
  int tpr;  // tiles per rank
  float scale;
};

struct ClSmem {
  char *ring;
  float *z;          // [Bc] scores, then probabilities, of this rank's slots
  uint32_t *vkey;    // [Bc] staged Acc, then variance keys
  float *mkey;       // [Bc] staged Acc^square, then mean keys
  int *nbuf;         // [Bc] staged Count
  int *posb;         // [Bc] staged positions
  SelectScratch *sel;
  float *qf, *vnew, *knew, *outred, *red;
  uint32_t *xh;      // [2][k][128] policy exchange: digit histograms, two 16-bit counts per word
  uint32_t *xs;      // [2][k][4]   policy exchange: small records
  float *xc;         // [2][k][2]   consumer exchange: (max, sum) per rank
  float *xo;         // [k][D]      partial outputs (read by rank 0)
  uint64_t *full, *empty;
  uint64_t *p_ready, *policy_done, *stats_full, *v_done;
  uint64_t *xbar_c, *xbar_p;  // [2] each: transaction barriers of the two groups' exchanges, by phase parity
  int *ctl;          // [0] abort flag, [1] slot of the new token (unit-wide index)
};

__host__ __device__ inline size_t cluster_smem_bytes(int Bc, int d, int stages, int k) {
  size_t b = (size_t)stages * kClTile;
  b += 5 * (size_t)Bc * 4;                        // z, vkey, mkey, nbuf, posb
  b += sizeof(SelectScratch);
  b += (size_t)(3 + kClConsumerWarps) * d * 4;    // qf, vnew, knew, outred
  b += 64 * 4;                                    // red
  b += (size_t)2 * k * 128 * 4 + (size_t)2 * k * 4 * 4 + (size_t)2 * k * 2 * 4 + (size_t)k * d * 4;
  b += (2 * (size_t)stages + 8) * sizeof(uint64_t);
  b += 8 * 4;
  return b + 128;
}

__device__ inline ClSmem cluster_carve(char *raw, int Bc, int d, int stages, int k) {
  ClSmem m;
  char *p = smem_align(raw, 128);
  m.ring = p; p += (size_t)stages * kClTile;
  m.z = (float *)p; p += (size_t)Bc * 4;
  m.vkey = (uint32_t *)p; p += (size_t)Bc * 4;
  m.mkey = (float *)p; p += (size_t)Bc * 4;
  m.nbuf = (int *)p; p += (size_t)Bc * 4;
  m.posb = (int *)p; p += (size_t)Bc * 4;
  m.sel = (SelectScratch *)p; p += sizeof(SelectScratch);
  m.qf = (float *)p; p += d * 4;
  m.vnew = (float *)p; p += d * 4;
  m.knew = (float *)p; p += d * 4;
  m.outred = (float *)p; p += (size_t)kClConsumerWarps * d * 4;
  m.red = (float *)p; p += 64 * 4;
  m.xh = (uint32_t *)p; p += (size_t)2 * k * 128 * 4;
  m.xs = (uint32_t *)p; p += (size_t)2 * k * 4 * 4;
  m.xc = (float *)p; p += (size_t)2 * k * 2 * 4;
  m.xo = (float *)p; p += (size_t)k * d * 4;
  m.full = (uint64_t *)p; p += stages * sizeof(uint64_t);
  m.empty = (uint64_t *)p; p += stages * sizeof(uint64_t);
  m.p_ready = (uint64_t *)p; p += sizeof(uint64_t);
  m.policy_done = (uint64_t *)p; p += sizeof(uint64_t);
  m.stats_full = (uint64_t *)p; p += sizeof(uint64_t);
  m.v_done = (uint64_t *)p; p += sizeof(uint64_t);
  m.xbar_c = (uint64_t *)p; p += 2 * sizeof(uint64_t);
  m.xbar_p = (uint64_t *)p; p += 2 * sizeof(uint64_t);
  m.ctl = (int *)p;
  return m;
}

// ---------------------------------------------------------------- cluster primitives (PTX)

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}

// Address of the same shared-memory location in the CTA of rank `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_rank(const void *local, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(local)), "r"(rank));
  return r;
}

// Asynchronous store of one word into a peer's shared memory; on landing it completes 4 bytes on the peer's
// transaction barrier `remote_bar`.
__device__ __forceinline__ void push_u32(uint32_t remote, uint32_t v, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];" ::"r"(remote), "r"(v),
               "r"(remote_bar)
               : "memory");
}

// All threads of all CTAs of the cluster.
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// One thread group's side of the exchanges: its pair of transaction barriers and the phases it has been through.
struct Exchange {
  uint64_t *bars;  // [2]
  uint32_t phase;
  int k, gt, gsize, bar_id;
  volatile int *abort_flag;
  int32_t *status;
  __device__ __forceinline__ int parity() const { return (int)(phase & 1u); }
  // One word of this phase into `slot` (a location of this CTA's layout) on rank r.
  __device__ __forceinline__ void push(const void *slot, int r, uint32_t v) const {
    push_u32(map_to_rank(slot, r), v, map_to_rank(&bars[phase & 1u], r));
  }
  __device__ __forceinline__ void push(const void *slot, int r, float v) const { push(slot, r, __float_as_uint(v)); }
  // Called by every thread of the group after its pushes of this phase; expect_bytes: what all ranks together push
  // into THIS CTA in this phase.  Returns once all of it has landed.  (The group barrier keeps a thread that is
  // still reading the data of two phases ago from being overtaken by the pushes that will replace it.)
  __device__ __forceinline__ void sync(uint32_t expect_bytes) {
    named_bar_sync(bar_id, gsize);
    uint64_t *bar = &bars[phase & 1u];
    if (gt == 0) mbar_expect_tx(bar, expect_bytes);
    mbar_wait(bar, (phase >> 1) & 1u, abort_flag, status);
    ++phase;
  }
};

// k-th smallest (0-based) of key(j) over this unit's slots with pred(j), where every rank holds the slots
// j in [0, nloc) of its own range: the cluster-wide counterpart of radix_select.  Called by the policy threads of
// all ranks in lockstep; every rank gets the same result.  (all_and, all_or): cluster-wide AND / OR of the keys.
template <typename KeyF, typename PredF>
__device__ __forceinline__ uint32_t cluster_radix_select(KeyF key, PredF pred, int nloc, uint32_t k_rank,
                                                         const ClSmem &sm, Exchange &x, int my_rank,
                                                         uint32_t *rank_in_ties, uint32_t *n_ties,
                                                         uint32_t all_and, uint32_t all_or) {
  SelectScratch &sc = *sm.sel;
  const int tid = x.gt, nthreads = x.gsize, lane = tid & 31;
  uint32_t prefix = 0, mask = 0, kk = k_rank;
  int shift0 = 24;
  {
    const uint32_t diff = all_and ^ all_or;
    while (shift0 > 0 && (diff >> shift0) == 0) shift0 -= 8;
    if (shift0 < 24) {
      mask = ~0u << (shift0 + 8);
      prefix = all_and & mask;
    }
  }
#pragma unroll 1
  for (int shift = shift0; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += nthreads) sc.hist[i] = 0;
    named_bar_sync(x.bar_id, nthreads);
#pragma unroll 4
    for (int j = tid; j < nloc; j += nthreads) {
      if (pred(j)) {
        const uint32_t v = key(j);
        if ((v & mask) == prefix) smem_red_add(&sc.hist[(v >> shift) & 255u], 1u);
      }
    }
    named_bar_sync(x.bar_id, nthreads);
    // this rank's histogram goes to every rank, two 16-bit counts per word (a rank holds at most 8192 slots)
    const int par = x.parity();
    if (tid < 128) {
      const uint32_t packed = sc.hist[2 * tid] | (sc.hist[2 * tid + 1] << 16);
      uint32_t *slot = sm.xh + ((size_t)(par * x.k + my_rank) * 128 + tid);
      for (int r = 0; r < x.k; ++r) x.push(slot, r, packed);
    }
    x.sync((uint32_t)x.k * 512u);
    if (tid < 128) {
      uint32_t t0 = 0, t1 = 0;
      for (int r = 0; r < x.k; ++r) {
        const uint32_t w = sm.xh[(size_t)(par * x.k + r) * 128 + tid];
        t0 += w & 0xffffu;
        t1 += w >> 16;
      }
      sc.hist[2 * tid] = t0;
      sc.hist[2 * tid + 1] = t1;
    }
    named_bar_sync(x.bar_id, nthreads);
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
      const uint32_t excl = incl - total;
      if (kk >= excl && kk < incl) {
        uint32_t rem = kk - excl;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (rem < c[i]) { sc.digit = lane * 8 + i; sc.rank = rem; sc.count = c[i]; break; }
          rem -= c[i];
        }
      }
    }
    named_bar_sync(x.bar_id, nthreads);
    prefix |= sc.digit << shift;
    mask |= 255u << shift;
    kk = sc.rank;
  }
  *rank_in_ties = kk;
  *n_ties = sc.count;
  named_bar_sync(x.bar_id, nthreads);
  return prefix;
}

// Victim slot (unit-wide index) among the unit's B occupied slots given scope size m (1 <= m <= B), from the keys
// every rank holds for its own slots [j0, j0 + nloc): vkey (variance), mkey (mean), posb (position).  (k_and, k_or):
// this thread's AND / OR over the variance keys it formed.  Same result on every rank; -1 if no slot qualifies.
__device__ __forceinline__ int cluster_select_victim(const ClSmem &sm, Exchange &x, int my_rank, int j0, int nloc,
                                                     int B, int m, uint32_t k_and, uint32_t k_or) {
  SelectScratch &sc = *sm.sel;
  const int tid = x.gt, nthreads = x.gsize;
  // A scope that leaves out only a few tokens almost always contains the token of lowest mean.  So: take the
  // tokens in (mean, position) order and test each for membership by counting the tokens before it in
  // (variance, position) order -- two exchanges per candidate instead of one per radix digit.  (Whatever enters an
  // SM, a peer's push included, queues behind the tiles that SM has requested: an exchange costs microseconds,
  // and their number is what the selection's latency is made of.)  The first candidate's exchange also carries a
  // histogram of the variance keys' exponent bytes: if the tokens whose exponent is not above the candidate's are
  // at most m, all of them are in scope and the count is not needed.  After three candidates outside the scope
  // the radix select below takes over.
  if (2 * m >= B) {
    int excl[3] = {-1, -1, -1};
    for (int i = tid; i < 256; i += nthreads) sc.hist[i] = 0;
    named_bar_sync(x.bar_id, nthreads);
#pragma unroll 4
    for (int j = tid; j < nloc; j += nthreads) smem_red_add(&sc.hist[sm.vkey[j] >> 24], 1u);
    for (int attempt = 0; attempt < 3; ++attempt) {
      float bm = INFINITY;
      int bs = -1, bp = 0x7fffffff;
#pragma unroll 4
      for (int j = tid; j < nloc; j += nthreads) {
        const int gj = j0 + j;
        if (gj == excl[0] || gj == excl[1] || gj == excl[2]) continue;
        const float mean = sm.mkey[j];
        if (mean < bm || (mean == bm && sm.posb[j] < bp)) { bm = mean; bs = j; bp = sm.posb[j]; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, bm, o);
        const int op = __shfl_xor_sync(0xffffffffu, bp, o);
        const int os = __shfl_xor_sync(0xffffffffu, bs, o);
        if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
      }
      const int warp = tid >> 5, nwarps = nthreads >> 5;
      if ((tid & 31) == 0) { sc.red_mean[warp] = bm; sc.red_pos[warp] = bp; sc.red_slot[warp] = bs; }
      named_bar_sync(x.bar_id, nthreads);
      bm = sc.red_mean[0]; bp = sc.red_pos[0]; bs = sc.red_slot[0];
      for (int w = 1; w < nwarps; ++w) {
        const float om = sc.red_mean[w];
        const int op = sc.red_pos[w], os = sc.red_slot[w];
        if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
      }
      uint32_t cv = 0;
      {
        const int par = x.parity();
        if (tid < x.k) {
          uint32_t *slot = sm.xs + (size_t)(par * x.k + my_rank) * 4;
          x.push(slot, tid, bm);
          x.push(slot + 1, tid, (uint32_t)bp);
          x.push(slot + 2, tid, (uint32_t)(bs >= 0 ? j0 + bs : -1));
          x.push(slot + 3, tid, bs >= 0 ? sm.vkey[bs] : 0u);
        }
        if (attempt == 0 && tid < 128) {  // (the barrier of the reduction above has published the histogram)
          const uint32_t packed = sc.hist[2 * tid] | (sc.hist[2 * tid + 1] << 16);
          uint32_t *slot = sm.xh + ((size_t)(par * x.k + my_rank) * 128 + tid);
          for (int r = 0; r < x.k; ++r) x.push(slot, r, packed);
        }
        x.sync((uint32_t)x.k * (attempt == 0 ? 16u + 512u : 16u));
        bm = INFINITY; bp = 0x7fffffff; bs = -1;
        for (int r = 0; r < x.k; ++r) {
          const uint32_t *rec = sm.xs + (size_t)(par * x.k + r) * 4;
          const float om = __uint_as_float(rec[0]);
          const int op = (int)rec[1], os = (int)rec[2];
          if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; cv = rec[3]; }
        }
      }
      if (bs < 0) return -1;  // no candidate left (NaN statistics)
      if (attempt == 0) {
        // tokens of the whole unit whose exponent byte is at most the candidate's
        const int par = (int)((x.phase - 1u) & 1u);
        const uint32_t ce = cv >> 24;
        uint32_t below = 0;
        if (tid < 128) {
          uint32_t t0 = 0, t1 = 0;
          for (int r = 0; r < x.k; ++r) {
            const uint32_t w = sm.xh[(size_t)(par * x.k + r) * 128 + tid];
            t0 += w & 0xffffu;
            t1 += w >> 16;
          }
          below = ((uint32_t)(2 * tid) <= ce ? t0 : 0u) + ((uint32_t)(2 * tid + 1) <= ce ? t1 : 0u);
        }
        below = __reduce_add_sync(0xffffffffu, below);
        if ((tid & 31) == 0) sc.red_slot[warp] = (int)below;
        named_bar_sync(x.bar_id, nthreads);
        below = 0;
        for (int w = 0; w < nwarps; ++w) below += (uint32_t)sc.red_slot[w];
        if (below <= (uint32_t)m) return bs;
      }
      // tokens before the candidate in (variance, position) order: it is in scope iff there are fewer than m
      uint32_t cnt = 0;
#pragma unroll 4
      for (int j = tid; j < nloc; j += nthreads) {
        const uint32_t kv = sm.vkey[j];
        cnt += (kv < cv || (kv == cv && sm.posb[j] < bp)) ? 1u : 0u;
      }
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      if ((tid & 31) == 0) sc.red_pos[warp] = (int)cnt;
      named_bar_sync(x.bar_id, nthreads);
      cnt = 0;
      for (int w = 0; w < nwarps; ++w) cnt += (uint32_t)sc.red_pos[w];
      {
        const int par = x.parity();
        if (tid < x.k) x.push(sm.xs + (size_t)(par * x.k + my_rank) * 4, tid, cnt);
        x.sync((uint32_t)x.k * 4u);
        cnt = 0;
        for (int r = 0; r < x.k; ++r) cnt += sm.xs[(size_t)(par * x.k + r) * 4];
      }
      if (cnt < (uint32_t)m) return bs;
      excl[attempt] = bs;
    }
  }
  uint32_t T = 0xffffffffu;
  int P = 0x7fffffff;
  if (m < B) {
    group_and_or(k_and, k_or, sc, tid, nthreads, x.bar_id);
    {  // cluster-wide AND / OR
      const int par = x.parity();
      if (tid < x.k) {
        uint32_t *slot = sm.xs + (size_t)(par * x.k + my_rank) * 4;
        x.push(slot, tid, k_and);
        x.push(slot + 1, tid, k_or);
      }
      x.sync((uint32_t)x.k * 8u);
      for (int r = 0; r < x.k; ++r) {
        k_and &= sm.xs[(size_t)(par * x.k + r) * 4];
        k_or |= sm.xs[(size_t)(par * x.k + r) * 4 + 1];
      }
    }
    uint32_t rank, ties;
    T = cluster_radix_select([&](int j) { return sm.vkey[j]; }, [&](int) { return true; }, nloc, (uint32_t)(m - 1),
                             sm, x, my_rank, &rank, &ties, k_and, k_or);
    if (ties != rank + 1) {  // only some of the tokens tied at the threshold are in scope: lowest positions
      uint32_t r2, t2;
      P = (int)cluster_radix_select([&](int j) { return (uint32_t)sm.posb[j]; },
                                    [&](int j) { return sm.vkey[j] == T; }, nloc, rank, sm, x, my_rank, &r2, &t2,
                                    0u, 0xffffffffu);
    }
  }
  // in-scope token of lowest mean, ties to the lowest position: this rank's candidate, then one per rank
  float bm = INFINITY;
  int bs = -1, bp = 0x7fffffff;
#pragma unroll 4
  for (int j = tid; j < nloc; j += nthreads) {
    const uint32_t kv = sm.vkey[j];
    if (kv > T) continue;
    const int pj = sm.posb[j];
    if (kv == T && P != 0x7fffffff && pj > P) continue;
    const float mean = sm.mkey[j];
    if (mean < bm || (mean == bm && pj < bp)) { bm = mean; bs = j; bp = pj; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, bm, o);
    const int op = __shfl_xor_sync(0xffffffffu, bp, o);
    const int os = __shfl_xor_sync(0xffffffffu, bs, o);
    if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
  }
  const int warp = tid >> 5, nwarps = nthreads >> 5;
  if ((tid & 31) == 0) { sc.red_mean[warp] = bm; sc.red_pos[warp] = bp; sc.red_slot[warp] = bs; }
  named_bar_sync(x.bar_id, nthreads);
  bm = sc.red_mean[0]; bp = sc.red_pos[0]; bs = sc.red_slot[0];
  for (int w = 1; w < nwarps; ++w) {
    const float om = sc.red_mean[w];
    const int op = sc.red_pos[w], os = sc.red_slot[w];
    if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
  }
  {
    const int par = x.parity();
    if (tid < x.k) {
      uint32_t *slot = sm.xs + (size_t)(par * x.k + my_rank) * 4;
      x.push(slot, tid, bm);
      x.push(slot + 1, tid, (uint32_t)bp);
      x.push(slot + 2, tid, (uint32_t)(bs >= 0 ? j0 + bs : -1));
    }
    x.sync((uint32_t)x.k * 12u);
    bm = INFINITY; bp = 0x7fffffff; bs = -1;
    for (int r = 0; r < x.k; ++r) {
      const float om = __uint_as_float(sm.xs[(size_t)(par * x.k + r) * 4]);
      const int op = (int)sm.xs[(size_t)(par * x.k + r) * 4 + 1], os = (int)sm.xs[(size_t)(par * x.k + r) * 4 + 2];
      if (os >= 0 && (bs < 0 || om < bm || (om == bm && op < bp))) { bm = om; bp = op; bs = os; }
    }
  }
  return bs;
}

__device__ __forceinline__ float cl_consumers_max(float v, float *red, int tid) {
  v = warp_max(v);
  if ((tid & 31) == 0) red[tid >> 5] = v;
  named_bar_sync(kClBarConsumers, kClConsumers);
  float r = red[0];
#pragma unroll
  for (int w = 1; w < kClConsumerWarps; ++w) r = fmaxf(r, red[w]);
  return r;
}

__device__ __forceinline__ float cl_consumers_sum(float v, float *red, int tid) {
  v = warp_sum(v);
  if ((tid & 31) == 0) red[16 + (tid >> 5)] = v;
  named_bar_sync(kClBarConsumers, kClConsumers);
  float r = red[16];
#pragma unroll
  for (int w = 1; w < kClConsumerWarps; ++w) r += red[16 + w];
  return r;
}

template <typename T, int D>
__global__ void __launch_bounds__(kClThreads, 2) decode_cluster_kernel(const ClusterParams p) {
  constexpr int kRowBytes = D * (int)sizeof(T);
  constexpr int kLanesPerRow = kRowBytes / 16;
  constexpr int kRowsPerLoad = 32 / kLanesPerRow;
  constexpr int kTileRows = kClTile / kRowBytes;
  constexpr int kRowsPerWarp = kTileRows / kClConsumerWarps;
  constexpr int kLoads = kRowsPerWarp / kRowsPerLoad;
  constexpr int kEPC = Elem<T>::kPerChunk;
  static_assert(kLanesPerRow <= 32 && kLoads >= 1, "tile shape");

  extern __shared__ char cl_smem_raw[];
  const int k = p.k, Bc = p.tpr * kTileRows;
  const ClSmem sm = cluster_carve(cl_smem_raw, Bc, D, p.stages, k);
  volatile int *abort_flag = sm.ctl;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rank = (int)cluster_ctarank();
  const int u = blockIdx.x / k;
  const int B = p.B, stages = p.stages;
  const size_t unit_kv = (size_t)u * B * kRowBytes;
  const size_t unit_st = (size_t)u * B;

  if (tid == 0) {
    for (int i = 0; i < stages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], kClConsumerWarps); }
    mbar_init(sm.p_ready, kClConsumerWarps);
    mbar_init(sm.policy_done, 1);
    mbar_init(sm.stats_full, 1);
    mbar_init(sm.v_done, kClConsumerWarps);
    for (int i = 0; i < 2; ++i) { mbar_init(&sm.xbar_c[i], 1); mbar_init(&sm.xbar_p[i], 1); }
    sm.ctl[0] = 0;
    mbar_init_fence();
  }
  // Every thread reads the unit's occupancy and next position BEFORE the cluster-wide barrier: the rank that owns
  // the new token's slot rewrites them later, and by then every rank has them.
  int live0 = p.live[u];
  const int t_new = p.t_next[u];
  if (live0 < 0 || live0 > B) {
    if (tid == 0 && rank == 0) atomicOr(p.status, ROCO_DEV_BAD_LIVE);
    live0 = live0 < 0 ? 0 : B;
  }
  cluster_sync_all();  // barriers initialised on every rank before anyone arrives on them remotely

  const bool full = (live0 == B);
  const bool evict_first = (p.order == ROCO_EVICT_FIRST);
  const int live_att = evict_first ? (full ? B : live0 + 1) : live0;  // slots the query attends over
  const int n_tiles_att = (live_att + kTileRows - 1) / kTileRows;
  const int t_begin = rank * p.tpr;
  int t_end = t_begin + p.tpr;
  if (t_end > n_tiles_att) t_end = n_tiles_att;
  const int n_tiles = t_end > t_begin ? t_end - t_begin : 0;  // tiles this rank streams
  const int j0 = t_begin * kTileRows;                         // first slot of this rank's range
  int nloc_att = live_att - j0;                               // attended slots of this rank
  if (nloc_att < 0) nloc_att = 0;
  if (nloc_att > Bc) nloc_att = Bc;
  int nloc_full = B - j0;                                     // slots of this rank when the cache is full
  if (nloc_full < 0) nloc_full = 0;
  if (nloc_full > Bc) nloc_full = Bc;

  if (warp == kClProducerWarp) {
    // ------------------------------------------------------------ producer: statistics, K tiles, then V tiles
    if (lane == 0) {
      if (full && nloc_full > 0) {  // the selection's inputs, ahead of the tiles
        const uint32_t bytes = (uint32_t)nloc_full * 4;
        mbar_expect_tx(sm.stats_full, 4 * bytes);
        bulk_g2s(sm.vkey, p.s + unit_st + j0, bytes, sm.stats_full);
        bulk_g2s(sm.mkey, p.q + unit_st + j0, bytes, sm.stats_full);
        bulk_g2s(sm.nbuf, p.n + unit_st + j0, bytes, sm.stats_full);
        bulk_g2s(sm.posb, p.pos + unit_st + j0, bytes, sm.stats_full);
      }
      for (int g = 0; g < 2 * n_tiles; ++g) {
        const int st = g % stages;
        if (g >= stages) mbar_wait(&sm.empty[st], ((g / stages) - 1) & 1, abort_flag, p.status);
        const int it = t_begin + ((g < n_tiles) ? g : g - n_tiles);
        const char *src = ((g < n_tiles) ? p.K : p.V) + unit_kv + (size_t)it * kClTile;
        int rows = live_att - it * kTileRows;
        if (rows > kTileRows) rows = kTileRows;
        const uint32_t bytes = (uint32_t)rows * kRowBytes;
        mbar_expect_tx(&sm.full[st], bytes);
        bulk_g2s(sm.ring + (size_t)st * kClTile, src, bytes, &sm.full[st]);
      }
    }
  } else if (warp >= kClPolicyWarp0) {
    // ------------------------------------------------------------ policy: scope, victim, overwrite, statistics
    const int ptid = tid - kClPolicyWarp0 * 32;
    Exchange x{sm.xbar_p, 0u, k, ptid, kClPolicyThreads, kClBarPolicy, abort_flag, p.status};
    // statistics of Sec. 4.3 for this rank's attended slots: Acc += p, Acc^square += p^2, Count += 1 (a slot that
    // has just received the new token starts from zero).  with_keys: the statistics come from the staged copies
    // and the selection keys of the updated values are left in their place (ATTEND_FIRST, full cache).
    uint32_t k_and = 0xffffffffu, k_or = 0u;
    auto update_statistics = [&](int fresh_slot, bool with_keys) {
      mbar_wait(sm.p_ready, 0, abort_flag, p.status);
      constexpr int kBatch = 4;
      for (int l0 = ptid; l0 < nloc_att; l0 += kBatch * kClPolicyThreads) {
        float s0[kBatch], q0[kBatch];
        int n0[kBatch];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
          const int l = l0 + b * kClPolicyThreads, j = j0 + l;
          const bool old = l < nloc_att && j != fresh_slot && j < live0;
          if (with_keys) {
            s0[b] = old ? __uint_as_float(sm.vkey[l]) : 0.f;
            q0[b] = old ? sm.mkey[l] : 0.f;
            n0[b] = old ? sm.nbuf[l] : 0;
          } else {
            s0[b] = old ? p.s[unit_st + j] : 0.f;
            q0[b] = old ? p.q[unit_st + j] : 0.f;
            n0[b] = old ? p.n[unit_st + j] : 0;
          }
        }
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
          const int l = l0 + b * kClPolicyThreads, j = j0 + l;
          if (l >= nloc_att) break;
          const float pj = sm.z[l];
          const float s1 = s0[b] + pj, q1 = fmaf(pj, pj, q0[b]);
          const int n1 = n0[b] + 1;
          p.s[unit_st + j] = s1;
          p.q[unit_st + j] = q1;
          p.n[unit_st + j] = n1;
          if (with_keys) {
            const uint32_t vk = variance_key_fast(s1, q1, n1);
            sm.vkey[l] = vk;
            sm.mkey[l] = mean_fast(s1, n1);
            k_and &= vk;
            k_or |= vk;
          }
        }
      }
    };
    // the part of k_new / v_new this thread will write into the freed slot (raw bytes: nothing waits for them
    // before the store)
    const bool writes_row = ptid >= 32 && ptid < 32 + 2 * kLanesPerRow;
    uint4 row_val = make_uint4(0u, 0u, 0u, 0u);
    if (writes_row) {
      const int c = ptid - 32;
      const bool isv = c >= kLanesPerRow;
      row_val = *((const uint4 *)((isv ? p.v_new : p.k_new) + (size_t)u * kRowBytes) + (isv ? c - kLanesPerRow : c));
    }
    int e = live0;
    if (full) {
      // Sec. 4, fixed-budget buffer: eviction runs only once the buffer is full
      const int m = scope_size(B, p.r, p.scope_mode);
      if (nloc_full > 0) mbar_wait(sm.stats_full, 0, abort_flag, p.status);
      if (evict_first) {  // keys of the statistics as they stand, formed in place
#pragma unroll 4
        for (int l = ptid; l < nloc_full; l += kClPolicyThreads) {
          const float sj = __uint_as_float(sm.vkey[l]);
          const uint32_t vk = variance_key_fast(sj, sm.mkey[l], sm.nbuf[l]);
          sm.mkey[l] = mean_fast(sj, sm.nbuf[l]);
          sm.vkey[l] = vk;
          k_and &= vk;
          k_or |= vk;
        }
      } else {  // keys of the updated statistics
        update_statistics(-1, true);
      }
      e = cluster_select_victim(sm, x, rank, j0, nloc_full, B, m, k_and, k_or);
      if (e < 0) {
        if (ptid == 0 && rank == 0) atomicOr(p.status, ROCO_DEV_BAD_VICTIM);
        e = 0;
      }
    } else if (!evict_first) {
      update_statistics(-1, false);
    }
    // the rank that owns slot e inserts the new token there
    const bool owner = (e >= j0 && e < j0 + Bc);
    if (owner) {
      if (ptid == 0) {
        p.ev_slot[u] = full ? e : -1;
        if (p.ev_pos) p.ev_pos[u] = full ? sm.posb[e - j0] : -1;
        p.pos[unit_st + e] = t_new;
        p.live[u] = full ? B : live0 + 1;
        p.t_next[u] = t_new + 1;
        if (!evict_first) { p.s[unit_st + e] = 0.f; p.q[unit_st + e] = 0.f; p.n[unit_st + e] = 0; }
      }
      if (writes_row) {  // in-place overwrite, 16 bytes per thread
        const int c = ptid - 32;
        const bool isv = c >= kLanesPerRow;
        // ATTEND_FIRST attends over the cache as it stood: the victim's value row goes only once this rank's
        // consumers have their last V tile behind them (the key row's pass has ended by then in any case)
        if (isv && !evict_first && full) mbar_wait(sm.v_done, 0, abort_flag, p.status);
        char *dst = const_cast<char *>(isv ? p.V : p.K) + unit_kv + (size_t)e * kRowBytes;
        *((uint4 *)dst + (isv ? c - kLanesPerRow : c)) = row_val;
      }
    }
    if (ptid == 0) sm.ctl[1] = e;
    named_bar_sync(kClBarPolicy, kClPolicyThreads);
    if (ptid == 0) mbar_arrive(sm.policy_done);
    if (evict_first) update_statistics(e, false);
  } else {
    // ------------------------------------------------------------ consumers
    Exchange x{sm.xbar_c, 0u, k, tid, kClConsumers, kClBarConsumers, abort_flag, p.status};
    if (tid < D) {
      const size_t o = (size_t)u * D + tid;
      sm.qf[tid] = Elem<T>::load((const T *)p.qv + o);
      if (evict_first) {
        sm.vnew[tid] = Elem<T>::load((const T *)p.v_new + o);
        sm.knew[tid] = Elem<T>::load((const T *)p.k_new + o);
      }
    }
    named_bar_sync(kClBarConsumers, kClConsumers);

    // ---- scores of this rank's slots: z_j = scale * q.K[j]  (Eq. 1), kept in base 2
    const float zscale = p.scale * kLog2e;
    const int lane_chunk = lane % kLanesPerRow, lane_row = lane / kLanesPerRow;
    float qreg[kEPC];
#pragma unroll
    for (int i = 0; i < kEPC; ++i) qreg[i] = sm.qf[lane_chunk * kEPC + i];
    for (int it = 0; it < n_tiles; ++it) {
      const int st = it % stages;
      mbar_wait(&sm.full[st], (it / stages) & 1, abort_flag, p.status);
      const char *tile = sm.ring + (size_t)st * kClTile;
      float acc[kLoads];
#pragma unroll
      for (int l = 0; l < kLoads; ++l) {
        const int row = warp * kRowsPerWarp + l * kRowsPerLoad + lane_row;
        const uint4 c = *(const uint4 *)(tile + (size_t)row * kRowBytes + lane_chunk * 16);
        float f[kEPC];
        Elem<T>::unpack(c, f);
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
        const int jl = it * kTileRows + warp * kRowsPerWarp + l * kRowsPerLoad + lane_row;
        if (lane_chunk == 0 && jl < nloc_att) sm.z[jl] = acc[l] * zscale;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[st]);
    }

    // EVICT_FIRST: the slot that takes the new token gets its score and value from k_new / v_new, not from the
    // stream (which may have read the slot before or after the overwrite); it belongs to one rank.
    int e_sub = -1;
    if (evict_first) {
      mbar_wait(sm.policy_done, 0, abort_flag, p.status);
      const int e = sm.ctl[1];
      if (e >= j0 && e < j0 + nloc_att) e_sub = e - j0;
    }
    named_bar_sync(kClBarConsumers, kClConsumers);  // all scores are in shared memory
    if (warp == 0 && e_sub >= 0) {  // the new token's own score, from k_new directly
      float a = 0.f;
#pragma unroll
      for (int i = 0; i < D / 32; ++i) a = fmaf(sm.qf[lane + 32 * i], sm.knew[lane + 32 * i], a);
      a = warp_sum(a);
      if (lane == 0) sm.z[e_sub] = a * zscale;
    }
    named_bar_sync(kClBarConsumers, kClConsumers);

    // ---- softmax over the unit's occupied slots: local (max, sum), one exchange, merged (max, sum)
    float zmax = -INFINITY;
    for (int j = tid; j < nloc_att; j += kClConsumers) zmax = fmaxf(zmax, sm.z[j]);
    zmax = cl_consumers_max(zmax, sm.red, tid);
    float zsum = 0.f;
    for (int j = tid; j < nloc_att; j += kClConsumers) {
      const float ex = exp2f(sm.z[j] - zmax);
      sm.z[j] = ex;
      zsum += ex;
    }
    zsum = cl_consumers_sum(zsum, sm.red, tid);
    float M, L;
    {
      const int par = x.parity();
      if (tid < k) {
        float *slot = sm.xc + (size_t)(par * k + rank) * 2;
        x.push(slot, tid, zmax);
        x.push(slot + 1, tid, zsum);
      }
      x.sync((uint32_t)k * 8u);
      M = -INFINITY;
      for (int r = 0; r < k; ++r) M = fmaxf(M, sm.xc[(size_t)(par * k + r) * 2]);
      L = 0.f;
      for (int r = 0; r < k; ++r) {
        const float mr = sm.xc[(size_t)(par * k + r) * 2];
        if (mr > -INFINITY) L = fmaf(sm.xc[(size_t)(par * k + r) * 2 + 1], exp2f(mr - M), L);
      }
    }
    const float factor = (L > 0.f && zmax > -INFINITY) ? exp2f(zmax - M) / L : 0.f;
    for (int j = tid; j < nloc_att; j += kClConsumers) sm.z[j] *= factor;
    // hand the probabilities to the policy warps (statistics update) before streaming V
    __syncwarp();
    if (lane == 0) mbar_arrive(sm.p_ready);
    if (tid == 0 && rank == 0 && p.lse) p.lse[u] = (L > 0.f) ? (M + log2f(L)) * kLn2 : -INFINITY;
    named_bar_sync(kClBarConsumers, kClConsumers);  // all probabilities are in shared memory

    // ---- this rank's part of out = sum_j p_j V[j]
    float acc[kEPC];
#pragma unroll
    for (int i = 0; i < kEPC; ++i) acc[i] = 0.f;
    for (int it = 0; it < n_tiles; ++it) {
      const int g = n_tiles + it;
      const int st = g % stages;
      mbar_wait(&sm.full[st], (g / stages) & 1, abort_flag, p.status);
      const char *tile = sm.ring + (size_t)st * kClTile;
#pragma unroll
      for (int l = 0; l < kLoads; ++l) {
        const int row = warp * kRowsPerWarp + l * kRowsPerLoad + lane_row;
        const int jl = it * kTileRows + row;
        if (jl < nloc_att && jl != e_sub) {
          const uint4 c = *(const uint4 *)(tile + (size_t)row * kRowBytes + lane_chunk * 16);
          float f[kEPC];
          Elem<T>::unpack(c, f);
          const float pj = sm.z[jl];
#pragma unroll
          for (int i = 0; i < kEPC; ++i) acc[i] = fmaf(pj, f[i], acc[i]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[st]);
    }
    if (lane == 0) mbar_arrive(sm.v_done);  // this warp has read its share of every V tile
#pragma unroll
    for (int i = 0; i < kEPC; ++i) {
#pragma unroll
      for (int o = kLanesPerRow; o < 32; o <<= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
    }
    if (lane_row == 0) {
#pragma unroll
      for (int i = 0; i < kEPC; ++i) sm.outred[warp * D + lane_chunk * kEPC + i] = acc[i];
    }
    named_bar_sync(kClBarConsumers, kClConsumers);
    if (tid < D) {
      float o = 0.f;
#pragma unroll
      for (int w = 0; w < kClConsumerWarps; ++w) o += sm.outred[w * D + tid];
      if (e_sub >= 0) o = fmaf(sm.z[e_sub], sm.vnew[tid], o);
      x.push(sm.xo + (size_t)rank * D + tid, 0, o);  // to rank 0
    }
    x.sync(rank == 0 ? (uint32_t)k * D * 4u : 0u);
    if (rank == 0 && tid < D) {
      float o = 0.f;
      for (int r = 0; r < k; ++r) o += sm.xo[(size_t)r * D + tid];
      Elem<T>::store((T *)p.out + (size_t)u * D + tid, o);
    }
  }
  // No CTA leaves while a peer may still push into its shared memory or arrive on its barriers.
  __syncwarp();
  cluster_sync_all();
}

// CTAs per unit for a call of U units with budget B: the largest cluster (a power of two) whose CTAs still fit
// the GPU in one wave of two per SM, as long as every rank keeps at least two tiles; 1 = one CTA per unit is the
// better shape.
int decode_cluster_ranks(int U, int B, int d, int elem, int sms) {
  const int rows_per_tile = kClTile / (d * elem);
  const int tpu = (B + rows_per_tile - 1) / rows_per_tile;
  if ((B & 3) != 0) return 1;  // the staged statistics need 16-byte aligned slices
  int k = 1;
  while (k < kClMaxRanks && (long long)U * k * 2 <= (long long)sms * 2 && tpu / (2 * k) >= 2) k *= 2;
  return k;
}

template <typename T, int D>
static cudaError_t launch_cluster_t(const ClusterParams &p, int U, size_t smem, cudaStream_t stream) {
  cudaError_t err = cudaFuncSetAttribute(decode_cluster_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
  if (err != cudaSuccess) return err;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(U * p.k));
  cfg.blockDim = dim3(kClThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)p.k;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_cluster_kernel<T, D>, p);
}

roco_status launch_decode_step_cluster(const roco_cache &c, int ranks, const void *q, const void *k_new,
                                       const void *v_new, int r, int scope_mode, int step_order, float scale,
                                       void *out, float *lse, int32_t *ev_slot, int32_t *ev_pos, cudaStream_t stream) {
  const int U = c.S * c.G;
  const int elem = c.kv_dtype == ROCO_BF16 ? 2 : 4;
  if (ranks != 2 && ranks != 4 && ranks != 8) return ROCO_ERR_INVALID_ARG;
  if ((c.B & 3) != 0) return ROCO_ERR_UNSUPPORTED;
  if (((reinterpret_cast<uintptr_t>(c.s) | reinterpret_cast<uintptr_t>(c.q) | reinterpret_cast<uintptr_t>(c.n) |
        reinterpret_cast<uintptr_t>(c.pos)) & 15) != 0)
    return ROCO_ERR_UNSUPPORTED;
  ClusterParams p;
  p.K = (const char *)c.K; p.V = (const char *)c.V;
  p.s = c.s; p.q = c.q; p.n = c.n; p.pos = c.pos; p.live = c.live; p.t_next = c.t_next; p.status = c.status;
  p.qv = (const char *)q; p.k_new = (const char *)k_new; p.v_new = (const char *)v_new;
  p.out = (char *)out; p.lse = lse; p.ev_slot = ev_slot; p.ev_pos = ev_pos;
  p.B = c.B; p.r = r; p.scope_mode = scope_mode; p.order = step_order; p.scale = scale;
  p.k = ranks;
  const int rows_per_tile = kClTile / (c.d * elem);
  const int tpu = (c.B + rows_per_tile - 1) / rows_per_tile;
  p.tpr = (tpu + ranks - 1) / ranks;
  const int Bc = p.tpr * rows_per_tile;
  // the deepest ring (3..8 stages) that lets two CTAs share an SM, else one
  const size_t per_sm = 227 * 1024;
  int stages = 0;
  for (int ctas = 2; ctas >= 1 && !stages; --ctas)
    for (int st = 8; st >= 3; --st)
      if ((cluster_smem_bytes(Bc, c.d, st, ranks) + 1024) * ctas <= per_sm) { stages = st; break; }
  if (!stages) return ROCO_ERR_UNSUPPORTED;
  p.stages = stages;
  const size_t smem = cluster_smem_bytes(Bc, c.d, stages, ranks);
  cudaError_t err;
  if (c.kv_dtype == ROCO_BF16 && c.d == 128) err = launch_cluster_t<__nv_bfloat16, 128>(p, U, smem, stream);
  else if (c.kv_dtype == ROCO_BF16 && c.d == 64) err = launch_cluster_t<__nv_bfloat16, 64>(p, U, smem, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 128) err = launch_cluster_t<float, 128>(p, U, smem, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 64) err = launch_cluster_t<float, 64>(p, U, smem, stream);
  else return ROCO_ERR_UNSUPPORTED;
  return err == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
