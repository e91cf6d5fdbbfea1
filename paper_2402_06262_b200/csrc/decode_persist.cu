// One decode step of KV-constrained inference with RoCo eviction (Sec. 3, Sec. 4.3, Fig. 1) for calls with few
// units -- one layer of a small batch -- in ONE launch of persistent CTAs.  With one CTA per unit such a call
// leaves most of the GPU idle, so here the work is cut by cache rows, not by units: the 16 KiB tiles of all units
// form one sequence that is divided evenly among the CTAs (one or two per SM), and a CTA's share is a few
// *pieces* (unit, tile range).  No CTA ever waits for another one:
//   - a producer warp streams the K tiles, then the V tiles, of piece after piece through one shared-memory ring
//     (bulk asynchronous copies, non-multicast), so the ring stays full across piece boundaries;
//   - each of the eight consumer warps keeps its own rows of a piece to itself: scores (saved to the workspace
//     for the statistics pass), its own maximum, then exp2(z - maximum) times its V rows; the eight
//     (max, sum, sum of p*V) triples are combined once per piece and the piece's triple goes to the workspace;
//   - under EVICT_FIRST the policy warps of the CTA that holds a unit's first tile build the eviction scope and
//     pick the victim (Sec. 4.3) while the tiles stream, and leave the slot in the workspace;
//   - once a CTA has streamed its share, its consumer and policy warps together draw one ticket (atomic counter)
//     per contribution to a unit -- a piece, the selection -- all in one go, one lane each; the CTA that draws a
//     unit's last ticket merges: Eq. 1 from the piece triples (log-sum-exp merge), the new token's own score and
//     value from k_new / v_new, the victim's stale row taken out again, the in-place overwrite of the freed
//     slot, and -- the cheap second pass -- Acc += p, Acc^square += p^2, Count += 1 from the saved scores and
//     the merged log-sum-exp.  Under ATTEND_FIRST the merger also runs the selection, on the updated statistics.
//     (While tiles stream, any other access to global memory queues behind them for microseconds, so nothing on
//     this path is attempted before the CTA's own stream has ended, and what a merge needs is requested at once.)
// K and V are read from HBM exactly once; the extra traffic is 8 bytes per slot of saved scores (written, read).
#include "common.cuh"
#include "launch.h"
#include "select.cuh"

namespace roco {

constexpr int kPsConsumerWarps = 8;
constexpr int kPsConsumers = kPsConsumerWarps * 32;
constexpr int kPsProducerWarp = kPsConsumerWarps;
constexpr int kPsPolicyWarp0 = kPsConsumerWarps + 1;
constexpr int kPsPolicyWarps = 4;
constexpr int kPsPolicyThreads = kPsPolicyWarps * 32;
constexpr int kPsThreads = kPsConsumers + 32 + kPsPolicyThreads;
constexpr int kPsTile = 16384;
constexpr int kPsBarConsumers = 1;  // named barrier ids
constexpr int kPsBarPolicy = 2;
constexpr int kPsBarFinal = 3;
constexpr int kPsFinalThreads = kPsConsumers + kPsPolicyThreads;  // everyone but the producer warp
constexpr int kPsMaxPieces = 32;    // pieces one unit may be cut into (one lane each in the merge)
constexpr int kPsMaxStages = 8;

struct PersistParams {
  const char *K, *V;
  float *s, *q;
  int *n, *pos, *live, *t_next, *status;
  const char *qv, *k_new, *v_new;
  char *out;
  float *lse;
  int *ev_slot, *ev_pos;
  int U, B, r, scope_mode, order, stages, stage_stats;
  float scale;
  int tpu;    // tiles per unit
  int tq;     // tiles per CTA
  int pmax;   // pieces per unit, at most
  int zlen;   // tiles of the longest piece
  int qcap;   // pieces one CTA can have, at most
  // workspace
  float *zbuf;  // [U][B]             log2-domain scores
  float *part;  // [U][pmax][2 + d]   per piece: max, sum, sum of p*V (reference = that max)
  int *ticket;  // [U]                zero between calls.  Bits 0..7: contributions that have arrived; bits 8..31:
                //                    victim slot + 1, added by the contribution that is the selection
};

constexpr int kPsBatch = 32;  // tickets drawn together, one lane each

// What the policy warps need while they draw tickets and merge.
struct alignas(16) MergeScratch {
  float w[kPsMaxPieces];
  float red[16];
  int ml_u[kPsBatch], ml_e[kPsBatch], ml_l[kPsBatch];  // units to merge: unit, victim slot (or -1), occupied slots
  float M, L, w_e, w_new, z_new;
  int slow, e, n_merge, pad0, pad1, pad2, pad3;
};

// the shared-memory regions carved after these two must stay 16-byte (barriers: 8-byte) aligned
static_assert(sizeof(MergeScratch) % 16 == 0 && sizeof(SelectScratch) % 16 == 0, "shared-memory carve alignment");

struct PsSmem {
  char *ring;
  float *zs;           // [8 warps][zlen * rows per warp] scores of the piece in hand
  uint32_t *vkey;      // selection: variance keys
  float *mkey;         //            mean keys
  int *nbuf;           //            staged Count array
  SelectScratch *sel;
  float *outred;       // [8][D]
  float *mw, *lw;      // [8] per-warp maximum and sum
  MergeScratch *ms;
  int *queue_u, *queue_l;          // [qcap] pieces of this CTA, in order: unit, its occupied slots
  int *selq_u, *selq_e, *selq_l;   // [qcap] selections made here: unit, victim slot (-1: cache not full), occupied slots
  uint64_t *full, *empty, *stats_full;
  int *ctl;            // [0] abort flag
};

__host__ __device__ inline size_t persist_smem_bytes(int B, int d, int rows_per_tile, int stages, int zlen,
                                                     int stage_stats, int qcap) {
  const size_t Bp = align_up((size_t)B, 4);
  size_t b = (size_t)stages * kPsTile;
  b += align_up((size_t)zlen * rows_per_tile * 4, 16);
  b += (stage_stats ? 3 : 2) * Bp * 4;
  b += sizeof(SelectScratch);
  b += (size_t)kPsConsumerWarps * d * 4 + 2 * kPsConsumerWarps * 4;
  b += sizeof(MergeScratch) + 5 * align_up((size_t)qcap * 4, 8);
  b += (2 * (size_t)stages + 1) * sizeof(uint64_t);
  b += 16;
  return b + 128;
}

__device__ inline PsSmem persist_carve(char *raw, int B, int d, int rows_per_tile, int stages, int zlen,
                                       int stage_stats, int qcap) {
  PsSmem m;
  char *p = smem_align(raw, 128);
  const size_t Bp = align_up((size_t)B, 4);
  const size_t qb = align_up((size_t)qcap * 4, 8);
  m.ring = p; p += (size_t)stages * kPsTile;
  m.zs = (float *)p; p += align_up((size_t)zlen * rows_per_tile * 4, 16);
  m.vkey = (uint32_t *)p; p += Bp * 4;
  m.mkey = (float *)p; p += Bp * 4;
  m.nbuf = (int *)p; p += stage_stats ? Bp * 4 : 0;
  m.sel = (SelectScratch *)p; p += sizeof(SelectScratch);
  m.outred = (float *)p; p += (size_t)kPsConsumerWarps * d * 4;
  m.mw = (float *)p; p += kPsConsumerWarps * 4;
  m.lw = (float *)p; p += kPsConsumerWarps * 4;
  m.ms = (MergeScratch *)p; p += sizeof(MergeScratch);
  m.queue_u = (int *)p; p += qb;
  m.queue_l = (int *)p; p += qb;
  m.selq_u = (int *)p; p += qb;
  m.selq_e = (int *)p; p += qb;
  m.selq_l = (int *)p; p += qb;
  m.full = (uint64_t *)p; p += stages * sizeof(uint64_t);
  m.empty = (uint64_t *)p; p += stages * sizeof(uint64_t);
  m.stats_full = (uint64_t *)p; p += sizeof(uint64_t);
  m.ctl = (int *)p;
  return m;
}

__device__ __forceinline__ int clamp_live(int live, int B) { return live < 0 ? 0 : (live > B ? B : live); }

// Orders this thread's earlier shared-memory accesses before later bulk copies into the same bytes.
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// max / sum over the `gsize` threads of a group (a multiple of 32, at most 512); every thread gets the result.
__device__ __forceinline__ float group_max(float v, float *red, int gt, int gsize, int bar) {
  v = warp_max(v);
  if ((gt & 31) == 0) red[gt >> 5] = v;
  named_bar_sync(bar, gsize);
  float r = red[0];
  for (int w = 1; w < (gsize >> 5); ++w) r = fmaxf(r, red[w]);
  named_bar_sync(bar, gsize);
  return r;
}

__device__ __forceinline__ float group_sum(float v, float *red, int gt, int gsize, int bar) {
  v = warp_sum(v);
  if ((gt & 31) == 0) red[gt >> 5] = v;
  named_bar_sync(bar, gsize);
  float r = red[0];
  for (int w = 1; w < (gsize >> 5); ++w) r += red[w];
  named_bar_sync(bar, gsize);
  return r;
}

// The CTA that drew unit u's last ticket finishes the step for it.  Called by all `gsize` threads of a group
// (gsize >= 128, a multiple of 32) that synchronise on named barrier `bar`.  e_sel: the victim the selection
// left in the ticket word (EVICT_FIRST with a full cache), else -1; live0: the unit's occupied slots before the
// step.  Everything the merge needs is requested in one go at the top, and nothing there depends on another
// load; what other CTAs produced in this launch is read past the L1 cache.  kPre: vector turns of the statistics pass
// requested up front (bounded by the registers the launch shape leaves).
template <typename T, int D, int kPre>
__device__ __forceinline__ void merge_unit(const PersistParams &p, int u, int e_sel, int live0, int gt, int gsize,
                                        int bar) {
  constexpr int kRowBytes = D * (int)sizeof(T);
  constexpr int kLanesPerRow = kRowBytes / 16;
  // the carve is recomputed here: a reference to the caller's copy would put that copy, and with it every
  // shared-memory pointer of the streaming loops, into local memory
  extern __shared__ char ps_smem_raw[];
  const PsSmem sm = persist_carve(ps_smem_raw, p.B, D, kPsTile / kRowBytes, p.stages, p.zlen, p.stage_stats, p.qcap);
  MergeScratch &ms = *sm.ms;
  constexpr int kInl = 4;  // piece triples whose sums are requested up front
  const int B = p.B, lane = gt & 31;
  const size_t unit_st = (size_t)u * B, unit_kv = (size_t)u * B * kRowBytes;
  const bool evict_first = (p.order == ROCO_EVICT_FIRST);
  const bool full = (live0 == B);
  const int first_cta = (int)(((long long)u * p.tpu) / p.tq);
  const int last_cta = (int)(((long long)(u + 1) * p.tpu - 1) / p.tq);
  const int np = last_cta - first_cta + 1;
  const float *part = p.part + (size_t)u * p.pmax * (2 + D);
  const float *zb = p.zbuf + unit_st;
  float *gs = p.s + unit_st, *gq = p.q + unit_st;
  int *gn = p.n + unit_st;
  const float zscale = p.scale * kLog2e;
  int e = -1;
  if (evict_first) {
    e = full ? e_sel : live0;
    if (e < 0 || e >= B) e = 0;  // only after an aborted wait
  }

  // ---- requests.  The statistics pass reads 16 bytes per slot: a full cache whose arrays are 16-byte aligned goes
  // four slots per thread and turn.
  const bool vec = full && (B & 3) == 0 &&
                   ((reinterpret_cast<uintptr_t>(p.s) | reinterpret_cast<uintptr_t>(p.q) |
                     reinterpret_cast<uintptr_t>(p.n)) & 15) == 0;
  const int nvec = B >> 2;
  float4 z4[kPre], s4[kPre], q4[kPre];
  int4 n4[kPre];
  if (vec) {
#pragma unroll
    for (int k = 0; k < kPre; ++k) {
      const int v = gt + k * gsize;
      if (v < nvec) {
        z4[k] = __ldcg((const float4 *)zb + v);
        s4[k] = *((const float4 *)gs + v);
        q4[k] = *((const float4 *)gq + v);
        n4[k] = *((const int4 *)gn + v);
      }
    }
  }
  float pa[kInl], v_old = 0.f, v_nw = 0.f;
  if (gt < D) {
#pragma unroll
    for (int k = 0; k < kInl; ++k) pa[k] = (k < np) ? __ldcg(part + (size_t)k * (2 + D) + 2 + gt) : 0.f;
    if (evict_first) {
      if (full) v_old = Elem<T>::load((const T *)(p.V + unit_kv) + (size_t)e * D + gt);
      v_nw = Elem<T>::load((const T *)p.v_new + (size_t)u * D + gt);
    }
  }
  uint4 row_val = make_uint4(0u, 0u, 0u, 0u);
  const bool writes_row = gt >= 32 && gt < 32 + 2 * kLanesPerRow;
  if (writes_row) {
    const int c = gt - 32;
    const bool isv = c >= kLanesPerRow;
    row_val = *((const uint4 *)((isv ? p.v_new : p.k_new) + (size_t)u * kRowBytes) + (isv ? c - kLanesPerRow : c));
  }
  int t_new = 0, old_pos = -1;
  if (gt == 0) {
    t_new = p.t_next[u];
    if (evict_first && full) old_pos = p.pos[unit_st + e];
  }

  // ---- the merged maximum and denominator (Eq. 1), by the group's first warp
  if (gt < 32) {
    float zn = -INFINITY, ze = -INFINITY;
    float acc = 0.f;
    if (evict_first) {  // the new token's own score, from k_new directly
#pragma unroll
      for (int i = 0; i < D / 32; ++i)
        acc = fmaf(Elem<T>::load((const T *)p.qv + (size_t)u * D + lane + 32 * i),
                   Elem<T>::load((const T *)p.k_new + (size_t)u * D + lane + 32 * i), acc);
      if (full) ze = __ldcg(zb + e);  // the stale row's score: part of its piece's triple, taken out below
    }
    const float mk = (lane < np) ? __ldcg(part + (size_t)lane * (2 + D)) : -INFINITY;
    const float lk = (lane < np) ? __ldcg(part + (size_t)lane * (2 + D) + 1) : 0.f;
    if (evict_first) zn = warp_sum(acc) * zscale;
    const float M = warp_max(fmaxf(mk, zn));
    const float wk = (mk > -INFINITY) ? exp2f(mk - M) : 0.f;  // an empty piece has max -inf and sum 0
    const float Lall = warp_sum(wk * lk);
    if (lane < np) ms.w[lane] = wk;
    const float we = (ze > -INFINITY) ? exp2f(ze - M) : 0.f;
    const float wn = (zn > -INFINITY) ? exp2f(zn - M) : 0.f;
    if (lane == 0) {
      ms.M = M; ms.L = Lall - we + wn; ms.w_e = we; ms.w_new = wn; ms.z_new = zn;
      // Taking the stale row out by subtraction is safe while it is a modest part of the sum; a victim that
      // dominates the softmax (it has the lowest mean score of its scope, so this is rare) is handled exactly.
      ms.slow = (we > 0.25f * Lall) ? 1 : 0;
    }
  }
  named_bar_sync(bar, gsize);
  if (ms.slow) {
    // exact recomputation from the saved scores and the V rows, without the stale row
    const float zn = ms.z_new;
    float mx = zn;
    for (int j = gt; j < B; j += gsize)
      if (j != e) mx = fmaxf(mx, __ldcg(zb + j));
    mx = group_max(mx, ms.red, gt, gsize, bar);
    float sum = 0.f;
    for (int j = gt; j < B; j += gsize)
      if (j != e) sum += exp2f(__ldcg(zb + j) - mx);
    sum = group_sum(sum, ms.red, gt, gsize, bar);
    const float wn = exp2f(zn - mx);
    sum += wn;
    if (gt < D) {
      float o = 0.f;
      const T *Vu = (const T *)(p.V + unit_kv);
      for (int j = 0; j < B; ++j)
        if (j != e) o = fmaf(exp2f(__ldcg(zb + j) - mx), Elem<T>::load(Vu + (size_t)j * D + gt), o);
      o = fmaf(wn, v_nw, o);
      Elem<T>::store((T *)p.out + (size_t)u * D + gt, o / sum);
    }
    if (gt == 0) { ms.M = mx; ms.L = sum; ms.w_new = wn; }
    named_bar_sync(bar, gsize);
  } else if (gt < D) {
    float o = 0.f;
#pragma unroll
    for (int k = 0; k < kInl; ++k)
      if (k < np) o = fmaf(ms.w[k], pa[k], o);
    for (int k = kInl; k < np; ++k) o = fmaf(ms.w[k], __ldcg(part + (size_t)k * (2 + D) + 2 + gt), o);
    if (evict_first) {
      o = fmaf(-ms.w_e, v_old, o);
      o = fmaf(ms.w_new, v_nw, o);
    }
    const float L0 = ms.L;
    Elem<T>::store((T *)p.out + (size_t)u * D + gt, L0 > 0.f ? o / L0 : 0.f);
  }
  const float M = ms.M, L = ms.L;
  const float inv = L > 0.f ? 1.f / L : 0.f;
  const float w_new = ms.w_new;
  named_bar_sync(bar, gsize);  // ms.* has been read (and, in the exact pass, the victim's old value row)
  if (gt == 0 && p.lse) p.lse[u] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;

  // Statistics of Sec. 4.3 for four slots: Acc += p, Acc^square += p^2, Count += 1 with p from the saved score
  // and the merged log-sum-exp; the slot that has just received the new token (EVICT_FIRST) starts from zero.
  // ATTEND_FIRST also leaves the selection keys of the updated statistics in shared memory.
  uint32_t k_and = 0xffffffffu, k_or = 0u;
  auto apply4 = [&](int v, const float4 &zz, float4 ss, float4 qq, int4 nn) {
    float pr[4] = {exp2f(zz.x - M) * inv, exp2f(zz.y - M) * inv, exp2f(zz.z - M) * inv, exp2f(zz.w - M) * inv};
    float sa[4] = {ss.x, ss.y, ss.z, ss.w}, qa[4] = {qq.x, qq.y, qq.z, qq.w};
    int na[4] = {nn.x, nn.y, nn.z, nn.w};
    uint32_t vk[4];
    float mk[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (evict_first && 4 * v + i == e) { pr[i] = w_new * inv; sa[i] = 0.f; qa[i] = 0.f; na[i] = 0; }
      sa[i] += pr[i];
      qa[i] = fmaf(pr[i], pr[i], qa[i]);
      na[i] += 1;
      if (!evict_first) {
        vk[i] = variance_key_fast(sa[i], qa[i], na[i]);
        mk[i] = mean_fast(sa[i], na[i]);
        k_and &= vk[i];
        k_or |= vk[i];
      }
    }
    *((float4 *)gs + v) = make_float4(sa[0], sa[1], sa[2], sa[3]);
    *((float4 *)gq + v) = make_float4(qa[0], qa[1], qa[2], qa[3]);
    *((int4 *)gn + v) = make_int4(na[0], na[1], na[2], na[3]);
    if (!evict_first) {
      *((uint4 *)sm.vkey + v) = make_uint4(vk[0], vk[1], vk[2], vk[3]);
      *((float4 *)sm.mkey + v) = make_float4(mk[0], mk[1], mk[2], mk[3]);
    }
  };
  auto stats_vectorised = [&]() {
#pragma unroll
    for (int k = 0; k < kPre; ++k) {
      const int v = gt + k * gsize;
      if (v < nvec) apply4(v, z4[k], s4[k], q4[k], n4[k]);
    }
    for (int v0 = gt + kPre * gsize; v0 < nvec; v0 += kPre * gsize) {
      float4 za[kPre], sa[kPre], qa[kPre];
      int4 na[kPre];
#pragma unroll
      for (int k = 0; k < kPre; ++k) {
        const int v = v0 + k * gsize;
        if (v < nvec) {
          za[k] = __ldcg((const float4 *)zb + v);
          sa[k] = *((const float4 *)gs + v);
          qa[k] = *((const float4 *)gq + v);
          na[k] = *((const int4 *)gn + v);
        }
      }
#pragma unroll
      for (int k = 0; k < kPre; ++k) {
        const int v = v0 + k * gsize;
        if (v < nvec) apply4(v, za[k], sa[k], qa[k], na[k]);
      }
    }
  };

  constexpr int kBatch = 4;
  if (evict_first) {
    // ---- Fig. 1 order: the freed (or first free) slot takes the new token, with statistics of one observation
    if (gt == 0) {
      p.pos[unit_st + e] = t_new;
      p.ev_slot[u] = full ? e : -1;
      if (p.ev_pos) p.ev_pos[u] = old_pos;
      p.live[u] = full ? B : live0 + 1;
      p.t_next[u] = t_new + 1;
    }
    if (writes_row) {  // in-place overwrite, 16 bytes per thread (every read of the old value row is behind us)
      const int c = gt - 32;
      const bool isv = c >= kLanesPerRow;
      *((uint4 *)(const_cast<char *>(isv ? p.V : p.K) + unit_kv + (size_t)e * kRowBytes) +
        (isv ? c - kLanesPerRow : c)) = row_val;
    }
    if (vec) {
      stats_vectorised();
    } else {
      const int live_att = full ? B : live0 + 1;
      for (int j0 = gt; j0 < live_att; j0 += kBatch * gsize) {
        float s0[kBatch], q0[kBatch], pj[kBatch];
        int n0[kBatch];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          const int j = j0 + k * gsize;
          const bool old = j < live_att && j != e;
          s0[k] = old ? gs[j] : 0.f;
          q0[k] = old ? gq[j] : 0.f;
          n0[k] = old ? gn[j] : 0;
          pj[k] = old ? __ldcg(zb + j) : 0.f;
        }
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          const int j = j0 + k * gsize;
          if (j >= live_att) break;
          const float pr = (j == e) ? w_new * inv : exp2f(pj[k] - M) * inv;
          gs[j] = s0[k] + pr;
          gq[j] = fmaf(pr, pr, q0[k]);
          gn[j] = n0[k] + 1;
        }
      }
    }
  } else {
    // ---- other order: statistics of the attended slots first, then the selection on them, then the insertion
    if (vec) {
      stats_vectorised();
    } else {
      for (int j0 = gt; j0 < live0; j0 += kBatch * gsize) {
        float s0[kBatch], q0[kBatch], pj[kBatch];
        int n0[kBatch];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          const int j = j0 + k * gsize;
          const bool in = j < live0;
          s0[k] = in ? gs[j] : 0.f;
          q0[k] = in ? gq[j] : 0.f;
          n0[k] = in ? gn[j] : 0;
          pj[k] = in ? __ldcg(zb + j) : 0.f;
        }
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          const int j = j0 + k * gsize;
          if (j >= live0) break;
          const float pr = exp2f(pj[k] - M) * inv;
          const float s1 = s0[k] + pr, q1 = fmaf(pr, pr, q0[k]);
          const int n1 = n0[k] + 1;
          gs[j] = s1;
          gq[j] = q1;
          gn[j] = n1;
          if (full) {
            const uint32_t vk = variance_key_fast(s1, q1, n1);
            sm.vkey[j] = vk;
            sm.mkey[j] = mean_fast(s1, n1);
            k_and &= vk;
            k_or |= vk;
          }
        }
      }
    }
    e = live0;
    if (full) {
      const int m = scope_size(B, p.r, p.scope_mode);
      e = group_select_from_keys(p.pos + unit_st, B, m, sm.vkey, sm.mkey, k_and, k_or, *sm.sel, gt, gsize, bar);
      if (e < 0) {
        if (gt == 0) atomicOr(p.status, ROCO_DEV_BAD_VICTIM);
        e = 0;
      }
    } else {
      named_bar_sync(bar, gsize);
    }
    if (gt == 0) {
      old_pos = full ? p.pos[unit_st + e] : -1;
      p.pos[unit_st + e] = t_new;
      gs[e] = 0.f; gq[e] = 0.f; gn[e] = 0;
      p.ev_slot[u] = full ? e : -1;
      if (p.ev_pos) p.ev_pos[u] = old_pos;
      p.live[u] = full ? B : live0 + 1;
      p.t_next[u] = t_new + 1;
    }
    if (writes_row) {
      const int c = gt - 32;
      const bool isv = c >= kLanesPerRow;
      *((uint4 *)(const_cast<char *>(isv ? p.V : p.K) + unit_kv + (size_t)e * kRowBytes) +
        (isv ? c - kLanesPerRow : c)) = row_val;
    }
  }
  if (gt == 0) p.ticket[u] = 0;  // the workspace is left as it was found
  named_bar_sync(bar, gsize);    // the scratch may be reused
}

template <typename T, int D, int kCtasPerSm>
__global__ void __launch_bounds__(kPsThreads, kCtasPerSm) decode_persist_kernel(const __grid_constant__ PersistParams p) {
  constexpr int kPre = 1;
  constexpr int kRowBytes = D * (int)sizeof(T);
  constexpr int kLanesPerRow = kRowBytes / 16;
  constexpr int kRowsPerLoad = 32 / kLanesPerRow;
  constexpr int kTileRows = kPsTile / kRowBytes;
  constexpr int kRowsPerWarp = kTileRows / kPsConsumerWarps;
  constexpr int kLoads = kRowsPerWarp / kRowsPerLoad;
  constexpr int kEPC = Elem<T>::kPerChunk;
  static_assert(kLanesPerRow <= 32 && kLoads >= 1, "tile shape");

  extern __shared__ char ps_smem_raw[];
  const PsSmem sm = persist_carve(ps_smem_raw, p.B, D, kTileRows, p.stages, p.zlen, p.stage_stats, p.qcap);
  volatile int *abort_flag = sm.ctl;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int B = p.B, stages = p.stages, tpu = p.tpu;
  const long long total_tiles = (long long)p.U * tpu;
  const long long g0 = (long long)blockIdx.x * p.tq;
  const long long g1 = (g0 + p.tq < total_tiles) ? g0 + p.tq : total_tiles;
  const bool evict_first = (p.order == ROCO_EVICT_FIRST);

  if (tid == 0) {
    for (int i = 0; i < stages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], kPsConsumerWarps); }
    mbar_init(sm.stats_full, 1);
    sm.ctl[0] = 0;
    mbar_init_fence();
  }
  __syncthreads();
  if (g0 >= g1) return;

  if (warp == kPsProducerWarp) {
    // ------------------------------------------------------------ producer: K tiles then V tiles, piece by piece
    if (lane == 0) {
      int slot = 0;
      for (long long g = g0; g < g1;) {
        const int u = (int)(g / tpu), t0 = (int)(g - (long long)u * tpu);
        const int t1 = (int)((g1 - g < tpu - t0) ? t0 + (g1 - g) : tpu);
        g += t1 - t0;
        const int live0 = clamp_live(p.live[u], B);
        const int tl = (live0 + kTileRows - 1) / kTileRows;  // tiles that hold occupied rows
        const int te = t1 < tl ? t1 : tl;
        const size_t unit_kv = (size_t)u * B * kRowBytes;
        for (int pass = 0; pass < 2; ++pass) {
          for (int it = t0; it < te; ++it, ++slot) {
            const int st = slot % stages;
            if (slot >= stages) mbar_wait(&sm.empty[st], ((slot / stages) - 1) & 1, abort_flag, p.status);
            int rows = live0 - it * kTileRows;
            if (rows > kTileRows) rows = kTileRows;
            const uint32_t bytes = (uint32_t)rows * kRowBytes;
            mbar_expect_tx(&sm.full[st], bytes);
            bulk_g2s(sm.ring + (size_t)st * kPsTile, (pass ? p.V : p.K) + unit_kv + (size_t)it * kPsTile, bytes,
                     &sm.full[st]);
          }
        }
      }
    }
    return;
  }

  const int first_unit_here = (int)((g0 + tpu - 1) / tpu);  // units whose first tile belongs to this CTA start here
  if (warp >= kPsPolicyWarp0) {
    // ------------------------------------------------------------ policy warps: selections
    const int ptid = tid - kPsPolicyWarp0 * 32;
    const bool can_stage =
        p.stage_stats && (B & 3) == 0 &&
        ((reinterpret_cast<uintptr_t>(p.s) | reinterpret_cast<uintptr_t>(p.q) | reinterpret_cast<uintptr_t>(p.n)) & 15) == 0;
    // Under EVICT_FIRST the selection sees the statistics as they stand at the start of the step: the units whose
    // first tile belongs to this CTA are done first, while the tiles stream.  (The other order selects on the
    // updated statistics: the merger does it.)
    int n_sel = 0;
    for (int u = first_unit_here; evict_first && u < p.U && (long long)u * tpu < g1; ++u, ++n_sel) {
      const size_t unit_st = (size_t)u * B;
      const int live_raw = p.live[u];
      const int live0 = clamp_live(live_raw, B);
      if (ptid == 0 && live_raw != live0) atomicOr(p.status, ROCO_DEV_BAD_LIVE);
      int e = -1;
      if (live0 == B) {
        // Sec. 4, fixed-budget buffer: eviction runs only once the buffer is full
        const int m = scope_size(B, p.r, p.scope_mode);
        if (can_stage) {  // s, q, n arrive in vkey, mkey, nbuf by bulk copy; the keys are formed in place
          if (ptid == 0) {
            const uint32_t bytes = (uint32_t)B * 4;
            mbar_expect_tx(sm.stats_full, 3 * bytes);
            bulk_g2s(sm.vkey, p.s + unit_st, bytes, sm.stats_full);
            bulk_g2s(sm.mkey, p.q + unit_st, bytes, sm.stats_full);
            bulk_g2s(sm.nbuf, p.n + unit_st, bytes, sm.stats_full);
          }
          mbar_wait(sm.stats_full, n_sel & 1, abort_flag, p.status);
          uint32_t k_and = 0xffffffffu, k_or = 0u;
#pragma unroll 4
          for (int j = ptid; j < B; j += kPsPolicyThreads) {
            const float sj = __uint_as_float(sm.vkey[j]);
            const uint32_t vk = variance_key_fast(sj, sm.mkey[j], sm.nbuf[j]);
            sm.mkey[j] = mean_fast(sj, sm.nbuf[j]);
            sm.vkey[j] = vk;
            k_and &= vk;
            k_or |= vk;
          }
          e = group_select_from_keys(p.pos + unit_st, B, m, sm.vkey, sm.mkey, k_and, k_or, *sm.sel, ptid,
                                     kPsPolicyThreads, kPsBarPolicy);
          fence_proxy_async_smem();  // the keys written here come before the next unit's bulk copies into them
        } else {
          e = group_select_victim(p.s + unit_st, p.q + unit_st, p.n + unit_st, p.pos + unit_st, B, m, sm.vkey,
                                  sm.mkey, *sm.sel, ptid, kPsPolicyThreads, kPsBarPolicy);
        }
        if (e < 0) {
          if (ptid == 0) atomicOr(p.status, ROCO_DEV_BAD_VICTIM);
          e = 0;
        }
      }
      if (ptid == 0) { sm.selq_u[n_sel] = u; sm.selq_e[n_sel] = e; sm.selq_l[n_sel] = live0; }
    }
  } else {
  // -------------------------------------------------------------- consumers
  const float zscale = p.scale * kLog2e;
  const int lane_chunk = lane % kLanesPerRow, lane_row = lane / kLanesPerRow;
  float *zw = sm.zs + (size_t)warp * p.zlen * kRowsPerWarp;  // this warp's scores of the piece in hand
  auto load_q = [&](int u, float (&qr)[kEPC]) {
    const uint4 c = *((const uint4 *)(p.qv + (size_t)u * kRowBytes) + lane_chunk);
    Elem<T>::unpack(c, qr);
  };
  float qreg[kEPC];
  load_q((int)(g0 / tpu), qreg);
  int slot = 0, n_posted = 0;
  for (long long g = g0; g < g1;) {
    const int u = (int)(g / tpu), t0 = (int)(g - (long long)u * tpu);
    const int t1 = (int)((g1 - g < tpu - t0) ? t0 + (g1 - g) : tpu);
    g += t1 - t0;
    const int live0 = clamp_live(p.live[u], B);
    const int tl = (live0 + kTileRows - 1) / kTileRows;
    const int te = t1 < tl ? t1 : tl;
    float *zb = p.zbuf + (size_t)u * B;

    // ---- scores of this warp's rows: z_j = scale * q.K[j] (Eq. 1), kept in base 2
    float mloc = -INFINITY;
    for (int it = t0; it < te; ++it, ++slot) {
      const int st = slot % stages;
      mbar_wait(&sm.full[st], (slot / stages) & 1, abort_flag, p.status);
      const char *tile = sm.ring + (size_t)st * kPsTile;
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
        const int rw = l * kRowsPerLoad + lane_row;  // row within this warp's share of the tile
        const int j = it * kTileRows + warp * kRowsPerWarp + rw;
        const float z = (j < live0) ? acc[l] * zscale : -INFINITY;
        mloc = fmaxf(mloc, z);
        if (lane_chunk == 0) {
          zw[(it - t0) * kRowsPerWarp + rw] = z;
          if (j < live0) zb[j] = z;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[st]);
    }
    // the next piece's query, requested now so that it arrives during the V pass
    float qnext[kEPC];
#pragma unroll
    for (int i = 0; i < kEPC; ++i) qnext[i] = 0.f;
    if (g < g1) load_q((int)(g / tpu), qnext);
    const float m_w = warp_max(mloc);
    __syncwarp();

    // ---- this warp's sum of exp2(z - m_w) * V[j]
    float acc[kEPC];
#pragma unroll
    for (int i = 0; i < kEPC; ++i) acc[i] = 0.f;
    float lsum = 0.f;
    for (int it = t0; it < te; ++it, ++slot) {
      const int st = slot % stages;
      mbar_wait(&sm.full[st], (slot / stages) & 1, abort_flag, p.status);
      const char *tile = sm.ring + (size_t)st * kPsTile;
#pragma unroll
      for (int l = 0; l < kLoads; ++l) {
        const int rw = l * kRowsPerLoad + lane_row;
        const int row = warp * kRowsPerWarp + rw;
        const int j = it * kTileRows + row;
        if (j < live0) {
          const uint4 c = *(const uint4 *)(tile + (size_t)row * kRowBytes + lane_chunk * 16);
          float f[kEPC];
          Elem<T>::unpack(c, f);
          const float pj = exp2f(zw[(it - t0) * kRowsPerWarp + rw] - m_w);
          if (lane_chunk == 0) lsum += pj;
#pragma unroll
          for (int i = 0; i < kEPC; ++i) acc[i] = fmaf(pj, f[i], acc[i]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[st]);
    }
#pragma unroll
    for (int i = 0; i < kEPC; ++i) {
#pragma unroll
      for (int o = kLanesPerRow; o < 32; o <<= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
    }
    lsum = warp_sum(lsum);
    if (lane_row == 0) {
#pragma unroll
      for (int i = 0; i < kEPC; ++i) sm.outred[warp * D + lane_chunk * kEPC + i] = acc[i];
    }
    if (lane == 0) { sm.mw[warp] = m_w; sm.lw[warp] = lsum; }
    named_bar_sync(kPsBarConsumers, kPsConsumers);

    // ---- the piece's (max, sum, sum of p*V) triple
    const int first_cta = (int)(((long long)u * tpu) / p.tq);
    float *part = p.part + ((size_t)u * p.pmax + ((int)blockIdx.x - first_cta)) * (2 + D);
    {
      float mc = sm.mw[0];
#pragma unroll
      for (int w = 1; w < kPsConsumerWarps; ++w) mc = fmaxf(mc, sm.mw[w]);
      float o = 0.f, l = 0.f;
#pragma unroll
      for (int w = 0; w < kPsConsumerWarps; ++w) {
        const float mwv = sm.mw[w];
        const float wt = (mwv > -INFINITY) ? exp2f(mwv - mc) : 0.f;  // a warp without occupied rows has max -inf
        if (tid < D) o = fmaf(wt, sm.outred[w * D + tid], o);
        l = fmaf(wt, sm.lw[w], l);
      }
      if (tid < D) part[2 + tid] = o;
      if (tid == 0) { part[0] = mc; part[1] = l; }
    }
    named_bar_sync(kPsBarConsumers, kPsConsumers);  // outred, mw, lw may be rewritten
    if (tid == 0) { sm.queue_u[n_posted] = u; sm.queue_l[n_posted] = live0; }
    ++n_posted;
#pragma unroll
    for (int i = 0; i < kEPC; ++i) qreg[i] = qnext[i];
  }
  }

  // ---------------------------------------------------------------- tickets and merges, once the stream has ended
  // Every contribution of this CTA to a unit -- a piece it streamed, a selection it made -- draws one ticket for
  // that unit, all of them together, one lane each (the fence before the atomic covers what the whole CTA stored,
  // ordered before it by the barrier); the lanes that drew a unit's last ticket leave the unit in the merge list,
  // and the consumer and policy warps merge those units together.
  const int ft = (warp < kPsConsumerWarps) ? tid : tid - 32;  // index among the threads of this phase
  MergeScratch &ms = *sm.ms;
  int n_pieces = 0;
  for (long long g = g0; g < g1; ++n_pieces) {
    const int t0 = (int)(g % tpu);
    g += (g1 - g < tpu - t0) ? (g1 - g) : (tpu - t0);
  }
  int n_sel = 0;
  if (evict_first)
    for (int u = first_unit_here; u < p.U && (long long)u * tpu < g1; ++u) ++n_sel;
  named_bar_sync(kPsBarFinal, kPsFinalThreads);
  for (int base = 0; base < n_sel + n_pieces; base += kPsBatch) {
    if (ft < 32) {
      const int idx = base + ft;
      int u = -1, add = 0, live0 = 0;
      if (idx < n_sel) {
        u = sm.selq_u[idx];
        add = 1 + ((sm.selq_e[idx] + 1) << 8);
        live0 = sm.selq_l[idx];
      } else if (idx < n_sel + n_pieces) {
        u = sm.queue_u[idx - n_sel];
        live0 = sm.queue_l[idx - n_sel];
        add = 1;
      }
      bool last = false;
      int e_sel = -1;
      if (u >= 0) {
        const int first_cta = (int)(((long long)u * tpu) / p.tq);
        const int last_cta = (int)(((long long)(u + 1) * tpu - 1) / p.tq);
        const int needed = last_cta - first_cta + 1 + (evict_first ? 1 : 0);
        __threadfence();
        const int total = atomicAdd(p.ticket + u, add) + add;
        last = (total & 0xff) == needed;
        e_sel = (total >> 8) - 1;
        if (last) __threadfence();
      }
      const uint32_t lm = __ballot_sync(0xffffffffu, last);
      if (last) {
        const int k = __popc(lm & ((1u << ft) - 1u));
        ms.ml_u[k] = u; ms.ml_e[k] = e_sel; ms.ml_l[k] = live0;
      }
      if (ft == 0) ms.n_merge = __popc(lm);
    }
    named_bar_sync(kPsBarFinal, kPsFinalThreads);
    const int n_merge = ms.n_merge;
    for (int i = 0; i < n_merge; ++i) {
      const int u = ms.ml_u[i], e_sel = ms.ml_e[i], live0 = ms.ml_l[i];
      merge_unit<T, D, kPre>(p, u, e_sel, live0, ft, kPsFinalThreads, kPsBarFinal);
    }
    named_bar_sync(kPsBarFinal, kPsFinalThreads);  // the merge list may be rewritten
  }
}

// Shape of one launch: CTAs, tiles per CTA, ring depth.  Returns false if nothing fits.
struct PersistPlan {
  int grid, tq, pmax, zlen, qcap, stages, stage_stats, ctas;
  size_t smem;
};

static bool persist_plan(int U, int B, int d, int elem, int sms, PersistPlan *pl) {
  const int rows_per_tile = kPsTile / (d * elem);
  const int tpu = (B + rows_per_tile - 1) / rows_per_tile;
  const long long total = (long long)U * tpu;
  const size_t per_sm = 227 * 1024;
  for (int ctas = 2; ctas >= 1; --ctas) {
    long long tq = (total + (long long)sms * ctas - 1) / ((long long)sms * ctas);
    const long long tq_min = (tpu + kPsMaxPieces - 2) / (kPsMaxPieces - 1);  // at most kPsMaxPieces pieces per unit
    if (tq < tq_min) tq = tq_min;
    if (tq < 1) tq = 1;
    const int zlen = (int)(tq < tpu ? tq : tpu);
    const int qcap = (int)((tq + tpu - 1) / tpu) + 1;  // units a run of tq tiles can touch
    for (int stage_stats = 1; stage_stats >= 0; --stage_stats) {
      for (int st = kPsMaxStages; st >= 3; --st) {
        const size_t smem = persist_smem_bytes(B, d, rows_per_tile, st, zlen, stage_stats, qcap);
        if ((smem + 1024) * ctas > per_sm) continue;
        if (stage_stats && st < 4 && ctas == 2) continue;  // a deeper ring is worth more than the staged statistics
        pl->grid = (int)((total + tq - 1) / tq);
        pl->tq = (int)tq;
        pl->pmax = (int)((tpu + tq - 1) / tq) + 1;
        pl->zlen = zlen;
        pl->qcap = qcap;
        pl->ctas = ctas;
        pl->stages = st;
        pl->stage_stats = stage_stats;
        pl->smem = smem;
        return true;
      }
    }
  }
  return false;
}

static int device_sms() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
}

struct PersistWs {
  size_t zbuf_off, part_off, ticket_off, total;
};

static PersistWs persist_ws(int U, int B, int d, int pmax) {
  PersistWs w;
  w.ticket_off = 0;  // first, so that the caller can clear it with one small memset
  w.zbuf_off = align_up((size_t)U * 4, 256);
  w.part_off = w.zbuf_off + align_up((size_t)U * B * 4, 256);
  w.total = w.part_off + align_up((size_t)U * pmax * (2 + d) * 4, 256);
  return w;
}

size_t decode_persist_workspace_bytes(int U, int B, int d, int elem) {
  const int sms = device_sms();
  PersistPlan pl;
  if (sms < 1 || !persist_plan(U, B, d, elem, sms, &pl)) return 0;
  return persist_ws(U, B, d, pl.pmax).total;
}

size_t decode_persist_ticket_bytes(int U) { return align_up((size_t)U * 4, 256); }

template <typename T, int D, int kCtasPerSm>
static cudaError_t launch_persist_tc(const PersistParams &p, const PersistPlan &pl, cudaStream_t stream) {
  cudaError_t err = cudaFuncSetAttribute(decode_persist_kernel<T, D, kCtasPerSm>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
  if (err != cudaSuccess) return err;
  decode_persist_kernel<T, D, kCtasPerSm><<<pl.grid, kPsThreads, pl.smem, stream>>>(p);
  return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t launch_persist_t(const PersistParams &p, const PersistPlan &pl, cudaStream_t stream) {
  return pl.ctas == 2 ? launch_persist_tc<T, D, 2>(p, pl, stream) : launch_persist_tc<T, D, 1>(p, pl, stream);
}

roco_status launch_decode_step_persistent(const roco_cache &c, const void *q, const void *k_new, const void *v_new,
                                          int r, int scope_mode, int step_order, float scale, void *out, float *lse,
                                          int32_t *ev_slot, int32_t *ev_pos, void *workspace, cudaStream_t stream) {
  const int U = c.S * c.G;
  const int elem = c.kv_dtype == ROCO_BF16 ? 2 : 4;
  const int sms = device_sms();
  if (sms < 1) return ROCO_ERR_CUDA;
  PersistPlan pl;
  if (!persist_plan(U, c.B, c.d, elem, sms, &pl)) return ROCO_ERR_UNSUPPORTED;
  PersistParams p;
  p.K = (const char *)c.K; p.V = (const char *)c.V;
  p.s = c.s; p.q = c.q; p.n = c.n; p.pos = c.pos; p.live = c.live; p.t_next = c.t_next; p.status = c.status;
  p.qv = (const char *)q; p.k_new = (const char *)k_new; p.v_new = (const char *)v_new;
  p.out = (char *)out; p.lse = lse; p.ev_slot = ev_slot; p.ev_pos = ev_pos;
  p.U = U; p.B = c.B; p.r = r; p.scope_mode = scope_mode; p.order = step_order; p.scale = scale;
  p.stages = pl.stages; p.stage_stats = pl.stage_stats;
  const int rows_per_tile = kPsTile / (c.d * elem);
  p.tpu = (c.B + rows_per_tile - 1) / rows_per_tile;
  p.tq = pl.tq; p.pmax = pl.pmax; p.zlen = pl.zlen; p.qcap = pl.qcap;
  const PersistWs w = persist_ws(U, c.B, c.d, pl.pmax);
  char *ws = (char *)workspace;
  p.ticket = (int *)(ws + w.ticket_off);
  p.zbuf = (float *)(ws + w.zbuf_off);
  p.part = (float *)(ws + w.part_off);
  cudaError_t err;
  if (c.kv_dtype == ROCO_BF16 && c.d == 128) err = launch_persist_t<__nv_bfloat16, 128>(p, pl, stream);
  else if (c.kv_dtype == ROCO_BF16 && c.d == 64) err = launch_persist_t<__nv_bfloat16, 64>(p, pl, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 128) err = launch_persist_t<float, 128>(p, pl, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 64) err = launch_persist_t<float, 64>(p, pl, stream);
  else return ROCO_ERR_UNSUPPORTED;
  return err == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
