// One decode step of KV-constrained inference with RoCo eviction (Sec. 3, Sec. 4.3, Fig. 1), one CTA per
// unit.  The step is bound by HBM traffic, so the kernel is organised around keeping each SM's share of the
// memory system busy:
//   - a producer warp streams the unit's K block, then its V block, exactly once, through a shared-memory
//     ring filled by bulk asynchronous copies (TMA, non-multicast);
//   - eight consumer warps turn K tiles into scores (kept in shared memory: B floats, no online softmax),
//     normalise, then turn V tiles into the output;
//   - four policy warps build the eviction scope and pick the victim (Sec. 4.3) and update Acc / Acc^square /
//     Count in global memory (read once, written once) *while* the consumers stream: under EVICT_FIRST the
//     selection runs during the K pass (the new token's score and value are patched in afterwards, so the
//     stream never waits for the decision) and the statistics update during the V pass; under ATTEND_FIRST
//     both run during the V pass.
// The freed slot is overwritten in place; the cache is never compacted.
#include "common.cuh"
#include "launch.h"
#include "select.cuh"

namespace roco {

constexpr int kConsumerWarps = 8;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kProducerWarp = kConsumerWarps;
constexpr int kPolicyWarp0 = kConsumerWarps + 1;
constexpr int kPolicyWarps = 4;
constexpr int kPolicyThreads = kPolicyWarps * 32;
constexpr int kDecodeThreads = kConsumers + 32 + kPolicyThreads;
constexpr int kBarConsumers = 1;  // named barrier ids
constexpr int kBarPolicy = 2;

struct DecodeParams {
  const char *K, *V;
  float *s, *q;
  int *n, *pos, *live, *t_next, *status;
  const char *qv, *k_new, *v_new;
  char *out;
  float *lse;
  int *ev_slot, *ev_pos;
  int B, r, scope_mode, order, stages;
  int stage_stats;      // shared memory has room for a copy of the Count array (see stats_staged in the kernel)
  int policy;           // roco_policy
  const unsigned *rnd;  // [U] random draws (ROCO_POLICY_RANDOM)
  float scale;
};

struct DecodeSmem {
  char *ring;          // `stages` tiles, 128-byte aligned
  float *z;            // scores, then probabilities
  uint32_t *vkey;      // policy warps: variance keys
  float *mkey;         // policy warps: mean keys
  SelectScratch *sel;  // policy warps: histogram and reduction scratch
  float *qf, *vnew, *knew, *outred, *red;
  uint64_t *full, *empty;  // ring barriers
  uint64_t *p_ready;       // consumers have left the probabilities in shared memory
  uint64_t *policy_done;   // victim chosen, new K/V written
  uint64_t *stats_full;    // the unit's s, q, n have landed in vkey, mkey, nbuf (bulk copies ahead of the K tiles)
  uint64_t *v_done;        // consumers have read their last V tile (ATTEND_FIRST: the freed V row may be overwritten)
  int *nbuf;               // staged Count array
  int *posb;               // staged positions
  int *ctl;                // [0] abort flag, [1] slot of the new token
};

template <int TILE>
__host__ __device__ inline size_t decode_smem_bytes(int B, int d, int stages, int stage_stats) {
  const size_t Bp = align_up((size_t)B, 4);
  size_t b = (size_t)stages * TILE;
  b += (stage_stats ? 5 : 3) * Bp * 4;  // z, vkey, mkey (, nbuf, posb)
  b += sizeof(SelectScratch);
  b += (size_t)3 * d * 4;  // qf, vnew, knew (outred reuses the ring once the V pass is over)
  b += 64 * 4;                                // red
  b += (2 * (size_t)stages + 4) * sizeof(uint64_t);
  b += 8 * 4;
  return b + 128;  // slack for aligning the base
}

template <int TILE>
__device__ inline DecodeSmem carve(char *raw, int B, int d, int stages, int stage_stats) {
  DecodeSmem m;
  char *p = smem_align(raw, 128);
  const size_t Bp = align_up((size_t)B, 4);
  m.ring = p; p += (size_t)stages * TILE;
  m.z = (float *)p; p += Bp * 4;
  m.vkey = (uint32_t *)p; p += Bp * 4;
  m.mkey = (float *)p; p += Bp * 4;
  m.nbuf = (int *)p; p += stage_stats ? Bp * 4 : 0;
  m.posb = (int *)p; p += stage_stats ? Bp * 4 : 0;
  m.sel = (SelectScratch *)p; p += sizeof(SelectScratch);
  m.qf = (float *)p; p += d * 4;
  m.vnew = (float *)p; p += d * 4;
  m.knew = (float *)p; p += d * 4;
  m.outred = (float *)m.ring;  // kConsumerWarps * d floats, written after every warp's last V tile
  m.red = (float *)p; p += 64 * 4;
  m.full = (uint64_t *)p; p += stages * sizeof(uint64_t);
  m.empty = (uint64_t *)p; p += stages * sizeof(uint64_t);
  m.p_ready = (uint64_t *)p; p += sizeof(uint64_t);
  m.policy_done = (uint64_t *)p; p += sizeof(uint64_t);
  m.stats_full = (uint64_t *)p; p += sizeof(uint64_t);
  m.v_done = (uint64_t *)p; p += sizeof(uint64_t);
  m.ctl = (int *)p;
  return m;
}

__device__ __forceinline__ float consumers_max(float v, float *red, int tid) {
  v = warp_max(v);
  if ((tid & 31) == 0) red[tid >> 5] = v;
  named_bar_sync(kBarConsumers, kConsumers);
  float r = red[0];
#pragma unroll
  for (int w = 1; w < kConsumerWarps; ++w) r = fmaxf(r, red[w]);
  return r;
}

__device__ __forceinline__ float consumers_sum(float v, float *red, int tid) {
  v = warp_sum(v);
  if ((tid & 31) == 0) red[16 + (tid >> 5)] = v;
  named_bar_sync(kBarConsumers, kConsumers);
  float r = red[16];
#pragma unroll
  for (int w = 1; w < kConsumerWarps; ++w) r += red[16 + w];
  return r;
}

// kEvictFirst: the order of the step (Fig. 1: evict, insert, attend; or attend, update, then evict and insert) is a
// compile-time choice, so that neither order carries the other's registers.
template <typename T, int D, int TILE, bool kEvictFirst>
__global__ void __launch_bounds__(kDecodeThreads) decode_step_kernel(const DecodeParams p) {
  constexpr int kRowBytes = D * (int)sizeof(T);
  constexpr int kLanesPerRow = kRowBytes / 16;
  constexpr int kRowsPerLoad = 32 / kLanesPerRow;
  constexpr int kTileRows = TILE / kRowBytes;
  constexpr int kRowsPerWarp = kTileRows / kConsumerWarps;
  constexpr int kLoads = kRowsPerWarp / kRowsPerLoad;
  constexpr int kEPC = Elem<T>::kPerChunk;
  static_assert(kLanesPerRow <= 32 && kLoads >= 1, "tile shape");

  extern __shared__ char smem_raw[];
  const DecodeSmem sm = carve<TILE>(smem_raw, p.B, D, p.stages, p.stage_stats);
  volatile int *abort_flag = sm.ctl;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int u = blockIdx.x;
  const int B = p.B;
  const size_t unit_kv = (size_t)u * B * kRowBytes;
  const size_t unit_st = (size_t)u * B;
  const int stages = p.stages;

  if (tid == 0) {
    for (int i = 0; i < stages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], kConsumerWarps); }
    mbar_init(sm.p_ready, kConsumerWarps);
    mbar_init(sm.policy_done, 1);
    mbar_init(sm.stats_full, 1);
    mbar_init(sm.v_done, kConsumerWarps);
    sm.ctl[0] = 0;
    mbar_init_fence();
  }
  int live0 = p.live[u];
  if (live0 < 0 || live0 > B) {
    if (tid == 0) atomicOr(p.status, ROCO_DEV_BAD_LIVE);
    live0 = live0 < 0 ? 0 : B;
  }
  const bool full = (live0 == B);
  constexpr bool evict_first = kEvictFirst;
  const int live_att = evict_first ? (full ? B : live0 + 1) : live0;  // slots the query attends over
  const int live_new = full ? B : live0 + 1;
  const int n_tiles = (live_att + kTileRows - 1) / kTileRows;
  // The statistics the selection reads are fetched by bulk copies issued ahead of the K tiles (plain loads would
  // queue behind the tile stream for microseconds).  Under ATTEND_FIRST the copies are brought up to date in shared
  // memory once the probabilities are there.  Only where the unit's arrays start on 16-byte boundaries.
  const bool stats_staged =
      p.stage_stats && full && p.policy != ROCO_POLICY_RANDOM && (B & 3) == 0 &&
      ((reinterpret_cast<uintptr_t>(p.s) | reinterpret_cast<uintptr_t>(p.q) | reinterpret_cast<uintptr_t>(p.n) |
        reinterpret_cast<uintptr_t>(p.pos)) & 15) == 0;
  __syncthreads();

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------ producer: statistics, K tiles, then V tiles
    if (lane == 0) {
      if (stats_staged) {
        const uint32_t bytes = (uint32_t)B * 4;
        mbar_expect_tx(sm.stats_full, 4 * bytes);
        bulk_g2s(sm.vkey, p.s + unit_st, bytes, sm.stats_full);
        bulk_g2s(sm.mkey, p.q + unit_st, bytes, sm.stats_full);
        bulk_g2s(sm.nbuf, p.n + unit_st, bytes, sm.stats_full);
        bulk_g2s(sm.posb, p.pos + unit_st, bytes, sm.stats_full);
      }
      for (int g = 0; g < 2 * n_tiles; ++g) {
        const int st = g % stages;
        if (g >= stages) mbar_wait(&sm.empty[st], ((g / stages) - 1) & 1, abort_flag, p.status);
        const int it = (g < n_tiles) ? g : g - n_tiles;
        const char *src = ((g < n_tiles) ? p.K : p.V) + unit_kv + (size_t)it * TILE;
        int rows = live_att - it * kTileRows;
        if (rows > kTileRows) rows = kTileRows;
        const uint32_t bytes = (uint32_t)rows * kRowBytes;
        mbar_expect_tx(&sm.full[st], bytes);
        bulk_g2s(sm.ring + (size_t)st * TILE, src, bytes, &sm.full[st]);
      }
    }
    return;
  }

  if (warp >= kPolicyWarp0) {
    // ------------------------------------------------------------ policy: scope, victim, in-place overwrite
    const int ptid = tid - kPolicyWarp0 * 32;
    const int t_new = p.t_next[u];  // read by these warps only: they also write the incremented value
    // What the tail of this branch needs from global memory and does not depend on the victim is requested now,
    // so that its latency passes during the selection: the 16 bytes of k_new / v_new this thread will write into
    // the freed slot (raw bytes: nothing waits for them before the store; a load whose value is converted at once
    // would hold its warp, and with it the group's next barrier, until the reply has made its way through the
    // queue of streamed tiles).
    const bool writes_row = ptid >= 32 && ptid < 32 + 2 * kLanesPerRow;
    uint4 row_val = make_uint4(0u, 0u, 0u, 0u);
    if (writes_row) {
      const int c = ptid - 32;
      const bool isv = c >= kLanesPerRow;
      row_val = *((const uint4 *)((isv ? p.v_new : p.k_new) + (size_t)u * kRowBytes) + (isv ? c - kLanesPerRow : c));
    }
    named_bar_sync(kBarPolicy, kPolicyThreads);
    uint32_t k_and = 0xffffffffu, k_or = 0u;
    // statistics of Sec. 4.3 for the slots the query attended over: Acc += p, Acc^square += p^2, Count += 1
    // (a slot that has just received the new token starts from zero).  form_keys: the selection follows on the
    // new values, so its keys are formed here instead of from a second round of loads.
    auto update_statistics = [&](int fresh_slot, bool form_keys) {
      mbar_wait(sm.p_ready, 0, abort_flag, p.status);
      // four slots per turn: all loads are issued before the first store (the compiler cannot move a load of
      // one array above a store to another, and the arrays are read-modify-written in place)
      constexpr int kBatch = 4;
      for (int j0 = ptid; j0 < live_att; j0 += kBatch * kPolicyThreads) {
        float s0[kBatch], q0[kBatch];
        int n0[kBatch];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          const int j = j0 + k * kPolicyThreads;
          const bool old = j < live_att && j != fresh_slot && j < live0;
          s0[k] = old ? p.s[unit_st + j] : 0.f;
          q0[k] = old ? p.q[unit_st + j] : 0.f;
          n0[k] = old ? p.n[unit_st + j] : 0;
        }
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          const int j = j0 + k * kPolicyThreads;
          if (j >= live_att) break;
          const float pj = sm.z[j];
          p.s[unit_st + j] = s0[k] + pj;
          // Acc^square, except for the two policies of Table 1 that keep something else in this array
          float q1 = fmaf(pj, pj, q0[k]);
          if (p.policy == ROCO_POLICY_SCISSORHANDS) q1 = q0[k] + (pj * (float)live_att > 1.f ? 1.f : 0.f);  // AQAS
          if (p.policy == ROCO_POLICY_TOVA) q1 = pj;                                                       // LTAS
          p.q[unit_st + j] = q1;
          p.n[unit_st + j] = n0[k] + 1;
          if (form_keys) {
            const uint32_t vk = variance_key_fast(s0[k] + pj, q1, n0[k] + 1);
            sm.mkey[j] = mean_fast(s0[k] + pj, n0[k] + 1);
            sm.vkey[j] = vk;
            k_and &= vk;
            k_or |= vk;
          }
        }
      }
    };
    const bool keys_with_update = !evict_first && full && p.policy == ROCO_POLICY_ROCO;
    if (!evict_first) {  // select on the updated statistics
      if (stats_staged) {
        // the staged copies plus this step's probabilities: the new values go to global memory (stores only) and
        // the selection's keys are formed from them in place, so nothing here waits for a reply from global memory
        mbar_wait(sm.p_ready, 0, abort_flag, p.status);
        mbar_wait(sm.stats_full, 0, abort_flag, p.status);
#pragma unroll 4
        for (int j = ptid; j < B; j += kPolicyThreads) {
          const float pj = sm.z[j], q0 = sm.mkey[j];
          const float s1 = __uint_as_float(sm.vkey[j]) + pj;
          float q1 = fmaf(pj, pj, q0);
          if (p.policy == ROCO_POLICY_SCISSORHANDS) q1 = q0 + (pj * (float)live_att > 1.f ? 1.f : 0.f);  // AQAS
          if (p.policy == ROCO_POLICY_TOVA) q1 = pj;                                                    // LTAS
          const int n1 = sm.nbuf[j] + 1;
          p.s[unit_st + j] = s1;
          p.q[unit_st + j] = q1;
          p.n[unit_st + j] = n1;
          if (p.policy == ROCO_POLICY_ROCO) {
            const uint32_t vk = variance_key_fast(s1, q1, n1);
            sm.mkey[j] = mean_fast(s1, n1);
            sm.vkey[j] = vk;
            k_and &= vk;
            k_or |= vk;
          } else {  // the other policies of Table 1 read the new values themselves
            sm.vkey[j] = __float_as_uint(s1);
            sm.mkey[j] = q1;
            sm.nbuf[j] = n1;
          }
        }
      } else {
        update_statistics(-1, keys_with_update);
        named_bar_sync(kBarPolicy, kPolicyThreads);
      }
    }
    int e = live0, ev_slot = -1, ev_pos = -1;
    if (full) {
      // Sec. 4, fixed-budget buffer: eviction runs only once the buffer is full
      const float *gs = p.s + unit_st, *gq = p.q + unit_st;
      const int *gn = p.n + unit_st, *gpos = p.pos + unit_st;
      if (p.policy == ROCO_POLICY_ROCO) {
        const int m = scope_size(B, p.r, p.scope_mode);
        if (stats_staged) {  // s, q, n sit in vkey, mkey, nbuf: form the keys in place
          if (evict_first) {
            mbar_wait(sm.stats_full, 0, abort_flag, p.status);
#pragma unroll 4
            for (int j = ptid; j < B; j += kPolicyThreads) {
              const float sj = __uint_as_float(sm.vkey[j]);
              const uint32_t vk = variance_key_fast(sj, sm.mkey[j], sm.nbuf[j]);
              sm.mkey[j] = mean_fast(sj, sm.nbuf[j]);
              sm.vkey[j] = vk;
              k_and &= vk;
              k_or |= vk;
            }
          }
          e = group_select_from_keys(sm.posb, B, m, sm.vkey, sm.mkey, k_and, k_or, *sm.sel, ptid, kPolicyThreads,
                                     kBarPolicy);
        } else if (keys_with_update) {
          e = group_select_from_keys(gpos, B, m, sm.vkey, sm.mkey, k_and, k_or, *sm.sel, ptid, kPolicyThreads,
                                     kBarPolicy);
        } else {
          e = group_select_victim(gs, gq, gn, gpos, B, m, sm.vkey, sm.mkey, *sm.sel, ptid, kPolicyThreads,
                                  kBarPolicy);
        }
      } else if (p.policy == ROCO_POLICY_RANDOM) {
        e = (int)(p.rnd[u] % (unsigned)B);
      } else {
        // Table 1: importance score (Sec. 4.1) and local window of the r most recent positions (Sec. 4.2)
        const int pol = p.policy, horizon = t_new - p.r;
        const bool windowed = pol == ROCO_POLICY_SCISSORHANDS || pol == ROCO_POLICY_H2O || pol == ROCO_POLICY_MAS_WINDOW;
        // the statistics as the selection has to see them: the staged copies (brought up to date above under
        // ATTEND_FIRST) where there are any, else global memory
        if (stats_staged) {
          if (evict_first) mbar_wait(sm.stats_full, 0, abort_flag, p.status);
          else named_bar_sync(kBarPolicy, kPolicyThreads);
        }
        const float *ss = stats_staged ? reinterpret_cast<const float *>(sm.vkey) : gs;
        const float *qq = stats_staged ? sm.mkey : gq;
        const int *nn = stats_staged ? sm.nbuf : gn, *pp = stats_staged ? sm.posb : gpos;
        e = group_argmin(
            [&](int j) {
              if (pol == ROCO_POLICY_H2O) return ss[j];
              if (pol == ROCO_POLICY_SCISSORHANDS || pol == ROCO_POLICY_TOVA) return qq[j];
              if (pol == ROCO_POLICY_MAS_WINDOW) return mean_fast(ss[j], nn[j]);
              return 0.f;  // recency, StreamLLM: the position alone decides
            },
            [&](int j) {
              if (windowed) return pp[j] < horizon;
              if (pol == ROCO_POLICY_STREAMLLM) return pp[j] >= 4;
              return true;
            },
            pp, B, *sm.sel, ptid, kPolicyThreads, kBarPolicy);
      }
      if (e < 0) {
        if (ptid == 0) atomicOr(p.status, ROCO_DEV_BAD_VICTIM);
        e = 0;
      }
      ev_slot = e;
      if (ptid == 0) ev_pos = stats_staged ? sm.posb[e] : p.pos[unit_st + e];
    }
    // the new token takes the slot with empty statistics
    if (ptid == 0) {
      sm.ctl[1] = e;
      p.pos[unit_st + e] = t_new;
      p.ev_slot[u] = ev_slot;
      p.live[u] = live_new;
      p.t_next[u] = t_new + 1;
      if (!evict_first) { p.s[unit_st + e] = 0.f; p.q[unit_st + e] = 0.f; p.n[unit_st + e] = 0; }
    }
    if (writes_row) {  // in-place overwrite, 16 bytes per thread
      const int c = ptid - 32;
      const bool isv = c >= kLanesPerRow;
      // ATTEND_FIRST attends over the cache as it stood before the step (Fig. 1, other order), and the victim's
      // value row is part of what the producer is still streaming: the row is replaced only once every consumer
      // warp has its last V tile behind it.  (The K pass has ended by p_ready, so the key row can go at once;
      // under EVICT_FIRST the consumers take the freed slot's score and value from k_new / v_new instead.)
      if (isv && !evict_first && full) mbar_wait(sm.v_done, 0, abort_flag, p.status);
      char *dst = const_cast<char *>(isv ? p.V : p.K) + unit_kv + (size_t)e * kRowBytes;
      *((uint4 *)dst + (isv ? c - kLanesPerRow : c)) = row_val;
    }
    named_bar_sync(kBarPolicy, kPolicyThreads);
    if (ptid == 0) {
      mbar_arrive(sm.policy_done);
      if (p.ev_pos) p.ev_pos[u] = ev_pos;  // waits for the load of the old position: after the signal
    }
    if (evict_first) update_statistics(e, false);
    return;
  }

  // -------------------------------------------------------------- consumers
  if (tid < D) {
    const size_t o = (size_t)u * D + tid;
    sm.qf[tid] = Elem<T>::load((const T *)p.qv + o);
    if (evict_first) {
      sm.vnew[tid] = Elem<T>::load((const T *)p.v_new + o);
      sm.knew[tid] = Elem<T>::load((const T *)p.k_new + o);
    }
  }
  named_bar_sync(kBarConsumers, kConsumers);

  // ---- scores: z_j = scale * q.K[j]  (Eq. 1), kept in base 2
  const float zscale = p.scale * kLog2e;
  const int lane_chunk = lane % kLanesPerRow, lane_row = lane / kLanesPerRow;
  float qreg[kEPC];
#pragma unroll
  for (int i = 0; i < kEPC; ++i) qreg[i] = sm.qf[lane_chunk * kEPC + i];

  for (int it = 0; it < n_tiles; ++it) {
    const int st = it % stages;
    mbar_wait(&sm.full[st], (it / stages) & 1, abort_flag, p.status);
    const char *tile = sm.ring + (size_t)st * TILE;
    // the partial dot products of all the rows this lane touches first, then one butterfly over the lanes of a
    // row for all of them together (independent shuffles back to back instead of kLoads dependent chains)
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
      const int j = it * kTileRows + warp * kRowsPerWarp + l * kRowsPerLoad + lane_row;
      if (lane_chunk == 0 && j < live_att) sm.z[j] = acc[l] * zscale;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[st]);
  }

  // EVICT_FIRST: the slot the policy warp has freed holds the new token; its score and value come from
  // k_new / v_new, not from the stream (which may have read the slot before or after the overwrite).
  int e_sub = -1;
  if (evict_first) {
    mbar_wait(sm.policy_done, 0, abort_flag, p.status);
    e_sub = sm.ctl[1];
    if (e_sub < 0 || e_sub >= B) e_sub = 0;  // only after an aborted wait
  }
  named_bar_sync(kBarConsumers, kConsumers);  // all scores are in shared memory
  if (warp == 0 && e_sub >= 0) {  // the new token's own score, from k_new directly
    float a = 0.f;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) a = fmaf(sm.qf[lane + 32 * i], sm.knew[lane + 32 * i], a);
    a = warp_sum(a);
    if (lane == 0) sm.z[e_sub] = a * zscale;
  }
  named_bar_sync(kBarConsumers, kConsumers);

  // ---- softmax over the occupied slots
  float zmax = -INFINITY;
  for (int j = tid; j < live_att; j += kConsumers) zmax = fmaxf(zmax, sm.z[j]);
  zmax = consumers_max(zmax, sm.red, tid);
  float zsum = 0.f;
  for (int j = tid; j < live_att; j += kConsumers) {
    const float ex = exp2f(sm.z[j] - zmax);
    sm.z[j] = ex;
    zsum += ex;
  }
  zsum = consumers_sum(zsum, sm.red, tid);
  const float inv = (live_att > 0) ? 1.f / zsum : 0.f;
  for (int j = tid; j < live_att; j += kConsumers) {
    const float pj = sm.z[j] * inv;
    sm.z[j] = pj;
  }
  // hand the probabilities to the policy warps (statistics update) before streaming V
  __syncwarp();
  if (lane == 0) mbar_arrive(sm.p_ready);
  if (tid == 0 && p.lse) p.lse[u] = (live_att > 0) ? (zmax + log2f(zsum)) * kLn2 : -INFINITY;
  named_bar_sync(kBarConsumers, kConsumers);  // all probabilities are in shared memory

  // ---- out = sum_j p_j V[j]
  float acc[kEPC];
#pragma unroll
  for (int i = 0; i < kEPC; ++i) acc[i] = 0.f;
  for (int it = 0; it < n_tiles; ++it) {
    const int g = n_tiles + it;
    const int st = g % stages;
    mbar_wait(&sm.full[st], (g / stages) & 1, abort_flag, p.status);
    const char *tile = sm.ring + (size_t)st * TILE;
#pragma unroll
    for (int l = 0; l < kLoads; ++l) {
      const int row = warp * kRowsPerWarp + l * kRowsPerLoad + lane_row;
      const int j = it * kTileRows + row;
      if (j < live_att && j != e_sub) {
        const uint4 c = *(const uint4 *)(tile + (size_t)row * kRowBytes + lane_chunk * 16);
        float f[kEPC];
        Elem<T>::unpack(c, f);
        const float pj = sm.z[j];
#pragma unroll
        for (int i = 0; i < kEPC; ++i) acc[i] = fmaf(pj, f[i], acc[i]);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[st]);
  }
  if (lane == 0) mbar_arrive(sm.v_done);  // this warp has read its share of every V tile
  named_bar_sync(kBarConsumers, kConsumers);  // ... and so have the others: the ring is free for the partial sums
#pragma unroll
  for (int i = 0; i < kEPC; ++i) {
#pragma unroll
    for (int o = kLanesPerRow; o < 32; o <<= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
  }
  if (lane_row == 0) {
#pragma unroll
    for (int i = 0; i < kEPC; ++i) sm.outred[warp * D + lane_chunk * kEPC + i] = acc[i];
  }
  named_bar_sync(kBarConsumers, kConsumers);
  if (tid < D) {
    float o = 0.f;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) o += sm.outred[w * D + tid];
    if (e_sub >= 0) o = fmaf(sm.z[e_sub], sm.vnew[tid], o);
    Elem<T>::store((T *)p.out + (size_t)u * D + tid, o);
  }
}

template <typename T, int D, int TILE>
static cudaError_t launch_decode_t(const DecodeParams &p, int U, cudaStream_t stream) {
  const size_t smem = decode_smem_bytes<TILE>(p.B, D, p.stages, p.stage_stats);
  auto kernel = p.order == ROCO_EVICT_FIRST ? decode_step_kernel<T, D, TILE, true> : decode_step_kernel<T, D, TILE, false>;
  cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  kernel<<<U, kDecodeThreads, smem, stream>>>(p);
  return cudaGetLastError();
}

// Tile size and ring depth: 16 KiB tiles and the deepest ring (3..6 stages) that still lets the most CTAs
// share an SM; budgets too large for that fall back to 8 KiB tiles.
constexpr int kMaxCtasPerSm = 3;

// Stages of the tile ring (3..6, 0 = does not fit) for the largest number of CTAs per SM that fits; *ctas_out
// gets that number.
template <int TILE>
static int pick_stages(int B, int d, int stage_stats, int *ctas_out) {
  const size_t per_sm = 227 * 1024;
  for (int ctas = kMaxCtasPerSm; ctas >= 1; --ctas) {
    for (int st = 6; st >= 3; --st)
      if ((decode_smem_bytes<TILE>(B, d, st, stage_stats) + 1024) * ctas <= per_sm) {
        *ctas_out = ctas;
        return st;
      }
  }
  *ctas_out = 0;
  return 0;
}

template <typename T, int D, int TILE>
static bool try_launch(DecodeParams &p, int U, cudaStream_t stream, cudaError_t *err) {
  // the copy of the Count array is kept only if it costs no CTA per SM
  int ctas0, ctas1;
  const int st0 = pick_stages<TILE>(p.B, D, 0, &ctas0), st1 = pick_stages<TILE>(p.B, D, 1, &ctas1);
  if (st0 == 0) return false;
  p.stage_stats = (st1 > 0 && ctas1 == ctas0) ? 1 : 0;
  p.stages = p.stage_stats ? st1 : st0;
  *err = launch_decode_t<T, D, TILE>(p, U, stream);
  return true;
}

template <typename T, int D>
static cudaError_t launch_decode_td(DecodeParams &p, int U, cudaStream_t stream) {
  cudaError_t err;
  if (try_launch<T, D, 16384>(p, U, stream, &err)) return err;
  if (try_launch<T, D, 8192>(p, U, stream, &err)) return err;
  return cudaErrorInvalidConfiguration;
}

roco_status launch_decode_step(const roco_cache &c, const void *q, const void *k_new, const void *v_new, int r,
                               int scope_mode, int step_order, int policy, const unsigned *rnd, float scale, void *out,
                               float *lse, int32_t *ev_slot, int32_t *ev_pos, cudaStream_t stream) {
  DecodeParams p;
  p.K = (const char *)c.K; p.V = (const char *)c.V;
  p.s = c.s; p.q = c.q; p.n = c.n; p.pos = c.pos; p.live = c.live; p.t_next = c.t_next; p.status = c.status;
  p.qv = (const char *)q; p.k_new = (const char *)k_new; p.v_new = (const char *)v_new;
  p.out = (char *)out; p.lse = lse; p.ev_slot = ev_slot; p.ev_pos = ev_pos;
  p.B = c.B; p.r = r; p.scope_mode = scope_mode; p.order = step_order; p.scale = scale;
  p.policy = policy; p.rnd = rnd;
  const int U = c.S * c.G;
  cudaError_t err;
  if (c.kv_dtype == ROCO_BF16 && c.d == 128) err = launch_decode_td<__nv_bfloat16, 128>(p, U, stream);
  else if (c.kv_dtype == ROCO_BF16 && c.d == 64) err = launch_decode_td<__nv_bfloat16, 64>(p, U, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 128) err = launch_decode_td<float, 128>(p, U, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 64) err = launch_decode_td<float, 64>(p, U, stream);
  else return ROCO_ERR_UNSUPPORTED;
  return err == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
