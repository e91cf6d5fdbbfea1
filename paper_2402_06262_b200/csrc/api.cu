// The C ABI of libroco: argument validation on the host, workspace carving, launches.
#include <nvtx3/nvToolsExt.h>

#include <cstring>
#include <mutex>

#include "common.cuh"
#include "launch.h"

using namespace roco;

namespace {

// A named range around every launching entry point, visible in the timeline of an attached profiler.
struct NvtxRange {
  explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};

constexpr int kMaxB = 8192;

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

roco_status check_cache(const roco_cache *c) {
  if (!c) return ROCO_ERR_INVALID_ARG;
  if (!c->K || !c->V || !c->s || !c->q || !c->n || !c->pos || !c->live || !c->t_next || !c->status)
    return ROCO_ERR_INVALID_ARG;
  if (c->S < 1 || c->G < 1 || c->B < 1) return ROCO_ERR_INVALID_ARG;
  if (!aligned16(c->K) || !aligned16(c->V)) return ROCO_ERR_INVALID_ARG;
  if (c->kv_dtype != ROCO_F32 && c->kv_dtype != ROCO_BF16) return ROCO_ERR_UNSUPPORTED;
  if (c->d != 64 && c->d != 128) return ROCO_ERR_UNSUPPORTED;
  if (c->B > kMaxB) return ROCO_ERR_UNSUPPORTED;
  if ((long long)c->S * c->G > 0x7fffffffLL / 64) return ROCO_ERR_UNSUPPORTED;
  return ROCO_OK;
}

roco_status check_scope(int r, int scope_mode, int B, bool decode) {
  if (scope_mode == ROCO_SCOPE_EXCLUDE_TOP_R) return (r >= 0 && (decode ? r < B : r <= B)) ? ROCO_OK : ROCO_ERR_INVALID_ARG;
  if (scope_mode == ROCO_SCOPE_LOWEST_R) return (r >= 1 && r <= B) ? ROCO_OK : ROCO_ERR_INVALID_ARG;
  return ROCO_ERR_INVALID_ARG;
}

struct PrefillWs {
  size_t lens_off, lse_off, s_off, q_off, dst_off, total;
};

PrefillWs prefill_ws(int S, int G, int Lmax) {
  PrefillWs w;
  const size_t per = align_up((size_t)S * G * (size_t)Lmax * 4, 256);
  w.lens_off = 0;
  w.lse_off = align_up((size_t)S * 4, 256);
  w.s_off = w.lse_off + per;
  w.q_off = w.s_off + per;
  w.dst_off = w.q_off + per;
  w.total = w.dst_off + per;
  return w;
}

// Copy stream and events of roco_decode_step_host, one set per device, created at the first call on that device
// and kept until the process exits.
constexpr int kHostChunks = 4;
constexpr int kHostMaxDevices = 64;
constexpr int kHostDepth = 2;  // steps in flight in the begin/end form
struct HostPipe {
  bool ready = false;
  cudaStream_t copy = nullptr;
  cudaEvent_t start = nullptr, done = nullptr, h2d[kHostChunks] = {}, ker[kHostChunks] = {};
  // begin/end form: an input and an output copy stream, and per staging set the three events of its last step
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t set_h2d[kHostDepth] = {}, set_ker[kHostDepth] = {}, set_d2h[kHostDepth] = {};
  bool set_used[kHostDepth] = {};
  unsigned long long begun = 0, ended = 0;
};

HostPipe *host_pipe() {
  static HostPipe pipes[kHostMaxDevices];
  static std::mutex mu;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kHostMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  HostPipe &hp = pipes[dev];
  if (!hp.ready) {
    bool ok = cudaStreamCreateWithFlags(&hp.copy, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&hp.done, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < kHostChunks; ++i)
      ok = cudaEventCreateWithFlags(&hp.h2d[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.ker[i], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) == cudaSuccess &&
         cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; ok && i < kHostDepth; ++i)
      ok = cudaEventCreateWithFlags(&hp.set_h2d[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.set_ker[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.set_d2h[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return nullptr;
    hp.ready = true;
  }
  return &hp;
}

int pow2_at_least(int x) {
  int p = 1;
  while (p < x) p <<= 1;
  return p;
}

}  // namespace

extern "C" {

int roco_version(void) { return 100; }

const char *roco_status_string(int st) {
  switch (st) {
    case ROCO_OK: return "ok";
    case ROCO_ERR_INVALID_ARG: return "invalid argument";
    case ROCO_ERR_UNSUPPORTED: return "unsupported shape, dtype or option";
    case ROCO_ERR_WORKSPACE: return "workspace missing or too small";
    case ROCO_ERR_CUDA: return "CUDA runtime error";
    case ROCO_ERR_STATE: return "device status word is set";
    default: return "unknown status";
  }
}

size_t roco_prefill_workspace_bytes(const roco_cache *cache, int Lmax) {
  if (!cache || Lmax < 1 || cache->S < 1 || cache->G < 1) return 0;
  return prefill_ws(cache->S, cache->G, Lmax).total;
}

size_t roco_prefill_workspace_bytes_lowest_r(const roco_cache *cache, int Lmax) {
  if (!cache || Lmax < 1 || cache->S < 1 || cache->G < 1) return 0;
  return prefill_ws(cache->S, cache->G, Lmax).total + (size_t)cache->S * cache->G * pow2_at_least(Lmax) * 8;
}

int roco_prefill_uses_tensor_cores(const roco_cache *cache) {
  return (cache && prefill_tc_supported(cache->kv_dtype, cache->d)) ? 1 : 0;
}

roco_status roco_prefill(const void *Q, const void *K, const void *V, const int32_t *lens_host, int Lmax, int B,
                         int r, int scope_mode, int count_self, float scale, roco_cache *cache, float *lse_out,
                         float *s_full, float *q_full, void *workspace, size_t workspace_bytes, void *stream) {
  return roco_prefill_with_output(Q, K, V, lens_host, Lmax, B, r, scope_mode, count_self, scale, cache, lse_out,
                                  s_full, q_full, nullptr, workspace, workspace_bytes, stream);
}

roco_status roco_prefill_with_output(const void *Q, const void *K, const void *V, const int32_t *lens_host, int Lmax,
                                     int B, int r, int scope_mode, int count_self, float scale, roco_cache *cache,
                                     float *lse_out, float *s_full, float *q_full, void *attn_out, void *workspace,
                                     size_t workspace_bytes, void *stream) {
  NvtxRange range("roco_prefill");
  roco_status st = check_cache(cache);
  if (st != ROCO_OK) return st;
  if (!Q || !K || !V || !lens_host || Lmax < 1 || B != cache->B) return ROCO_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V)) return ROCO_ERR_INVALID_ARG;
  if ((st = check_scope(r, scope_mode, B, false)) != ROCO_OK) return st;
  if (count_self != 1) return ROCO_ERR_UNSUPPORTED;
  // The tensor-core kernels take maxima on the raw scores and mask before scaling: right for a positive scale only
  // (any other goes to the CUDA-core path).
  const bool tc = prefill_tc_supported(cache->kv_dtype, cache->d) && scale > 0.f;
  if (attn_out && !aligned16(attn_out)) return ROCO_ERR_INVALID_ARG;
  int maxlen = 0;
  for (int b = 0; b < cache->S; ++b) {
    if (lens_host[b] < 1 || lens_host[b] > Lmax) return ROCO_ERR_INVALID_ARG;
    if (lens_host[b] > maxlen) maxlen = lens_host[b];
  }
  const bool lowest_evicts = scope_mode == ROCO_SCOPE_LOWEST_R && maxlen > B;
  if (lowest_evicts && r > budget_lowest_max_r()) return ROCO_ERR_UNSUPPORTED;
  if ((long long)cache->S * cache->G * ((maxlen + 63) / 64 + 1) > 0x7fffffffLL) return ROCO_ERR_UNSUPPORTED;
  const PrefillWs w = prefill_ws(cache->S, cache->G, Lmax);
  const size_t need = lowest_evicts ? roco_prefill_workspace_bytes_lowest_r(cache, Lmax) : w.total;
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return ROCO_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char *ws = static_cast<char *>(workspace);
  int *lens_dev = reinterpret_cast<int *>(ws + w.lens_off);
  float *lse = lse_out ? lse_out : reinterpret_cast<float *>(ws + w.lse_off);
  float *sf = s_full ? s_full : reinterpret_cast<float *>(ws + w.s_off);
  float *qf = q_full ? q_full : reinterpret_cast<float *>(ws + w.q_off);
  int *dst = reinterpret_cast<int *>(ws + w.dst_off);
  if (cudaMemcpyAsync(lens_dev, lens_host, (size_t)cache->S * 4, cudaMemcpyHostToDevice, cs) != cudaSuccess)
    return ROCO_ERR_CUDA;
  if (attn_out && tc) {
    st = launch_prefill_attend_tc(cache->S, cache->G, Lmax, lens_dev, maxlen, Q, K, V, scale, nullptr, lse, attn_out,
                                  cache->status, cs);
    if (st == ROCO_OK)
      st = launch_prefill_stats_tc(cache->S, cache->G, Lmax, lens_dev, maxlen, Q, K, scale, lse, sf, qf,
                                   cache->status, cs, true);
  } else if (tc) {
    st = launch_prefill_stats_tc(cache->S, cache->G, Lmax, lens_dev, maxlen, Q, K, scale, lse, sf, qf, cache->status,
                                 cs);
  } else {  // CUDA cores: log-sum-exp pass, statistics pass, and -- if asked for -- the output from that log-sum-exp
    st = launch_prefill_stats_simt(cache->kv_dtype, cache->d, cache->S, cache->G, Lmax, lens_dev, maxlen, Q, K, scale,
                                   lse, sf, qf, cs);
    if (st == ROCO_OK && attn_out)
      st = launch_prefill_attend_simt(cache->kv_dtype, cache->d, cache->S, cache->G, Lmax, lens_dev, maxlen, Q, K, V,
                                      scale, lse, attn_out, cs);
  }
  if (st != ROCO_OK) return st;
  return launch_budget_select_gather(*cache, Lmax, lens_dev, maxlen, r, scope_mode, K, V, sf, qf, dst,
                                     reinterpret_cast<unsigned long long *>(ws + w.total), pow2_at_least(Lmax), cs);
}

size_t roco_prefill_attend_workspace_bytes(const roco_cache *cache) {
  if (!cache || cache->S < 1) return 0;
  return align_up((size_t)cache->S * 4, 256);
}

roco_status roco_prefill_attend(const roco_cache *cache, const void *Q, const void *K, const void *V,
                                const int32_t *lens_host, int Lmax, float scale, const float *lse, void *attn_out,
                                void *workspace, size_t workspace_bytes, void *stream) {
  NvtxRange range("roco_prefill_attend");
  if (!cache || !cache->status || cache->S < 1 || cache->G < 1) return ROCO_ERR_INVALID_ARG;
  if (!Q || !K || !V || !lens_host || !lse || !attn_out || Lmax < 1) return ROCO_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(attn_out)) return ROCO_ERR_INVALID_ARG;
  if ((cache->kv_dtype != ROCO_F32 && cache->kv_dtype != ROCO_BF16) || (cache->d != 64 && cache->d != 128))
    return ROCO_ERR_UNSUPPORTED;
  int maxlen = 0;
  for (int b = 0; b < cache->S; ++b) {
    if (lens_host[b] < 1 || lens_host[b] > Lmax) return ROCO_ERR_INVALID_ARG;
    if (lens_host[b] > maxlen) maxlen = lens_host[b];
  }
  if ((long long)cache->S * cache->G * ((maxlen + 63) / 64 + 1) > 0x7fffffffLL) return ROCO_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < roco_prefill_attend_workspace_bytes(cache) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return ROCO_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  int *lens_dev = static_cast<int *>(workspace);
  if (cudaMemcpyAsync(lens_dev, lens_host, (size_t)cache->S * 4, cudaMemcpyHostToDevice, cs) != cudaSuccess)
    return ROCO_ERR_CUDA;
  if (!prefill_tc_supported(cache->kv_dtype, cache->d) || !(scale > 0.f))
    return launch_prefill_attend_simt(cache->kv_dtype, cache->d, cache->S, cache->G, Lmax, lens_dev, maxlen, Q, K, V,
                                      scale, lse, attn_out, cs);
  return launch_prefill_attend_tc(cache->S, cache->G, Lmax, lens_dev, maxlen, Q, K, V, scale, lse, nullptr, attn_out,
                                  cache->status, cs);
}

roco_status roco_decode_step(roco_cache *cache, const void *q, const void *k_new, const void *v_new, int r,
                             int scope_mode, int step_order, float scale, void *attn_out, float *lse_out,
                             int32_t *evicted_slot, int32_t *evicted_pos, void *stream) {
  // the launch shape follows the call's size: one CTA per unit, or a cluster of CTAs per unit when the units are few
  return roco_decode_step_cluster(cache, q, k_new, v_new, r, scope_mode, step_order, 0, scale, attn_out, lse_out,
                                  evicted_slot, evicted_pos, stream);
}

size_t roco_decode_split_workspace_bytes(const roco_cache *cache, int splits) {
  if (!cache || cache->S < 1 || cache->G < 1 || splits < 1 || splits > 64) return 0;
  return decode_split_workspace_bytes(cache->S * cache->G, cache->B, cache->d, splits);
}

roco_status roco_decode_step_split(roco_cache *cache, const void *q, const void *k_new, const void *v_new, int r,
                                   int scope_mode, int splits, float scale, void *attn_out, float *lse_out,
                                   int32_t *evicted_slot, int32_t *evicted_pos, void *workspace,
                                   size_t workspace_bytes, void *stream) {
  return roco_decode_step_split_ordered(cache, q, k_new, v_new, r, scope_mode, ROCO_EVICT_FIRST, splits, scale,
                                        attn_out, lse_out, evicted_slot, evicted_pos, workspace, workspace_bytes,
                                        stream);
}

roco_status roco_decode_step_split_ordered(roco_cache *cache, const void *q, const void *k_new, const void *v_new,
                                           int r, int scope_mode, int step_order, int splits, float scale,
                                           void *attn_out, float *lse_out, int32_t *evicted_slot,
                                           int32_t *evicted_pos, void *workspace, size_t workspace_bytes,
                                           void *stream) {
  NvtxRange range("roco_decode_step_split");
  roco_status st = check_cache(cache);
  if (st != ROCO_OK) return st;
  if (!q || !k_new || !v_new || !attn_out || !evicted_slot) return ROCO_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(attn_out)) return ROCO_ERR_INVALID_ARG;
  if ((st = check_scope(r, scope_mode, cache->B, true)) != ROCO_OK) return st;
  if (splits < 1 || splits > 64) return ROCO_ERR_INVALID_ARG;
  if (step_order != ROCO_EVICT_FIRST && step_order != ROCO_ATTEND_FIRST) return ROCO_ERR_INVALID_ARG;
  const size_t need = roco_decode_split_workspace_bytes(cache, splits);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return ROCO_ERR_WORKSPACE;
  return launch_decode_step_split(*cache, q, k_new, v_new, r, scope_mode, step_order, splits, scale, attn_out,
                                  lse_out, evicted_slot, evicted_pos, workspace, static_cast<cudaStream_t>(stream));
}

int roco_decode_cluster_ranks(const roco_cache *cache) {
  if (check_cache(cache) != ROCO_OK) return 0;
  static int sm_count[kHostMaxDevices] = {};  // per device, asked once (racing first calls write the same value)
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kHostMaxDevices) return 0;
  if (sm_count[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 0;
    sm_count[dev] = n;
  }
  const int sms = sm_count[dev];
  if (((reinterpret_cast<uintptr_t>(cache->s) | reinterpret_cast<uintptr_t>(cache->q) |
        reinterpret_cast<uintptr_t>(cache->n) | reinterpret_cast<uintptr_t>(cache->pos)) & 15) != 0)
    return 1;
  return decode_cluster_ranks(cache->S * cache->G, cache->B, cache->d, cache->kv_dtype == ROCO_BF16 ? 2 : 4, sms);
}

roco_status roco_decode_step_cluster(roco_cache *cache, const void *q, const void *k_new, const void *v_new, int r,
                                     int scope_mode, int step_order, int ranks, float scale, void *attn_out,
                                     float *lse_out, int32_t *evicted_slot, int32_t *evicted_pos, void *stream) {
  NvtxRange range("roco_decode_step");
  roco_status st = check_cache(cache);
  if (st != ROCO_OK) return st;
  if (!q || !k_new || !v_new || !attn_out || !evicted_slot) return ROCO_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(attn_out)) return ROCO_ERR_INVALID_ARG;
  if ((st = check_scope(r, scope_mode, cache->B, true)) != ROCO_OK) return st;
  if (step_order != ROCO_EVICT_FIRST && step_order != ROCO_ATTEND_FIRST) return ROCO_ERR_INVALID_ARG;
  const bool automatic = ranks == 0;
  if (automatic) {
    ranks = roco_decode_cluster_ranks(cache);
    if (ranks > 1) {
      // a cluster launch can be refused where the device cannot co-schedule that many CTAs (a partitioned GPU):
      // nothing has been enqueued then, and the step still runs with one CTA per unit
      st = launch_decode_step_cluster(*cache, ranks, q, k_new, v_new, r, scope_mode, step_order, scale, attn_out,
                                      lse_out, evicted_slot, evicted_pos, static_cast<cudaStream_t>(stream));
      if (st == ROCO_OK) return st;
      (void)cudaGetLastError();
      ranks = 1;
    }
  }
  if (ranks == 1)
    return launch_decode_step(*cache, q, k_new, v_new, r, scope_mode, step_order, ROCO_POLICY_ROCO, nullptr, scale,
                              attn_out, lse_out, evicted_slot, evicted_pos, static_cast<cudaStream_t>(stream));
  if (ranks != 2 && ranks != 4 && ranks != 8) return ROCO_ERR_INVALID_ARG;
  return launch_decode_step_cluster(*cache, ranks, q, k_new, v_new, r, scope_mode, step_order, scale, attn_out,
                                    lse_out, evicted_slot, evicted_pos, static_cast<cudaStream_t>(stream));
}

roco_status roco_decode_step_policy_ordered(roco_cache *cache, const void *q, const void *k_new, const void *v_new,
                                            int policy, int r, int step_order, const uint32_t *rnd, float scale,
                                            void *attn_out, float *lse_out, int32_t *evicted_slot,
                                            int32_t *evicted_pos, void *stream) {
  NvtxRange range("roco_decode_step_policy");
  roco_status st = check_cache(cache);
  if (st != ROCO_OK) return st;
  if (!q || !k_new || !v_new || !attn_out || !evicted_slot) return ROCO_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(attn_out)) return ROCO_ERR_INVALID_ARG;
  if (policy < ROCO_POLICY_ROCO || policy > ROCO_POLICY_MAS_WINDOW) return ROCO_ERR_INVALID_ARG;
  if (step_order != ROCO_EVICT_FIRST && step_order != ROCO_ATTEND_FIRST) return ROCO_ERR_INVALID_ARG;
  if (r < 0 || r >= cache->B) return ROCO_ERR_INVALID_ARG;
  if (policy == ROCO_POLICY_RANDOM && !rnd) return ROCO_ERR_INVALID_ARG;
  if (policy == ROCO_POLICY_STREAMLLM && cache->B <= 4) return ROCO_ERR_INVALID_ARG;  // room for the four sinks
  return launch_decode_step(*cache, q, k_new, v_new, r, ROCO_SCOPE_EXCLUDE_TOP_R, step_order, policy, rnd, scale,
                            attn_out, lse_out, evicted_slot, evicted_pos, static_cast<cudaStream_t>(stream));
}

roco_status roco_decode_step_policy(roco_cache *cache, const void *q, const void *k_new, const void *v_new,
                                    int policy, int r, const uint32_t *rnd, float scale, void *attn_out,
                                    float *lse_out, int32_t *evicted_slot, int32_t *evicted_pos, void *stream) {
  return roco_decode_step_policy_ordered(cache, q, k_new, v_new, policy, r, ROCO_EVICT_FIRST, rnd, scale, attn_out,
                                         lse_out, evicted_slot, evicted_pos, stream);
}

roco_status roco_gqa_block_step(roco_cache *cache, const void *Q, const void *K_new, const void *V_new, int b,
                                int group, int r, int scope_mode, float scale, void *attn_out, float *lse_out,
                                int32_t *evicted_slot, int32_t *evicted_pos, void *stream) {
  NvtxRange range("roco_gqa_block_step");
  roco_status st = check_cache(cache);
  if (st != ROCO_OK) return st;
  if (!Q || !K_new || !V_new || !attn_out || !evicted_slot) return ROCO_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K_new) || !aligned16(V_new) || !aligned16(attn_out)) return ROCO_ERR_INVALID_ARG;
  if (b < 1 || group < 1) return ROCO_ERR_INVALID_ARG;
  if ((st = check_scope(r, scope_mode, cache->B, true)) != ROCO_OK) return st;
  if ((long long)b * group > multi_max_queries()) return ROCO_ERR_UNSUPPORTED;
  if (b > 1 && r + b > cache->B) return ROCO_ERR_INVALID_ARG;  // the scope must hold the b victims
  if (b == 1 && group == 1)  // one token, one head: the decode step in the order of Fig. 1 (same layouts), which
                             // also picks its launch shape from the number of units
    return roco_decode_step(cache, Q, K_new, V_new, r, scope_mode, ROCO_EVICT_FIRST, scale, attn_out, lse_out,
                            evicted_slot, evicted_pos, stream);
  if (!multi_fits(cache->B, cache->d, b * group, b)) return ROCO_ERR_UNSUPPORTED;
  return launch_multi_step(*cache, b * group, b, Q, K_new, V_new, r, scope_mode, scale, attn_out, lse_out,
                           evicted_slot, evicted_pos, static_cast<cudaStream_t>(stream));
}

roco_status roco_block_step(roco_cache *cache, const void *Q, const void *K_new, const void *V_new, int b, int r,
                            int scope_mode, float scale, void *attn_out, float *lse_out, int32_t *evicted_slot,
                            int32_t *evicted_pos, void *stream) {
  return roco_gqa_block_step(cache, Q, K_new, V_new, b, 1, r, scope_mode, scale, attn_out, lse_out, evicted_slot,
                             evicted_pos, stream);
}

roco_status roco_prefill_blockwise_gqa(const void *Q, const void *K, const void *V, const int32_t *lens_host,
                                       int Lmax, int b, int group, int r, float scale, roco_cache *cache,
                                       void *attn_out, int32_t *evicted_slot, void *stream) {
  NvtxRange range("roco_prefill_blockwise");
  roco_status st = check_cache(cache);
  if (st != ROCO_OK) return st;
  if (!Q || !K || !V || !lens_host || !attn_out || !evicted_slot || Lmax < 1 || b < 1 || group < 1)
    return ROCO_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(attn_out)) return ROCO_ERR_INVALID_ARG;
  if ((st = check_scope(r, ROCO_SCOPE_EXCLUDE_TOP_R, cache->B, true)) != ROCO_OK) return st;
  if ((long long)b * group > multi_max_queries()) return ROCO_ERR_UNSUPPORTED;
  if (b > 1 && r + b > cache->B) return ROCO_ERR_INVALID_ARG;
  if (!multi_fits(cache->B, cache->d, b * group, b)) return ROCO_ERR_UNSUPPORTED;
  for (int s = 0; s < cache->S; ++s)
    if (lens_host[s] < 1 || lens_host[s] > Lmax) return ROCO_ERR_INVALID_ARG;
  const size_t elem = cache->kv_dtype == ROCO_BF16 ? 2 : 4;
  const size_t G = (size_t)cache->G, B = (size_t)cache->B, d = (size_t)cache->d;
  // Consecutive sequences of equal length advance together: one launch per block for the whole run.
  for (int s0 = 0; s0 < cache->S;) {
    int s1 = s0 + 1;
    while (s1 < cache->S && lens_host[s1] == lens_host[s0]) ++s1;
    const int len = lens_host[s0];
    roco_cache sub = *cache;  // the units of sequences s0 .. s1 - 1
    sub.S = s1 - s0;
    sub.K = static_cast<char *>(cache->K) + s0 * G * B * d * elem;
    sub.V = static_cast<char *>(cache->V) + s0 * G * B * d * elem;
    sub.s = cache->s + s0 * G * B; sub.q = cache->q + s0 * G * B;
    sub.n = cache->n + s0 * G * B; sub.pos = cache->pos + s0 * G * B;
    sub.live = cache->live + s0 * G; sub.t_next = cache->t_next + s0 * G;
    for (int t0 = 0; t0 < len; t0 += b) {
      const int m = len - t0 < b ? len - t0 : b;
      const size_t off = ((size_t)s0 * G * Lmax + t0) * d * elem;  // K, V: one row per token; Q, out: `group` rows
      st = launch_multi_step(sub, m * group, m, static_cast<const char *>(Q) + off * group,
                             static_cast<const char *>(K) + off, static_cast<const char *>(V) + off, r,
                             ROCO_SCOPE_EXCLUDE_TOP_R, scale, static_cast<char *>(attn_out) + off * group, nullptr,
                             evicted_slot + (size_t)s0 * G * b, nullptr, static_cast<cudaStream_t>(stream), Lmax);
      if (st != ROCO_OK) return st;
    }
    s0 = s1;
  }
  return ROCO_OK;
}

roco_status roco_prefill_blockwise(const void *Q, const void *K, const void *V, const int32_t *lens_host, int Lmax,
                                   int b, int r, float scale, roco_cache *cache, void *attn_out,
                                   int32_t *evicted_slot, void *stream) {
  return roco_prefill_blockwise_gqa(Q, K, V, lens_host, Lmax, b, 1, r, scale, cache, attn_out, evicted_slot, stream);
}

roco_status roco_gqa_decode_step(roco_cache *cache, const void *Q, const void *k_new, const void *v_new, int group,
                                 int r, int scope_mode, float scale, void *attn_out, float *lse_out,
                                 int32_t *evicted_slot, int32_t *evicted_pos, void *stream) {
  NvtxRange range("roco_gqa_decode_step");
  roco_status st = check_cache(cache);
  if (st != ROCO_OK) return st;
  if (!Q || !k_new || !v_new || !attn_out || !evicted_slot) return ROCO_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(attn_out)) return ROCO_ERR_INVALID_ARG;
  if (group < 1) return ROCO_ERR_INVALID_ARG;
  if ((st = check_scope(r, scope_mode, cache->B, true)) != ROCO_OK) return st;
  if (group > multi_max_queries() || !multi_fits(cache->B, cache->d, group, 1)) return ROCO_ERR_UNSUPPORTED;
  return launch_multi_step(*cache, group, 1, Q, k_new, v_new, r, scope_mode, scale, attn_out, lse_out,
                           evicted_slot, evicted_pos, static_cast<cudaStream_t>(stream));
}

roco_status roco_consistency_step(const roco_cache *full, const roco_cache *budgeted, int policy, int32_t *overlap,
                                  float *jaccard_sum, int32_t *samples, void *stream) {
  NvtxRange range("roco_consistency_step");
  roco_status st = check_cache(full);
  if (st != ROCO_OK) return st;
  if ((st = check_cache(budgeted)) != ROCO_OK) return st;
  if (!overlap || !jaccard_sum || !samples) return ROCO_ERR_INVALID_ARG;
  if (full->S != budgeted->S || full->G != budgeted->G || full->B < budgeted->B) return ROCO_ERR_INVALID_ARG;
  if (policy != ROCO_POLICY_ROCO && policy != ROCO_POLICY_SCISSORHANDS && policy != ROCO_POLICY_H2O &&
      policy != ROCO_POLICY_TOVA && policy != ROCO_POLICY_MAS_WINDOW)
    return ROCO_ERR_INVALID_ARG;  // the other policies have no attention-based score
  return launch_consistency_step(*full, *budgeted, policy, overlap, jaccard_sum, samples,
                                 static_cast<cudaStream_t>(stream));
}

size_t roco_decode_host_staging_bytes(const roco_cache *cache) {
  if (!cache || cache->S < 1 || cache->G < 1) return 0;
  const size_t U = (size_t)cache->S * cache->G;
  const size_t vec = align_up(U * cache->d * (cache->kv_dtype == ROCO_BF16 ? 2 : 4), 256);
  return 4 * vec + 2 * align_up(U * 4, 256);
}

roco_status roco_decode_step_host(roco_cache *cache, const void *q_host, const void *k_new_host,
                                  const void *v_new_host, int r, int scope_mode, int step_order, float scale,
                                  void *attn_out_host, int32_t *evicted_slot_host, int32_t *evicted_pos_host,
                                  void *staging, size_t staging_bytes, void *stream) {
  NvtxRange range("roco_decode_step_host");
  roco_status st = check_cache(cache);
  if (st != ROCO_OK) return st;
  if (!q_host || !k_new_host || !v_new_host || !attn_out_host || !evicted_slot_host) return ROCO_ERR_INVALID_ARG;
  if (!staging || staging_bytes < roco_decode_host_staging_bytes(cache) ||
      (reinterpret_cast<uintptr_t>(staging) & 255u))
    return ROCO_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const size_t U = (size_t)cache->S * cache->G;
  const size_t esz = cache->kv_dtype == ROCO_BF16 ? 2 : 4;
  const size_t row = (size_t)cache->d * esz;  // bytes of one unit's vector
  const size_t vbytes = U * row;
  const size_t vec = align_up(vbytes, 256), ivec = align_up(U * 4, 256);
  char *p = static_cast<char *>(staging);
  char *dq = p, *dk = p + vec, *dv = p + 2 * vec, *dout = p + 3 * vec;
  int32_t *dslot = reinterpret_cast<int32_t *>(p + 4 * vec), *dpos = reinterpret_cast<int32_t *>(p + 4 * vec + ivec);

  HostPipe *hp = U >= 2048 ? host_pipe() : nullptr;
  if (!hp) {  // few units (or no copy stream): copy in, one launch, copy out, all on the caller's stream
    if (cudaMemcpyAsync(dq, q_host, vbytes, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
        cudaMemcpyAsync(dk, k_new_host, vbytes, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
        cudaMemcpyAsync(dv, v_new_host, vbytes, cudaMemcpyHostToDevice, cs) != cudaSuccess)
      return ROCO_ERR_CUDA;
    st = roco_decode_step(cache, dq, dk, dv, r, scope_mode, step_order, scale, dout, nullptr, dslot, dpos, stream);
    if (st != ROCO_OK) return st;
    if (cudaMemcpyAsync(attn_out_host, dout, vbytes, cudaMemcpyDeviceToHost, cs) != cudaSuccess ||
        cudaMemcpyAsync(evicted_slot_host, dslot, U * 4, cudaMemcpyDeviceToHost, cs) != cudaSuccess)
      return ROCO_ERR_CUDA;
    if (evicted_pos_host &&
        cudaMemcpyAsync(evicted_pos_host, dpos, U * 4, cudaMemcpyDeviceToHost, cs) != cudaSuccess)
      return ROCO_ERR_CUDA;
    return cudaStreamSynchronize(cs) == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
  }

  // Units are independent, so the step is cut into kHostChunks unit ranges: the copies of a range run on the copy
  // stream while the kernel of the previous range runs on the caller's stream.
  const char *hq = static_cast<const char *>(q_host), *hk = static_cast<const char *>(k_new_host),
             *hv = static_cast<const char *>(v_new_host);
  char *hout = static_cast<char *>(attn_out_host);
  auto ok = [](cudaError_t e) { return e == cudaSuccess; };
  if (!ok(cudaEventRecord(hp->start, cs)) || !ok(cudaStreamWaitEvent(hp->copy, hp->start, 0))) return ROCO_ERR_CUDA;
  size_t lo[kHostChunks + 1];
  for (int c = 0; c <= kHostChunks; ++c) lo[c] = U * c / kHostChunks;
  for (int c = 0; c < kHostChunks && st == ROCO_OK; ++c) {  // inputs of range c in, then its kernel (launched early)
    const size_t u0 = lo[c], nu = lo[c + 1] - lo[c], off = u0 * row, nb = nu * row;
    if (!ok(cudaMemcpyAsync(dq + off, hq + off, nb, cudaMemcpyHostToDevice, hp->copy)) ||
        !ok(cudaMemcpyAsync(dk + off, hk + off, nb, cudaMemcpyHostToDevice, hp->copy)) ||
        !ok(cudaMemcpyAsync(dv + off, hv + off, nb, cudaMemcpyHostToDevice, hp->copy)) ||
        !ok(cudaEventRecord(hp->h2d[c], hp->copy)) || !ok(cudaStreamWaitEvent(cs, hp->h2d[c], 0))) {
      st = ROCO_ERR_CUDA;
      break;
    }
    roco_cache view = *cache;  // the units u0 .. u0 + nu - 1 as a cache of their own
    view.S = 1;
    view.G = (int32_t)nu;
    view.K = static_cast<char *>(cache->K) + u0 * cache->B * row;
    view.V = static_cast<char *>(cache->V) + u0 * cache->B * row;
    view.s = cache->s + u0 * cache->B;
    view.q = cache->q + u0 * cache->B;
    view.n = cache->n + u0 * cache->B;
    view.pos = cache->pos + u0 * cache->B;
    view.live = cache->live + u0;
    view.t_next = cache->t_next + u0;
    st = roco_decode_step(&view, dq + off, dk + off, dv + off, r, scope_mode, step_order, scale, dout + off, nullptr,
                          dslot + u0, dpos + u0, stream);
    if (st == ROCO_OK && !ok(cudaEventRecord(hp->ker[c], cs))) st = ROCO_ERR_CUDA;
  }
  for (int c = 0; c < kHostChunks && st == ROCO_OK; ++c) {  // results out, behind the last input copy
    const size_t u0 = lo[c], nu = lo[c + 1] - lo[c];
    if (!ok(cudaStreamWaitEvent(hp->copy, hp->ker[c], 0)) ||
        !ok(cudaMemcpyAsync(hout + u0 * row, dout + u0 * row, nu * row, cudaMemcpyDeviceToHost, hp->copy)) ||
        !ok(cudaMemcpyAsync(evicted_slot_host + u0, dslot + u0, nu * 4, cudaMemcpyDeviceToHost, hp->copy)) ||
        (evicted_pos_host &&
         !ok(cudaMemcpyAsync(evicted_pos_host + u0, dpos + u0, nu * 4, cudaMemcpyDeviceToHost, hp->copy))))
      st = ROCO_ERR_CUDA;
  }
  // whatever was enqueued is drained before returning, also after an error
  const bool drained = ok(cudaEventRecord(hp->done, hp->copy)) && ok(cudaStreamWaitEvent(cs, hp->done, 0)) &&
                       ok(cudaStreamSynchronize(cs)) && ok(cudaStreamSynchronize(hp->copy));
  if (st != ROCO_OK) return st;
  return drained ? ROCO_OK : ROCO_ERR_CUDA;
}

size_t roco_decode_host_pipeline_staging_bytes(const roco_cache *cache) {
  return kHostDepth * roco_decode_host_staging_bytes(cache);
}

roco_status roco_decode_step_host_begin(roco_cache *cache, const void *q_host, const void *k_new_host,
                                        const void *v_new_host, int r, int scope_mode, int step_order, float scale,
                                        void *attn_out_host, int32_t *evicted_slot_host, int32_t *evicted_pos_host,
                                        void *staging, size_t staging_bytes, void *stream) {
  NvtxRange range("roco_decode_step_host_begin");
  roco_status st = check_cache(cache);
  if (st != ROCO_OK) return st;
  if (!q_host || !k_new_host || !v_new_host || !attn_out_host || !evicted_slot_host) return ROCO_ERR_INVALID_ARG;
  const size_t one = roco_decode_host_staging_bytes(cache);
  if (!staging || staging_bytes < kHostDepth * one || (reinterpret_cast<uintptr_t>(staging) & 255u))
    return ROCO_ERR_WORKSPACE;
  HostPipe *hp = host_pipe();
  if (!hp) return ROCO_ERR_CUDA;
  if (hp->begun - hp->ended >= kHostDepth) return ROCO_ERR_STATE;  // end a step first
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int set = (int)(hp->begun % kHostDepth);
  const size_t U = (size_t)cache->S * cache->G;
  const size_t vbytes = U * cache->d * (cache->kv_dtype == ROCO_BF16 ? 2 : 4);
  const size_t vec = align_up(vbytes, 256), ivec = align_up(U * 4, 256);
  char *p = static_cast<char *>(staging) + set * one;
  char *dq = p, *dk = p + vec, *dv = p + 2 * vec, *dout = p + 3 * vec;
  int32_t *dslot = reinterpret_cast<int32_t *>(p + 4 * vec), *dpos = reinterpret_cast<int32_t *>(p + 4 * vec + ivec);
  auto ok = [](cudaError_t e) { return e == cudaSuccess; };
  // inputs of this step: the set's input buffers were last read by the kernel two steps ago
  if (hp->set_used[set] && !ok(cudaStreamWaitEvent(hp->in, hp->set_ker[set], 0))) return ROCO_ERR_CUDA;
  if (!ok(cudaMemcpyAsync(dq, q_host, vbytes, cudaMemcpyHostToDevice, hp->in)) ||
      !ok(cudaMemcpyAsync(dk, k_new_host, vbytes, cudaMemcpyHostToDevice, hp->in)) ||
      !ok(cudaMemcpyAsync(dv, v_new_host, vbytes, cudaMemcpyHostToDevice, hp->in)) ||
      !ok(cudaEventRecord(hp->set_h2d[set], hp->in)) || !ok(cudaStreamWaitEvent(cs, hp->set_h2d[set], 0)))
    return ROCO_ERR_CUDA;
  // the kernel: the set's output buffers were last read by the copy-out two steps ago
  if (hp->set_used[set] && !ok(cudaStreamWaitEvent(cs, hp->set_d2h[set], 0))) return ROCO_ERR_CUDA;
  st = roco_decode_step(cache, dq, dk, dv, r, scope_mode, step_order, scale, dout, nullptr, dslot, dpos, stream);
  if (st != ROCO_OK) return st;
  if (!ok(cudaEventRecord(hp->set_ker[set], cs)) || !ok(cudaStreamWaitEvent(hp->out, hp->set_ker[set], 0)) ||
      !ok(cudaMemcpyAsync(attn_out_host, dout, vbytes, cudaMemcpyDeviceToHost, hp->out)) ||
      !ok(cudaMemcpyAsync(evicted_slot_host, dslot, U * 4, cudaMemcpyDeviceToHost, hp->out)) ||
      (evicted_pos_host && !ok(cudaMemcpyAsync(evicted_pos_host, dpos, U * 4, cudaMemcpyDeviceToHost, hp->out))) ||
      !ok(cudaEventRecord(hp->set_d2h[set], hp->out)))
    return ROCO_ERR_CUDA;
  hp->set_used[set] = true;
  ++hp->begun;
  return ROCO_OK;
}

roco_status roco_decode_step_host_end(void) {
  NvtxRange range("roco_decode_step_host_end");
  HostPipe *hp = host_pipe();
  if (!hp) return ROCO_ERR_CUDA;
  if (hp->begun == hp->ended) return ROCO_ERR_STATE;  // nothing in flight
  const int set = (int)(hp->ended % kHostDepth);
  ++hp->ended;
  return cudaEventSynchronize(hp->set_d2h[set]) == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

roco_status roco_device_status(const roco_cache *cache, void *stream, int32_t *flags_host) {
  if (!cache || !cache->status || !flags_host) return ROCO_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(flags_host, cache->status, 4, cudaMemcpyDeviceToHost, cs) != cudaSuccess) return ROCO_ERR_CUDA;
  if (cudaStreamSynchronize(cs) != cudaSuccess) return ROCO_ERR_CUDA;
  return *flags_host ? ROCO_ERR_STATE : ROCO_OK;
}

}  // extern "C"
