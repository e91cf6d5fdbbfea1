// One decode step of KV-constrained inference with RoCo eviction (Sec. 3, Sec. 4.3, Fig. 1), one CTA per
// unit.  The step is bound by HBM traffic: each unit's K and V blocks are streamed exactly once through a
// shared-memory ring filled by bulk asynchronous copies (TMA, one producer warp), the B scores stay in
// shared memory (no online softmax needed), the statistics update rides between the two passes, and the
// scope / victim selection and the in-place slot overwrite happen in the same launch while the ring is
// being filled -- so the per-unit traffic is 2*B*d elements of K/V plus the B-sized statistics arrays.
#include "common.cuh"
#include "launch.h"
#include "select.cuh"

namespace roco {

constexpr int kConsumerWarps = 8;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kDecodeThreads = kConsumers + 32;  // + one producer warp
constexpr int kTileBytes = 16384;
constexpr int kBarConsumers = 1;  // named barrier id used by the consumer warps

struct DecodeParams {
  const char *K, *V;
  float *s, *q;
  int *n, *pos, *live, *t_next, *status;
  const char *qv, *k_new, *v_new;
  char *out;
  float *lse;
  int *ev_slot, *ev_pos;
  int B, r, scope_mode, order, stages;
  float scale;
};

struct DecodeSmem {
  // carve-up of dynamic shared memory; `stages` ring buffers come first (128-byte aligned)
  char *ring;
  uint64_t *full, *empty;
  float *z;  // scores, then probabilities; doubles as the selection's key array
  float *s, *q;
  int *n, *pos;
  float *qf, *knew, *vnew, *outred, *red;
  SelectScratch *sel;
  int *flags;  // [0] abort flag
};

__host__ __device__ inline size_t decode_smem_bytes(int B, int d, int stages) {
  size_t Bp = align_up((size_t)B, 4);
  size_t b = (size_t)stages * kTileBytes;
  b += 2 * (size_t)stages * sizeof(uint64_t);
  b = align_up(b, 16);
  b += 5 * Bp * 4;                            // z, s, q, n, pos
  b += (size_t)(3 + kConsumerWarps) * d * 4;  // qf, knew, vnew, outred
  b += 64 * 4;                                // red
  b = align_up(b, 16);
  b += sizeof(SelectScratch);
  b += 16;
  return b + 128;  // slack for aligning the base
}

__device__ inline DecodeSmem carve(char *raw, int B, int d, int stages) {
  DecodeSmem m;
  char *p = (char *)align_up((size_t)raw, 128);
  m.ring = p; p += (size_t)stages * kTileBytes;
  m.full = (uint64_t *)p; p += stages * sizeof(uint64_t);
  m.empty = (uint64_t *)p; p += stages * sizeof(uint64_t);
  p = (char *)align_up((size_t)p, 16);
  size_t Bp = align_up((size_t)B, 4);
  m.z = (float *)p; p += Bp * 4;
  m.s = (float *)p; p += Bp * 4;
  m.q = (float *)p; p += Bp * 4;
  m.n = (int *)p; p += Bp * 4;
  m.pos = (int *)p; p += Bp * 4;
  m.qf = (float *)p; p += d * 4;
  m.knew = (float *)p; p += d * 4;
  m.vnew = (float *)p; p += d * 4;
  m.outred = (float *)p; p += (size_t)kConsumerWarps * d * 4;
  m.red = (float *)p; p += 64 * 4;
  p = (char *)align_up((size_t)p, 16);
  m.sel = (SelectScratch *)p; p += sizeof(SelectScratch);
  m.flags = (int *)p;
  return m;
}

__device__ __forceinline__ float consumers_max(float v, float *red, int tid) {
  v = warp_max(v);
  if ((tid & 31) == 0) red[tid >> 5] = v;
  named_bar_sync(kBarConsumers, kConsumers);
  float r = red[0];
#pragma unroll
  for (int w = 1; w < kConsumerWarps; ++w) r = fmaxf(r, red[w]);
  named_bar_sync(kBarConsumers, kConsumers);
  return r;
}

__device__ __forceinline__ float consumers_sum(float v, float *red, int tid) {
  v = warp_sum(v);
  if ((tid & 31) == 0) red[tid >> 5] = v;
  named_bar_sync(kBarConsumers, kConsumers);
  float r = red[0];
#pragma unroll
  for (int w = 1; w < kConsumerWarps; ++w) r += red[w];
  named_bar_sync(kBarConsumers, kConsumers);
  return r;
}

template <typename T, int D>
__global__ void __launch_bounds__(kDecodeThreads) decode_step_kernel(const DecodeParams p) {
  constexpr int kRowBytes = D * (int)sizeof(T);
  constexpr int kLanesPerRow = kRowBytes / 16;
  constexpr int kRowsPerLoad = 32 / kLanesPerRow;
  constexpr int kTileRows = kTileBytes / kRowBytes;
  constexpr int kRowsPerWarp = kTileRows / kConsumerWarps;
  constexpr int kLoads = kRowsPerWarp / kRowsPerLoad;
  constexpr int kEPC = Elem<T>::kPerChunk;
  static_assert(kLanesPerRow <= 32 && kLoads >= 1, "tile shape");

  extern __shared__ char smem_raw[];
  const DecodeSmem sm = carve(smem_raw, p.B, D, p.stages);
  volatile int *abort_flag = sm.flags;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int u = blockIdx.x;
  const int B = p.B;
  const size_t unit_kv = (size_t)u * B * kRowBytes;
  const size_t unit_st = (size_t)u * B;

  int live0 = p.live[u];
  if (live0 < 0 || live0 > B) {
    if (tid == 0) atomicOr(p.status, ROCO_DEV_BAD_LIVE);
    live0 = live0 < 0 ? 0 : B;
  }
  const bool full = (live0 == B);
  const bool evict_first = (p.order == ROCO_EVICT_FIRST);
  const int live_att = evict_first ? (full ? B : live0 + 1) : live0;  // slots the query attends over
  const int live_new = full ? B : live0 + 1;
  const int n_tiles = (live_att + kTileRows - 1) / kTileRows;
  const int stages = p.stages;

  if (tid == 0) {
    for (int i = 0; i < stages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], kConsumerWarps); }
    sm.flags[0] = 0;
    mbar_init_fence();
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------ producer: K tiles, then V tiles
    if (lane == 0) {
      for (int g = 0; g < 2 * n_tiles; ++g) {
        const int st = g % stages;
        if (g >= stages) mbar_wait(&sm.empty[st], ((g / stages) - 1) & 1, abort_flag, p.status);
        const int it = (g < n_tiles) ? g : g - n_tiles;
        const char *src = ((g < n_tiles) ? p.K : p.V) + unit_kv + (size_t)it * kTileBytes;
        int rows = live_att - it * kTileRows;
        if (rows > kTileRows) rows = kTileRows;
        const uint32_t bytes = (uint32_t)rows * kRowBytes;
        mbar_expect_tx(&sm.full[st], bytes);
        bulk_g2s(sm.ring + (size_t)st * kTileBytes, src, bytes, &sm.full[st]);
      }
    }
    return;
  }

  // -------------------------------------------------------------- consumers
  const int t_new = p.t_next[u];
  for (int j = tid; j < live0; j += kConsumers) {
    sm.s[j] = p.s[unit_st + j];
    sm.q[j] = p.q[unit_st + j];
    sm.n[j] = p.n[unit_st + j];
    sm.pos[j] = p.pos[unit_st + j];
  }
  if (tid < D) {
    const size_t o = (size_t)u * D + tid;
    sm.qf[tid] = Elem<T>::load((const T *)p.qv + o);
    sm.knew[tid] = Elem<T>::load((const T *)p.k_new + o);
    sm.vnew[tid] = Elem<T>::load((const T *)p.v_new + o);
  }
  named_bar_sync(kBarConsumers, kConsumers);

  int e = -1;  // slot the new token goes to
  int ev_slot = -1, ev_pos = -1;

  // Frees a slot if the buffer is full (Sec. 4: "when the buffer is full, an eviction policy is
  // executed"), writes the new token there with empty statistics.
  auto evict_and_insert = [&]() {
    if (full) {
      const int m = scope_size(B, p.r, p.scope_mode);
      e = block_select_victim(sm.s, sm.q, sm.n, sm.pos, B, m, (uint32_t *)sm.z, *sm.sel, tid, kConsumers,
                              kBarConsumers);
      if (e < 0) {
        if (tid == 0) atomicOr(p.status, ROCO_DEV_BAD_VICTIM);
        e = 0;
      }
      ev_slot = e;
      ev_pos = sm.pos[e];
    } else {
      e = live0;
    }
    named_bar_sync(kBarConsumers, kConsumers);  // everyone has read pos[e]
    if (tid == 0) { sm.s[e] = 0.f; sm.q[e] = 0.f; sm.n[e] = 0; sm.pos[e] = t_new; }
    if (tid < 2 * kLanesPerRow) {  // in-place overwrite of the freed slot, 16 bytes per thread
      const bool isv = tid >= kLanesPerRow;
      const int c = isv ? tid - kLanesPerRow : tid;
      const uint4 val = *((const uint4 *)((isv ? p.v_new : p.k_new) + (size_t)u * kRowBytes) + c);
      char *dst = const_cast<char *>(isv ? p.V : p.K) + unit_kv + (size_t)e * kRowBytes;
      *((uint4 *)dst + c) = val;
    }
    named_bar_sync(kBarConsumers, kConsumers);
  };

  if (evict_first) evict_and_insert();
  const int e_sub = evict_first ? e : -1;  // slot whose K/V come from k_new/v_new rather than the stream

  // ---- scores: z_j = scale * q.K[j]  (Eq. 1), kept in base 2
  const float zscale = p.scale * kLog2e;
  const int lane_chunk = lane % kLanesPerRow, lane_row = lane / kLanesPerRow;
  float qreg[kEPC];
#pragma unroll
  for (int i = 0; i < kEPC; ++i) qreg[i] = sm.qf[lane_chunk * kEPC + i];

  for (int it = 0; it < n_tiles; ++it) {
    const int st = it % stages;
    mbar_wait(&sm.full[st], (it / stages) & 1, abort_flag, p.status);
    const char *tile = sm.ring + (size_t)st * kTileBytes;
#pragma unroll
    for (int l = 0; l < kLoads; ++l) {
      const int row = warp * kRowsPerWarp + l * kRowsPerLoad + lane_row;
      const uint4 c = *(const uint4 *)(tile + (size_t)row * kRowBytes + lane_chunk * 16);
      float f[kEPC];
      Elem<T>::unpack(c, f);
      float acc = 0.f;
#pragma unroll
      for (int i = 0; i < kEPC; ++i) acc = fmaf(f[i], qreg[i], acc);
#pragma unroll
      for (int o = kLanesPerRow / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      const int j = it * kTileRows + row;
      if (lane_chunk == 0 && j < live_att) sm.z[j] = acc * zscale;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[st]);
  }
  if (e_sub >= 0 && warp == 0) {  // the new token's own score, from k_new directly
    float acc = 0.f;
    for (int c = lane; c < D; c += 32) acc = fmaf(sm.qf[c], sm.knew[c], acc);
    acc = warp_sum(acc);
    if (lane == 0) sm.red[32] = acc * zscale;
  }
  named_bar_sync(kBarConsumers, kConsumers);
  if (e_sub >= 0 && tid == 0) sm.z[e_sub] = sm.red[32];
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
    // statistics of Sec. 4.3: Acc, Acc^square, Count
    sm.s[j] += pj;
    sm.q[j] = fmaf(pj, pj, sm.q[j]);
    sm.n[j] += 1;
  }
  named_bar_sync(kBarConsumers, kConsumers);

  // ---- out = sum_j p_j V[j]
  float acc[kEPC];
#pragma unroll
  for (int i = 0; i < kEPC; ++i) acc[i] = 0.f;
  for (int it = 0; it < n_tiles; ++it) {
    const int g = n_tiles + it;
    const int st = g % stages;
    mbar_wait(&sm.full[st], (g / stages) & 1, abort_flag, p.status);
    const char *tile = sm.ring + (size_t)st * kTileBytes;
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

  if (!evict_first) {
    named_bar_sync(kBarConsumers, kConsumers);  // sm.z (probabilities) no longer needed
    evict_and_insert();
  }

  // ---- write the statistics back; only the freed slot's position changes
  for (int j = tid; j < live_new; j += kConsumers) {
    p.s[unit_st + j] = sm.s[j];
    p.q[unit_st + j] = sm.q[j];
    p.n[unit_st + j] = sm.n[j];
  }
  if (tid == 0) {
    p.pos[unit_st + e] = t_new;
    p.live[u] = live_new;
    p.t_next[u] = t_new + 1;
    p.ev_slot[u] = ev_slot;
    if (p.ev_pos) p.ev_pos[u] = ev_pos;
    if (p.lse) p.lse[u] = (live_att > 0) ? (zmax + log2f(zsum)) * kLn2 : -INFINITY;
  }
}

template <typename T, int D>
static cudaError_t launch_decode_t(const DecodeParams &p, int U, cudaStream_t stream) {
  const size_t smem = decode_smem_bytes(p.B, D, p.stages);
  cudaError_t err = cudaFuncSetAttribute(decode_step_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
  if (err != cudaSuccess) return err;
  decode_step_kernel<T, D><<<U, kDecodeThreads, smem, stream>>>(p);
  return cudaGetLastError();
}

// Ring depth: the deepest ring (3..6 stages of 16 KiB) that still lets the most CTAs share an SM.
static int pick_stages(int B, int d) {
  const size_t per_sm = 227 * 1024;
  for (int ctas = 3; ctas >= 1; --ctas) {
    for (int st = 6; st >= 3; --st)
      if ((decode_smem_bytes(B, d, st) + 1024) * ctas <= per_sm) return st;
  }
  return 0;
}

roco_status launch_decode_step(const roco_cache &c, const void *q, const void *k_new, const void *v_new, int r,
                               int scope_mode, int step_order, float scale, void *out, float *lse, int32_t *ev_slot,
                               int32_t *ev_pos, cudaStream_t stream) {
  DecodeParams p;
  p.K = (const char *)c.K; p.V = (const char *)c.V;
  p.s = c.s; p.q = c.q; p.n = c.n; p.pos = c.pos; p.live = c.live; p.t_next = c.t_next; p.status = c.status;
  p.qv = (const char *)q; p.k_new = (const char *)k_new; p.v_new = (const char *)v_new;
  p.out = (char *)out; p.lse = lse; p.ev_slot = ev_slot; p.ev_pos = ev_pos;
  p.B = c.B; p.r = r; p.scope_mode = scope_mode; p.order = step_order; p.scale = scale;
  p.stages = pick_stages(c.B, c.d);
  if (p.stages == 0) return ROCO_ERR_UNSUPPORTED;
  const int U = c.S * c.G;
  cudaError_t err;
  if (c.kv_dtype == ROCO_BF16 && c.d == 128) err = launch_decode_t<__nv_bfloat16, 128>(p, U, stream);
  else if (c.kv_dtype == ROCO_BF16 && c.d == 64) err = launch_decode_t<__nv_bfloat16, 64>(p, U, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 128) err = launch_decode_t<float, 128>(p, U, stream);
  else if (c.kv_dtype == ROCO_F32 && c.d == 64) err = launch_decode_t<float, 64>(p, U, stream);
  else return ROCO_ERR_UNSUPPORTED;
  return err == cudaSuccess ? ROCO_OK : ROCO_ERR_CUDA;
}

}  // namespace roco
