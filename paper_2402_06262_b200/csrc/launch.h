// Internal launch functions behind the C ABI (one per kernel family).  Arguments are validated by the
// callers in api.cu; these only pick a template instance and enqueue.
#pragma once

#include <cuda_runtime.h>

#include "../../include/roco.h"

namespace roco {

roco_status launch_decode_step(const roco_cache &c, const void *q, const void *k_new, const void *v_new, int r,
                               int scope_mode, int step_order, int policy, const unsigned *rnd, float scale, void *out,
                               float *lse, int32_t *ev_slot, int32_t *ev_pos, cudaStream_t stream);

// The same step (order evict, insert, attend) with each unit's slots divided among `splits` CTAs: three launches,
// partial results and saved scores in `workspace` (decode_split_workspace_bytes).
size_t decode_split_workspace_bytes(int U, int B, int d, int splits);
roco_status launch_decode_step_split(const roco_cache &c, const void *q, const void *k_new, const void *v_new, int r,
                                     int scope_mode, int step_order, int splits, float scale, void *out, float *lse,
                                     int32_t *ev_slot, int32_t *ev_pos, void *workspace, cudaStream_t stream);

// The same step (either order) with a thread-block cluster of `ranks` CTAs (2, 4 or 8) per unit that exchange
// partial results through distributed shared memory; no workspace.  decode_cluster_ranks: the cluster size that
// suits a call of U units (1 = one CTA per unit is the better shape).
int decode_cluster_ranks(int U, int B, int d, int elem, int sms);
roco_status launch_decode_step_cluster(const roco_cache &c, int ranks, const void *q, const void *k_new,
                                       const void *v_new, int r, int scope_mode, int step_order, float scale,
                                       void *out, float *lse, int32_t *ev_slot, int32_t *ev_pos, cudaStream_t stream);

// Row log-sum-exp and column statistics of the causal softmax, CUDA-core path (any supported dtype/d).
// lens_dev: [S] device copy of the prompt lengths.  lse, s_full, q_full: [U][Lmax].
roco_status launch_prefill_stats_simt(int kv_dtype, int d, int S, int G, int Lmax, const int *lens_dev, int maxlen,
                                      const void *Q, const void *K, float scale, float *lse, float *s_full,
                                      float *q_full, cudaStream_t stream);

// Causal attention output of the prompt pass on CUDA cores from the row log-sum-exp (any supported dtype/d):
// out_i = sum_{j<=i} exp(scale Q_i.K_j - lse_i) V_j.  out: [U][Lmax][d], rows >= lens untouched.
roco_status launch_prefill_attend_simt(int kv_dtype, int d, int S, int G, int Lmax, const int *lens_dev, int maxlen,
                                       const void *Q, const void *K, const void *V, float scale, const float *lse,
                                       void *out, cudaStream_t stream);

// The same two passes on tcgen05 tensor cores with TMA-fed operands (bf16, d = 128 only).  lse_ready: `lse`
// already holds the row log-sum-exp (from the one-sweep attention kernel), so only the statistics pass runs.
bool prefill_tc_supported(int kv_dtype, int d);
roco_status launch_prefill_stats_tc(int S, int G, int Lmax, const int *lens_dev, int maxlen, const void *Q,
                                    const void *K, float scale, float *lse, float *s_full, float *q_full, int *status,
                                    cudaStream_t stream, bool lse_ready = false);

// Tensor map (CUtensorMap, 128 bytes, passed as void*) over a [U][Lmax][128] bf16 prompt tensor with boxes of
// 64 columns x 128 rows x 1 unit and the 128-byte swizzle; rows past Lmax read as zero.
bool make_tensor_map_prompt_bf16(void *map, const void *base, int U, int Lmax);

// Causal attention output of the prompt pass on the tensor cores (bf16, d = 128): out_i = sum_{j<=i}
// exp(scale Q_i.K_j - lse_i) V_j.  out: [U][Lmax][128].  With lse_in the row log-sum-exp is taken from there
// (lse_out unused); with lse_in == nullptr one sweep with a running row maximum produces both the output and
// lse_out [U][Lmax] (scale > 0).
roco_status launch_prefill_attend_tc(int S, int G, int Lmax, const int *lens_dev, int maxlen, const void *Q,
                                     const void *K, const void *V, float scale, const float *lse_in, float *lse_out,
                                     void *out, int *status, cudaStream_t stream);

// Select-to-budget on frozen statistics and gather of the survivors into the cache.
// dst: [U][Lmax] int32 scratch (destination slot per token, -1 = evicted).  LOWEST_R with eviction also needs
// sortbuf: [U][Lp2max] 64-bit scratch, Lp2max = Lmax rounded up to a power of two, and r <= budget_lowest_max_r().
int budget_lowest_max_r();
roco_status launch_budget_select_gather(const roco_cache &c, int Lmax, const int *lens_dev, int maxlen, int r,
                                        int scope_mode, const void *K, const void *V, const float *s_full,
                                        const float *q_full, int *dst, unsigned long long *sortbuf, int Lp2max,
                                        cudaStream_t stream);

// Tensor map (CUtensorMap, 128 bytes, passed as void*) over a [rows][128] bf16 matrix with boxes of 64 columns x
// box_rows rows and the 128-byte swizzle; false when the driver entry point is unavailable or the encode fails.
bool make_tensor_map_rows128_bf16(void *map, const void *base, unsigned long long rows, unsigned box_rows);

// Multi-query steps: nb new tokens per unit, each with M / nb query heads (M = nb * group query rows, row
// t * group + g = head g of token t).  Block-wise evict-and-encode: group 1; grouped-query decode: nb 1.
int multi_max_queries();
bool multi_fits(int B, int d, int M, int nb);
roco_status launch_multi_step(const roco_cache &c, int M, int nb, const void *Q, const void *k_new,
                              const void *v_new, int r, int scope_mode, float scale, void *out, float *lse,
                              int32_t *ev_slot, int32_t *ev_pos, cudaStream_t stream, long long unit_stride_rows = 0);
// unit_stride_rows > 0: k_new and v_new are slices of [U][rows][d] tensors with that many rows (tokens) per unit,
// Q and out of [U][rows][group][d] tensors (used to step through a prompt block by block); 0: dense [U][M][d] /
// [U][nb][d].

// Overlap of the budgeted cache's retained positions with the full cache's B most important tokens (one CTA per
// unit; full.B * 8 bytes of shared memory).
roco_status launch_consistency_step(const roco_cache &full, const roco_cache &budgeted, int policy, int32_t *overlap,
                                    float *jaccard_sum, int32_t *samples, cudaStream_t stream);

}  // namespace roco
