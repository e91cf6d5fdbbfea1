/*
 * libroco -- KV-constrained attention with the RoCo eviction policy on one GPU (sm_100a).
 *
 * Notation follows the paper.  A *unit* is one (sequence, layer, head); units are independent
 * (Fig. 1: heads evict at different positions).  d is the head dimension d', B the per-head token
 * budget of Sec. 3 (the cache of a unit never holds more than B tokens), r the eviction-scope
 * parameter of Sec. 4.2/4.3.  Per cached token the library keeps the three B-sized arrays of
 * Sec. 4.3 -- Acc (s), Acc^square (q), Count (n) -- plus the token's original position (pos), which
 * the paper's rule needs once heads have evicted at different positions and which breaks ties.
 *
 *     mean attention score  = s / n                         (Sec. 4.3, "MAS")
 *     variance              = max(0, q / n - (s / n)^2)      (Sec. 4.3, Std formula; sqrt is monotone)
 *     eviction scope        = the m lowest-variance cached tokens, order (variance, position):
 *                             m = live - r  (EXCLUDE_TOP_R, Sec. 4.3: exclude the r highest-Std tokens)
 *                             m = r         (LOWEST_R, Sec. 1 reading: the scope is the r lowest-variance tokens)
 *                             m is clipped to [1, live]
 *     victim                = the in-scope token of lowest mean, order (mean, position)   (Sec. 4.3)
 *
 * Conventions for every entry point
 *   - All array arguments are DEVICE pointers owned by the caller unless the name ends in _host.
 *     The library allocates no device memory, and keeps no state between calls with two exceptions that are
 *     described at their entry points: the built-in scratch array of roco_prefill_static, and the copy stream
 *     with its events that the host-buffer decode calls create per device at first use.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls enqueue work
 *     and return; outputs are valid once the stream reaches that point.  The *_host variants
 *     synchronise the stream before returning.
 *   - Argument errors are detected on the host before anything is launched and reported by the
 *     return value; nothing throws or aborts.  Device-side anomalies (a wait that ran out, a
 *     corrupt `live`) set bits in the caller-owned status word `roco_cache.status` and the kernel
 *     returns normally; read it with roco_device_status().
 *   - Q/K/V element type is roco_cache.kv_dtype (fp32 or bf16); statistics are fp32, counts int32.
 *   - Supported shapes: d in {64, 128}; 1 <= B <= 8192; K, V, Q pointers 16-byte aligned.
 */
#ifndef ROCO_H_
#define ROCO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ROCO_OK = 0,
  ROCO_ERR_INVALID_ARG = 1, /* null/misaligned pointer, r or B out of range, bad lens          */
  ROCO_ERR_UNSUPPORTED = 2, /* d, dtype, B or option outside what the kernels are built for     */
  ROCO_ERR_WORKSPACE = 3,   /* workspace missing or smaller than roco_*_workspace_bytes()       */
  ROCO_ERR_CUDA = 4,        /* a CUDA runtime call failed (launch, copy)                        */
  ROCO_ERR_STATE = 5        /* the device status word is non-zero                               */
} roco_status;

typedef enum { ROCO_F32 = 0, ROCO_BF16 = 1 } roco_dtype;

typedef enum {
  ROCO_SCOPE_EXCLUDE_TOP_R = 0, /* Sec. 4.3: scope = cached tokens minus the r of highest variance  */
  ROCO_SCOPE_LOWEST_R = 1       /* Sec. 1:   scope = the r cached tokens of lowest variance         */
} roco_scope_mode;

typedef enum {
  ROCO_EVICT_FIRST = 0, /* Fig. 1: evict, write the new K/V, then attend (the query sees its own key) */
  ROCO_ATTEND_FIRST = 1 /* attend over the cache, update statistics, then evict and write the new K/V */
} roco_step_order;

/* Bits of the device status word. */
enum {
  ROCO_DEV_WAIT_TIMEOUT = 1, /* a bounded wait on a shared-memory barrier ran out */
  ROCO_DEV_BAD_LIVE = 2,     /* live[u] outside [0, B]                            */
  ROCO_DEV_BAD_VICTIM = 4    /* the selection produced no slot (NaN statistics)   */
};

/* The budgeted cache of Sec. 3/4 for S sequences x G (= layers*heads) units each; U = S*G.
 * Slot order inside a unit is not position order once eviction has happened: pos[] says what a
 * slot holds.  Slots live[u]..B-1 are empty (pos = -1). */
typedef struct {
  int32_t kv_dtype;  /* roco_dtype of K and V                                      */
  int32_t S, G, d, B;
  void *K, *V;       /* [S][G][B][d]                                               */
  float *s, *q;      /* [S][G][B]   Acc and Acc^square                             */
  int32_t *n, *pos;  /* [S][G][B]   Count; original position (-1 = empty slot)     */
  int32_t *live;     /* [S][G]      occupied slots, always <= B                    */
  int32_t *t_next;   /* [S][G]      position the next token of this unit will get  */
  int32_t *status;   /* [1]         device status word, zeroed by the caller       */
} roco_cache;

/* Library version (major*100 + minor). */
int roco_version(void);
const char *roco_status_string(int st);

/* Bytes of device workspace roco_prefill needs for prompts of up to Lmax tokens (host function). */
size_t roco_prefill_workspace_bytes(const roco_cache *cache, int Lmax);

/* The same for ROCO_SCOPE_LOWEST_R when a prompt is longer than the budget: that mode replays the evictions one
 * by one on a sorted order and needs 8 more bytes per token, rounded up to a power of two (host function). */
size_t roco_prefill_workspace_bytes_lowest_r(const roco_cache *cache, int Lmax);

/* 1 if roco_prefill will run the score contraction of Eq. 1 on the tensor cores for this cache's dtype and
 * head dimension (bf16, d = 128; and a positive scale -- zero or negative scales always take the CUDA-core path),
 * 0 if it will use the CUDA-core path (host function). */
int roco_prefill_uses_tensor_cores(const roco_cache *cache);

/*
 * Prefill with eviction to budget (Sec. 4.3 last paragraph; Sec. 5.1 "Other Details": the budget is
 * fixed from the prompt length and eviction happens once, at the prefilling stage).
 *
 * For every unit: causal attention probabilities P (Eq. 1 with the mask of Sec. 2.1: row i sees
 * keys 0..i), without storing P; column statistics n_j = lens - j, s_j = sum_i P_ij,
 * q_j = sum_i P_ij^2 over rows i >= j; then, if lens > B, tokens are evicted down to B by applying
 * the per-step rule lens - B times on these frozen statistics, and the survivors' K, V, s, q, n, pos
 * are written to the cache in increasing position order.  live = min(lens, B); t_next = lens.
 *
 *   Q, K, V        [S][G][Lmax][d], cache->kv_dtype; rows >= lens_host[b] are ignored
 *   lens_host      [S] HOST array, 1 <= lens <= Lmax (all units of a sequence share the length)
 *   B              must equal cache->B;   r: 0 <= r <= B
 *   scope_mode     ROCO_SCOPE_EXCLUDE_TOP_R, or ROCO_SCOPE_LOWEST_R (then, when lens > B: r <= 2048, else
 *                  ROCO_ERR_UNSUPPORTED, and the workspace of roco_prefill_workspace_bytes_lowest_r)
 *   count_self     1: a token's own query counts towards its statistics (0: ROCO_ERR_UNSUPPORTED)
 *   scale          multiplies Q.K (1/sqrt(d) in Eq. 1)
 *   lse_out        [S][G][Lmax] row log-sum-exp, or NULL
 *   s_full, q_full [S][G][Lmax] pre-eviction column statistics, or NULL
 *   workspace      >= roco_prefill_workspace_bytes(cache, Lmax), 256-byte aligned
 */
roco_status roco_prefill(const void *Q, const void *K, const void *V, const int32_t *lens_host, int Lmax,
                         int B, int r, int scope_mode, int count_self, float scale, roco_cache *cache,
                         float *lse_out, float *s_full, float *q_full, void *workspace,
                         size_t workspace_bytes, void *stream);

/*
 * roco_prefill that also returns the prompt's attention output (Eq. 1 with the causal mask of Sec. 2.1), for
 * callers that need the layer's output and not only the budgeted cache:
 *     attn_out_i = sum_{j<=i} softmax_j(scale * Q_i.K_j) V_j,      i < lens
 * The output comes from the same sweep over the score tiles that yields the row log-sum-exp (running row maximum,
 * output accumulator rescaled when the maximum moves), so the whole call costs three L x L contractions (scores
 * and P.V in the sweep, scores again for the column statistics) instead of the four of roco_prefill followed by
 * roco_prefill_attend.  That is the tensor-core path (kv_dtype ROCO_BF16, d = 128, scale > 0); for the other
 * dtypes and head dimensions, and for a scale that is not positive, the output comes from a CUDA-core pass over
 * the row log-sum-exp, after the two statistics passes.
 *   attn_out     [S][G][Lmax][d] device, 16-byte aligned; rows >= lens are left untouched; NULL: roco_prefill
 * All other arguments, results and errors as roco_prefill.
 */
roco_status roco_prefill_with_output(const void *Q, const void *K, const void *V, const int32_t *lens_host, int Lmax,
                                     int B, int r, int scope_mode, int count_self, float scale, roco_cache *cache,
                                     float *lse_out, float *s_full, float *q_full, void *attn_out, void *workspace,
                                     size_t workspace_bytes, void *stream);

/*
 * roco_prefill without a caller-provided workspace.  The paper has no counterpart: this exists for callers
 * that cannot allocate device memory at call time -- code running inside a serving runtime whose memory
 * pool already owns the GPU (cudaMalloc fails there), or a latency-critical loop that must not call
 * cudaMalloc/cudaFree because they synchronise the device.  Same arguments, results and errors as
 * roco_prefill, minus `workspace`; the scratch is an array of ROCO_PREFILL_STATIC_SCRATCH_BYTES built into
 * the library (every GPU that loads the library holds it until the process exits).  The call allocates
 * nothing.
 *   - Limit: roco_prefill_workspace_bytes(cache, Lmax) must not exceed ROCO_PREFILL_STATIC_SCRATCH_BYTES
 *     (S*G*Lmax up to about 524 000 tokens, e.g. 63 units x 8192); larger problems get ROCO_ERR_WORKSPACE.
 *     With ROCO_SCOPE_LOWEST_R and a prompt longer than the budget the need is
 *     roco_prefill_workspace_bytes_lowest_r(cache, Lmax) (8 more bytes per token, Lmax rounded up to a power of
 *     two: about 349 000 tokens), checked the same way.
 *   - The first call on a device looks up the array's device address (with that device current); make that
 *     first call before starting any stream capture on the device.
 *   - All calls on a device share the one array, which keeps the previous call's contents (no buffer in it
 *     needs to start at zero).  Two calls that overlap on the GPU -- different streams, or another host
 *     thread -- race on it: issue them on one stream or order them yourself.
 */
#define ROCO_PREFILL_STATIC_SCRATCH_BYTES (8u << 20)
roco_status roco_prefill_static(const void *Q, const void *K, const void *V, const int32_t *lens_host, int Lmax,
                                int B, int r, int scope_mode, int count_self, float scale, roco_cache *cache,
                                float *lse_out, float *s_full, float *q_full, void *stream);

/*
 * One decode step for every unit (Sec. 3 constrained inference; Sec. 4, fixed-budget buffer: eviction runs
 * once the buffer is full; Sec. 4.3 RoCo rule; Fig. 1 ordering).
 *
 * EVICT_FIRST: if live == B the victim's slot is freed, else slot `live` is taken; the new token's
 * K/V are written there with empty statistics and pos = t_next; the query attends over all occupied
 * slots (Eq. 1); every occupied slot gets n += 1, s += p, q += p^2.  ATTEND_FIRST: attention and the
 * statistics update run over the cache as it stands, then the eviction and the in-place write.
 * The cache is never compacted: only the freed slot is overwritten.
 * One launch.  Its shape follows the call's size: one CTA per unit when the units fill the GPU, a cluster of
 * 2, 4 or 8 CTAs per unit when they are few (roco_decode_step_cluster with ranks = 0, below).
 *
 *   q, k_new, v_new  [S][G][d], cache->kv_dtype
 *   r                EXCLUDE_TOP_R: 0 <= r < B;  LOWEST_R: 1 <= r <= B
 *   attn_out         [S][G][d], cache->kv_dtype
 *   lse_out          [S][G] fp32 log-sum-exp of the scaled scores, or NULL
 *   evicted_slot     [S][G] int32, -1 where nothing was evicted
 *   evicted_pos      [S][G] int32 original position of the evicted token (-1 if none), or NULL
 */
roco_status roco_decode_step(roco_cache *cache, const void *q, const void *k_new, const void *v_new, int r,
                             int scope_mode, int step_order, float scale, void *attn_out, float *lse_out,
                             int32_t *evicted_slot, int32_t *evicted_pos, void *stream);

/* The eviction policies of Table 1 (importance score of Sec. 4.1 + eviction scope of Sec. 4.2 / 4.3). */
typedef enum {
  ROCO_POLICY_ROCO = 0,         /* mean attention score + standard-deviation scope (EXCLUDE_TOP_R)            */
  ROCO_POLICY_RANDOM = 1,       /* a random cached pair: victim slot = rnd[unit] mod B                        */
  ROCO_POLICY_RECENCY = 2,      /* the farthest token (lowest position)                                       */
  ROCO_POLICY_STREAMLLM = 3,    /* the first token after the 4 initial attention-sink tokens                  */
  ROCO_POLICY_SCISSORHANDS = 4, /* lowest accumulated quantised score outside the local window of size r      */
  ROCO_POLICY_H2O = 5,          /* lowest accumulated attention score outside the local window of size r      */
  ROCO_POLICY_TOVA = 6,         /* lowest attention score from the last query                                 */
  ROCO_POLICY_MAS_WINDOW = 7    /* lowest mean attention score outside the local window (Sec. 4.3 experiment) */
} roco_policy;

/*
 * roco_decode_step (order ROCO_EVICT_FIRST) under any policy of Table 1, on the same cache layout.
 * The local window of Sec. 4.2 is the r most recent positions: a cached token is evictable if pos < t_next - r.
 * Ties go to the lowest position.  s and n are Acc and Count for every policy; the q array holds Acc^square,
 * except under ROCO_POLICY_SCISSORHANDS (accumulated quantised score: +1 when the token's probability exceeds
 * the average 1/live of the step) and under ROCO_POLICY_TOVA (the last query's probability) -- so a cache should
 * be stepped with one policy throughout.
 *   rnd   [S][G] uint32 device array of random draws, read only by ROCO_POLICY_RANDOM (else may be NULL)
 *   r     0 <= r < B: scope parameter of ROCO_POLICY_ROCO, window size of the windowed policies, else ignored
 */
roco_status roco_decode_step_policy(roco_cache *cache, const void *q, const void *k_new, const void *v_new,
                                    int policy, int r, const uint32_t *rnd, float scale, void *attn_out,
                                    float *lse_out, int32_t *evicted_slot, int32_t *evicted_pos, void *stream);
/* The same in either order of a step (roco_step_order): under ROCO_ATTEND_FIRST the query attends over the cache as
 * it stands, the policy's statistics are updated, and the eviction is decided on the updated statistics (the last
 * score of ROCO_POLICY_TOVA is then this step's own query's). */
roco_status roco_decode_step_policy_ordered(roco_cache *cache, const void *q, const void *k_new, const void *v_new,
                                            int policy, int r, int step_order, const uint32_t *rnd, float scale,
                                            void *attn_out, float *lse_out, int32_t *evicted_slot,
                                            int32_t *evicted_pos, void *stream);

/*
 * Block-wise evict-and-encode (Sec. 5.3 "Overhead", App. B, where one eviction step frees and encodes a block of
 * b tokens): b new tokens per unit in one pass over the cache.
 *   1. live + b - B tokens (if positive) leave: the rule of Sec. 4.3 applied that many times on the statistics as
 *      they stand (frozen), each time on the tokens still cached.
 *   2. The new tokens (positions t_next .. t_next + b - 1) take, in order, the freed slots and -- while the buffer
 *      is not full -- slots live, live + 1, ..., all in increasing slot order.
 *   3. Query i attends over the remaining old tokens and the new tokens 0..i (causal inside the block); every
 *      attended token gets Count += 1, Acc += p, Acc^square += p^2.
 * b = 1 is roco_decode_step with ROCO_EVICT_FIRST.
 *
 *   Q, K_new, V_new  [S][G][b][d], cache->kv_dtype
 *   b                1..16, r + b <= B.  Under ROCO_SCOPE_LOWEST_R the scope refills after each of the step's
 *                    evictions (the token next in (variance, position) order is admitted before the next victim
 *                    is taken), all on the statistics as they stand before the step;
 *                    the step's working set must fit on an SM, else ROCO_ERR_UNSUPPORTED: for bf16, d = 128 and
 *                    scale > 0: B <= 4096 (scores in tensor memory), otherwise b * B floats of scores in shared
 *                    memory
 *   attn_out         [S][G][b][d];   lse_out [S][G][b] or NULL
 *   evicted_slot     [S][G][b] freed slots in increasing order, padded with -1;  evicted_pos likewise, or NULL
 */
roco_status roco_block_step(roco_cache *cache, const void *Q, const void *K_new, const void *V_new, int b, int r,
                            int scope_mode, float scale, void *attn_out, float *lse_out, int32_t *evicted_slot,
                            int32_t *evicted_pos, void *stream);

/*
 * Key-value constrained prompt encoding, block by block (Sec. 5.3 "Overhead": evict-and-encode "in a block-wise
 * manner"; b = 1 is the token-wise scheme of the prior policies): the prompt of every sequence is fed through
 * roco_block_step b tokens at a time (the last block may be shorter), so the cache never exceeds the budget while
 * the prompt is encoded.  The cache is continued from its current state: start from live = 0, t_next = 0 for a
 * fresh prompt.  Unlike roco_prefill no L x L work is done: each block attends over at most B cached tokens.
 *
 *   Q, K, V        [S][G][Lmax][d], cache->kv_dtype; rows >= lens_host[b] are ignored
 *   lens_host      [S] HOST array, 1 <= lens <= Lmax
 *   b              block size 1..16; r as for roco_block_step (EXCLUDE_TOP_R reading, r + b <= B)
 *   attn_out       [S][G][Lmax][d] attention output of every prompt token over the budgeted cache
 *   evicted_slot   [S][G][b] scratch; on return the slots the last block of each sequence freed (-1 padded)
 * Launches ceil(len / b) kernels per run of consecutive sequences of equal length (one launch advances the whole
 * run by a block), so a batch of equal-length prompts costs ceil(len / b) launches in all.
 */
roco_status roco_prefill_blockwise(const void *Q, const void *K, const void *V, const int32_t *lens_host, int Lmax,
                                   int b, int r, float scale, roco_cache *cache, void *attn_out,
                                   int32_t *evicted_slot, void *stream);

/*
 * Attention output of the one-pass prompt encoding (Eq. 1 with the causal mask of Sec. 2.1), for callers that
 * also need the layer's output and not only the budgeted cache:
 *     out_i = sum_{j<=i} exp(scale * Q_i.K_j - lse_i) V_j,      i < lens
 * where lse is the row log-sum-exp roco_prefill returned in lse_out for the same Q, K, lens, Lmax and scale
 * (call roco_prefill first, on the same stream).  On the tensor cores for kv_dtype ROCO_BF16 and d = 128, on the
 * CUDA cores otherwise.  Only S, G, d, kv_dtype and status of `cache` are read.
 *
 *   Q, K, V      [S][G][Lmax][d] device; rows >= lens may hold anything
 *   lens_host    [S] HOST array, 1 <= lens <= Lmax
 *   lse          [S][G][Lmax] fp32 device
 *   attn_out     [S][G][Lmax][d] device, cache->kv_dtype; rows >= lens are left untouched
 *   workspace    >= roco_prefill_attend_workspace_bytes(cache) device bytes, 256-byte aligned
 */
size_t roco_prefill_attend_workspace_bytes(const roco_cache *cache);
roco_status roco_prefill_attend(const roco_cache *cache, const void *Q, const void *K, const void *V,
                                const int32_t *lens_host, int Lmax, float scale, const float *lse, void *attn_out,
                                void *workspace, size_t workspace_bytes, void *stream);

/*
 * Block-wise evict-and-encode on a grouped-query model (Sec. 5.3 "Extension to Grouped-Query Attention", App. A;
 * App. B / Table 9 run block-wise eviction on such a model): the cache belongs to a key-value head that `group`
 * query heads share.  Steps 1 and 2 as roco_block_step.  Step 3: for token i of the block each of its query heads
 * attends over the remaining old tokens and the new tokens 0..i; the statistics receive, once per token of the
 * block, the group-wise averaged probability: Count += 1, Acc += pbar_i, Acc^square += pbar_i^2.
 * group = 1 is roco_block_step; b = 1 is roco_gqa_decode_step.
 *
 *   Q            [S][G][b][group][d];   K_new, V_new [S][G][b][d]
 *   b, group     b * group <= 16 query rows per pass; other limits as roco_block_step
 *   attn_out     [S][G][b][group][d];   lse_out [S][G][b][group] or NULL;   evicted_slot, evicted_pos [S][G][b]
 *
 * roco_prefill_blockwise_gqa is roco_prefill_blockwise for such a model: Q and attn_out are
 * [S][G][Lmax][group][d], K and V [S][G][Lmax][d].
 */
roco_status roco_gqa_block_step(roco_cache *cache, const void *Q, const void *K_new, const void *V_new, int b,
                                int group, int r, int scope_mode, float scale, void *attn_out, float *lse_out,
                                int32_t *evicted_slot, int32_t *evicted_pos, void *stream);
roco_status roco_prefill_blockwise_gqa(const void *Q, const void *K, const void *V, const int32_t *lens_host,
                                       int Lmax, int b, int group, int r, float scale, roco_cache *cache,
                                       void *attn_out, int32_t *evicted_slot, void *stream);

/*
 * Decode step for grouped-query attention (Sec. 5.3 "Extension to Grouped-Query Attention", App. A): the cache
 * belongs to a key-value head that `group` query heads share.  Order as ROCO_EVICT_FIRST.  Each query head g
 * attends over the same cache, out_g = Softmax(scale * q_g K^T) V; the statistics receive the group-wise
 * averaged probability pbar = (1/group) sum_g p_g: Count += 1, Acc += pbar, Acc^square += pbar^2.
 *
 *   Q            [S][G][group][d]  (G counts key-value heads);  k_new, v_new [S][G][d]
 *   group        1..16 (the working set must fit on an SM as for roco_block_step, with group query rows)
 *   attn_out     [S][G][group][d];  lse_out [S][G][group] or NULL;  evicted_slot, evicted_pos [S][G]
 */
roco_status roco_gqa_decode_step(roco_cache *cache, const void *Q, const void *k_new, const void *v_new, int group,
                                 int r, int scope_mode, float scale, void *attn_out, float *lse_out,
                                 int32_t *evicted_slot, int32_t *evicted_pos, void *stream);

/*
 * roco_decode_step (order ROCO_EVICT_FIRST) for calls with few units -- one layer of a small batch -- where one
 * CTA per unit cannot fill the GPU: each unit's slots are divided among `splits` CTAs (Eq. 1 is merged from the
 * partial (max, sum, sum of p*V) triples; the statistics of Sec. 4.3 are then accumulated in a second, cheap pass
 * from the saved scores and the merged log-sum-exp).  Same arguments and results as roco_decode_step.
 *   splits      1..64 CTAs per unit (a good value makes S*G*splits a few times the number of SMs)
 *   workspace   >= roco_decode_split_workspace_bytes(cache, splits), 256-byte aligned, device; S*G <= 65535
 */
size_t roco_decode_split_workspace_bytes(const roco_cache *cache, int splits);
roco_status roco_decode_step_split(roco_cache *cache, const void *q, const void *k_new, const void *v_new, int r,
                                   int scope_mode, int splits, float scale, void *attn_out, float *lse_out,
                                   int32_t *evicted_slot, int32_t *evicted_pos, void *workspace,
                                   size_t workspace_bytes, void *stream);
/* The same in either order of a step (roco_step_order): under ROCO_ATTEND_FIRST the attention and merge launches
 * run first, over the cache as it stands, and the selection launch last, on the updated statistics. */
roco_status roco_decode_step_split_ordered(roco_cache *cache, const void *q, const void *k_new, const void *v_new,
                                           int r, int scope_mode, int step_order, int splits, float scale,
                                           void *attn_out, float *lse_out, int32_t *evicted_slot,
                                           int32_t *evicted_pos, void *workspace, size_t workspace_bytes,
                                           void *stream);

/*
 * roco_decode_step (either step order, both scope readings) for calls with few units -- one layer of a small
 * batch, a few long sequences -- with a thread-block cluster of `ranks` CTAs per unit: every rank streams the K/V
 * rows of its own slot range exactly once and keeps that range's scores and statistics; the ranks agree on the
 * softmax maximum and denominator of Eq. 1, on the eviction scope and on the victim (Sec. 4.3; a radix select and
 * an argmin that run on all ranks in lockstep) by exchanging a few words through distributed shared memory, the
 * partial outputs are added up on the first rank, the rank that owns the freed slot overwrites it in place
 * (Fig. 1), and each rank updates the statistics of its own slots.  One launch, no workspace, no global-memory
 * traffic besides what roco_decode_step has.  Same arguments, results and parity bounds as roco_decode_step.
 *
 *   ranks   2, 4 or 8 CTAs per unit; 1: the one-CTA-per-unit kernel; 0: roco_decode_cluster_ranks(cache), which is
 *           what roco_decode_step does
 * Needs B a multiple of 4 and 16-byte aligned statistics arrays (else ROCO_ERR_UNSUPPORTED for ranks > 1).
 * roco_decode_cluster_ranks: the cluster size that suits this cache's shape on the current device -- the
 * largest whose CTAs fit the GPU in one wave of two per SM while every rank keeps at least two 16 KiB tiles;
 * 1 when one CTA per unit already fills the GPU (host function; 0 on error).
 */
int roco_decode_cluster_ranks(const roco_cache *cache);
roco_status roco_decode_step_cluster(roco_cache *cache, const void *q, const void *k_new, const void *v_new, int r,
                                     int scope_mode, int step_order, int ranks, float scale, void *attn_out,
                                     float *lse_out, int32_t *evicted_slot, int32_t *evicted_pos, void *stream);


/*
 * Consistency of an importance score under a budget with its full-cache version (Sec. 4.3, preliminary
 * experiments, set-up): `full` and `budgeted` are two caches of the same units that have been fed the same tokens
 * with roco_decode_step_policy under `policy`, `full` with a budget large enough never to evict.  For every unit
 * the call finds the B = budgeted->live[u] most important tokens of the full cache by the policy's own score
 * (accumulated score for ROCO_POLICY_H2O, accumulated quantised score for ROCO_POLICY_SCISSORHANDS, last score for
 * ROCO_POLICY_TOVA, mean attention score for ROCO_POLICY_MAS_WINDOW and ROCO_POLICY_ROCO) -- the tokens left when
 * the policy's eviction order (score asc, position asc) has removed the rest -- and counts how many of them the
 * budgeted cache retains.  Both sets have B tokens, so the Jaccard similarity is overlap / (2B - overlap).
 *
 *   overlap      [S][G] int32: the count of this call (-1 for a unit whose full cache holds fewer than B tokens)
 *   jaccard_sum  [S][G] fp32, samples [S][G] int32: running sum of the similarity and number of calls that
 *                added to it (zero both before the first call; mean similarity = sum / samples)
 *   full->B <= 8192; full and budgeted have the same S and G; device anomalies go to budgeted->status.
 */
roco_status roco_consistency_step(const roco_cache *full, const roco_cache *budgeted, int policy, int32_t *overlap,
                                  float *jaccard_sum, int32_t *samples, void *stream);

/* Bytes of device staging roco_decode_step_host needs (host function). */
size_t roco_decode_host_staging_bytes(const roco_cache *cache);

/*
 * The same step for callers whose per-step tensors live in (pinned) HOST memory: copies q, k_new,
 * v_new to `staging`, runs roco_decode_step, copies attn_out / evicted_slot / evicted_pos back and
 * synchronises the stream.  The cache stays on the device.  *_host arguments are host pointers with
 * the shapes above; evicted_pos_host may be NULL.  staging: device,
 * >= roco_decode_host_staging_bytes(cache), 256-byte aligned.
 * With 2048 units or more the step is cut into four unit ranges (units are independent) and the copies of one
 * range overlap the kernel of another: the copies then run on a copy stream that the library creates, with a
 * handful of events, at the first such call on a device and keeps until the process exits -- the one piece of
 * state besides the scratch of roco_prefill_static.  Host buffers must be pinned for the overlap to happen.
 * Large calls on one device share those events, so they must not be issued from several host threads at once.
 */
roco_status roco_decode_step_host(roco_cache *cache, const void *q_host, const void *k_new_host,
                                  const void *v_new_host, int r, int scope_mode, int step_order, float scale,
                                  void *attn_out_host, int32_t *evicted_slot_host, int32_t *evicted_pos_host,
                                  void *staging, size_t staging_bytes, void *stream);

/*
 * The host-buffer step in two halves, so that the copies of one step run under the kernel of another: _begin
 * enqueues the input copies (on an input stream of the library), the step's kernel (on `stream`) and the result
 * copies (on an output stream) and returns without waiting; _end blocks the calling host thread until the oldest
 * begun step's results are in its host buffers.  Up to two steps may be in flight: begin(t), begin(t + 1),
 * end() [t is done], begin(t + 2), ...  A third _begin without an _end returns ROCO_ERR_STATE, as does an _end
 * with nothing in flight.  Steps of one cache must be begun on one stream (they are ordered by it); the host
 * buffers of a step must stay valid and untouched until its _end, and be pinned for the copies to overlap.
 * Arguments as roco_decode_step_host; staging >= roco_decode_host_pipeline_staging_bytes(cache) (two sets),
 * 256-byte aligned.  The two copy streams and six events are created per device at the first call and kept (see
 * roco_decode_step_host); the in-flight count is per device, so one host thread drives one pipeline per device.
 */
size_t roco_decode_host_pipeline_staging_bytes(const roco_cache *cache);
roco_status roco_decode_step_host_begin(roco_cache *cache, const void *q_host, const void *k_new_host,
                                        const void *v_new_host, int r, int scope_mode, int step_order, float scale,
                                        void *attn_out_host, int32_t *evicted_slot_host, int32_t *evicted_pos_host,
                                        void *staging, size_t staging_bytes, void *stream);
roco_status roco_decode_step_host_end(void);

/*
 * Self-test of the bounded waits (the paper has no counterpart: this checks the library's own failure reporting).
 * Every kernel here waits on shared-memory barriers with a time limit of about two seconds; a wait that runs out
 * sets ROCO_DEV_WAIT_TIMEOUT in the status word and the kernel carries on to its end instead of hanging.  This
 * call launches one small CTA that waits on a barrier nothing completes, so that limit is reached on purpose:
 * afterwards *status has ROCO_DEV_WAIT_TIMEOUT set and *waited_ms (device, may be NULL) holds how long the wait
 * took.  The kernel occupies one SM for that time and touches no other memory.
 */
roco_status roco_selftest_wait_timeout(int32_t *status, int32_t *waited_ms, void *stream);

/*
 * Measurement aid (the paper has no counterpart): one launch that reads `bytes` bytes (16-byte aligned buffer,
 * a multiple of 16 is read) with plain 16-byte loads and adds a checksum to *sink (device, may be NULL).  Timed
 * by the caller, it gives the read-only streaming rate of the device, the ceiling for the read-dominated decode
 * step; a copy (half reads, half writes) runs below it.
 */
roco_status roco_selftest_read_stream(const void *buf, size_t bytes, unsigned long long *sink, void *stream);

/* Copies the device status word to *flags_host (synchronises the stream).  Returns ROCO_ERR_STATE
 * when it is non-zero. */
roco_status roco_device_status(const roco_cache *cache, void *stream, int32_t *flags_host);

#ifdef __cplusplus
}
#endif
#endif /* ROCO_H_ */
