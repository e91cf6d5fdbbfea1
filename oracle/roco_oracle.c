/*
 * CPU oracle for KV-constrained inference with the RoCo eviction policy.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of the
 * paper's definitions that the CUDA library is checked against.  It shares no
 * code with the CUDA path and must never be called from it: only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Everything is fp64.  Inputs are the exact fp32/bf16 input values widened to
 * double by the caller.  One "unit" = one (sequence, layer, head); units are
 * independent (Fig. 1: heads evict at different positions), and the only
 * parallelism here is an OpenMP loop over units in the *_batch drivers.
 *
 * What each function follows:
 *   softmax / attention ............ Eq. 1 (scaled dot-product attention, one head)
 *   causal prefill ................. Sec. 2.1 "Key-Value Cache": a token sees itself and earlier tokens
 *   Acc, Acc^square, Count ......... Sec. 4.3: three B-sized arrays per head
 *   mean attention score (MAS) ..... Sec. 4.3: Acc / Count
 *   Std ............................ Sec. 4.3: sqrt(Acc^square/Count - (Acc/Count)^2); ranking uses the
 *                                    variance (sqrt is monotone), population form (divide by Count)
 *   eviction scope ................. Sec. 4.3: exclude the r tokens of highest Std (EXCLUDE_TOP_R);
 *                                    Sec. 1 describes the scope as the low-variance tokens, read as the r lowest
 *                                    (LOWEST_R).  Both are "the m lowest-variance tokens" with
 *                                    m = live - r or m = r.
 *   victim ......................... Sec. 4.3: the in-scope token of lowest mean attention score
 *   fixed buffer, evict when full .. Sec. 3 (n <= B at every step), Sec. 4 first paragraph
 *   evict before appending ......... Fig. 1 caption (EVICT_FIRST step order)
 *   prefill-stage eviction to B .... Sec. 4.3 last paragraph / Sec. 5.1 "Other Details" (B = len x rate)
 *   block-wise evict-and-encode .... Sec. 5.3 "Overhead", App. B (b tokens freed and encoded per eviction step)
 *   grouped-query attention ........ Sec. 5.3 / App. A (group-wise averaged attention score updates the statistics)
 *   other policies ................. Table 1 with Sec. 4.1 (importance scores), Sec. 4.2 (local window), Sec. 5.1
 *   consistency diagnostic ......... Sec. 4.3 "Preliminary Experiments", set-up (top-B of a full cache against the
 *                                    tokens a budgeted cache retains; Jaccard similarity)
 *   margin analysis ................ the parity rule only (not in the paper): which victims are admissible when the
 *                                    statistics carry a relative error, and a select-to-budget replay guided by
 *                                    another implementation's survivor set
 *
 * Readings where the paper is silent (stated once here, in words):
 *   - ties: scope membership by (variance asc, position asc); victim by (mean asc, position asc);
 *   - a token's own query counts (count_self = 1) unless asked otherwise; with count_self = 0 tokens
 *     whose Count is still 0 are not evictable;
 *   - statistics are raw accumulations: no reset or renormalisation after an eviction;
 *   - a freed slot is overwritten in place; while the buffer is not full the new token goes to slot
 *     `live`; after prefill the survivors sit in increasing position order;
 *   - select-to-budget at prefill = the per-step rule applied L-B times on frozen statistics;
 *   - a block step frees its slots the same way (rule applied on frozen statistics), the b new tokens take the
 *     freed / free slots in increasing slot order, and attention inside the block is causal;
 *   - grouped queries: the probabilities are averaged over the group first, then the mean enters Acc and its
 *     square Acc^square, with one Count per step.
 *
 * Parity pins: every function here is pinned by tests that do not call it to produce their expected
 * values (hand-worked rationals, harmonic-number closed forms, library softmax/logsumexp, brute-force
 * history recomputation, invariants).  No function is "parity unpinned".
 */
#include <float.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ROCO_ORACLE_EXCLUDE_TOP_R = 0, ROCO_ORACLE_LOWEST_R = 1 };
enum { ROCO_ORACLE_EVICT_FIRST = 0, ROCO_ORACLE_ATTEND_FIRST = 1 };

int roco_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ---------------------------------------------------------------- Eq. 1 -- */

/* p = Softmax(scale * qv . K[j]) over j = 0..count-1, with max subtraction.
 * Returns log-sum-exp of the scaled scores (-inf when count == 0). */
static double softmax_row(const double *qv, const double *K, int count, int d, double scale, double *p) {
  if (count <= 0) return -INFINITY;
  double zmax = -INFINITY;
  for (int j = 0; j < count; ++j) {
    double z = 0.0;
    for (int c = 0; c < d; ++c) z += qv[c] * K[(size_t)j * d + c];
    z *= scale;
    p[j] = z;
    if (z > zmax) zmax = z;
  }
  double Z = 0.0;
  for (int j = 0; j < count; ++j) {
    p[j] = exp(p[j] - zmax);
    Z += p[j];
  }
  for (int j = 0; j < count; ++j) p[j] /= Z;
  return zmax + log(Z);
}

/* Eq. 1 for one query over `count` keys: probabilities p[count]; returns the log-sum-exp of the scaled scores. */
double roco_oracle_attention_row(const double *qv, const double *K, int count, int d, double scale, double *p) {
  return softmax_row(qv, K, count, d, scale, p);
}

/* Causal prefill statistics of one unit (Eq. 1 with the causal mask; Sec. 4.3 arrays).
 * Q, K: [L][d].  lse: [L] (may be NULL).  s, q: [L] doubles; n: [L] ints.
 * P_out: [L][L] row-major full probability matrix (may be NULL; zeros above the diagonal). */
void roco_oracle_prefill_stats(const double *Q, const double *K, int L, int d, double scale, int count_self,
                               double *lse, double *s, double *q, int *n, double *P_out) {
  double *p = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
  for (int j = 0; j < L; ++j) { s[j] = 0.0; q[j] = 0.0; n[j] = 0; }
  if (P_out) memset(P_out, 0, sizeof(double) * (size_t)L * L);
  for (int i = 0; i < L; ++i) {
    double l = softmax_row(Q + (size_t)i * d, K, i + 1, d, scale, p);   /* row i sees keys 0..i */
    if (lse) lse[i] = l;
    for (int j = 0; j <= i; ++j) {
      if (P_out) P_out[(size_t)i * L + j] = p[j];
      if (j == i && !count_self) continue;
      s[j] += p[j];
      q[j] += p[j] * p[j];
      n[j] += 1;
    }
  }
  free(p);
}

/* ------------------------------------------------- scope and victim (4.3) -- */

typedef struct {
  double var, mean, ab; /* ab = Acc^square/Count + mean^2: the uncancelled magnitude of the variance */
  int pos, slot;
} cand_t;

static int cmp_var_pos(const void *a, const void *b) {
  const cand_t *x = (const cand_t *)a, *y = (const cand_t *)b;
  if (x->var < y->var) return -1;
  if (x->var > y->var) return 1;
  return (x->pos > y->pos) - (x->pos < y->pos);
}

static int before_mean_pos(const cand_t *x, const cand_t *y) {
  if (x->mean < y->mean) return 1;
  if (x->mean > y->mean) return 0;
  return x->pos < y->pos;
}

/* Victim among slots 0..live-1.  Returns the slot; *near_tie is set when the decision margin is
 * below delta (relative): the runner-up's mean is within delta*(sum of the two means); or the victim,
 * or a lower-mean outsider, sits within delta*(uncancelled variance terms) of the scope boundary.
 * *scope_size receives m. */
int roco_oracle_select(const double *s, const double *q, const int *n, const int *pos, int live, int r,
                       int mode, double delta, int *near_tie, int *scope_size) {
  if (near_tie) *near_tie = 0;
  if (scope_size) *scope_size = 0;
  if (live <= 0) return -1;
  cand_t *c = (cand_t *)malloc(sizeof(cand_t) * (size_t)live);
  int nc = 0;
  for (int j = 0; j < live; ++j) {
    if (n[j] <= 0) continue; /* never attended yet (count_self = 0 only): not evictable */
    double mean = s[j] / n[j];
    double a = q[j] / n[j];
    double var = a - mean * mean;
    if (var < 0.0) var = 0.0;
    c[nc].mean = mean; c[nc].var = var; c[nc].ab = a + mean * mean;
    c[nc].pos = pos[j]; c[nc].slot = j;
    ++nc;
  }
  if (nc == 0) { /* nothing has statistics: fall back to the oldest token */
    int best = 0;
    for (int j = 1; j < live; ++j) if (pos[j] < pos[best]) best = j;
    free(c);
    return best;
  }
  qsort(c, (size_t)nc, sizeof(cand_t), cmp_var_pos);
  int m = (mode == ROCO_ORACLE_EXCLUDE_TOP_R) ? nc - r : r;
  if (m < 1) m = 1;
  if (m > nc) m = nc;
  if (scope_size) *scope_size = m;
  int v = 0;
  for (int k = 1; k < m; ++k) if (before_mean_pos(&c[k], &c[v])) v = k;
  if (near_tie) {
    int near = 0;
    /* (i) runner-up in scope */
    int u = -1;
    for (int k = 0; k < m; ++k) {
      if (k == v) continue;
      if (u < 0 || before_mean_pos(&c[k], &c[u])) u = k;
    }
    if (u >= 0 && c[u].mean - c[v].mean <= delta * (c[u].mean + c[v].mean)) near = 1;
    if (m < nc) {
      /* (ii) the victim could drop out of the scope */
      double lo_out = INFINITY; /* lowest reachable variance of any outsider */
      for (int k = m; k < nc; ++k) {
        double t = c[k].var - delta * c[k].ab;
        if (t < lo_out) lo_out = t;
      }
      if (lo_out <= c[v].var + delta * c[v].ab) near = 1;
      /* (iii) an outsider that would win on mean could enter the scope */
      double hi_in = -INFINITY; /* highest reachable variance of any insider */
      for (int k = 0; k < m; ++k) {
        double t = c[k].var + delta * c[k].ab;
        if (t > hi_in) hi_in = t;
      }
      for (int k = m; k < nc && !near; ++k) {
        if (c[k].mean <= c[v].mean + delta * (c[k].mean + c[v].mean) && c[k].var - delta * c[k].ab <= hi_in)
          near = 1;
      }
    }
    *near_tie = near;
  }
  int slot = c[v].slot;
  free(c);
  return slot;
}

/* Select-to-budget, literal form: apply the per-step rule L-B times on frozen statistics, removing the
 * victim each time.  keep[j] = 1 for survivors.  Works for both scope modes.  Returns how many of the
 * iterations were near-ties at relative margin delta (after one, later iterations may legitimately differ). */
int roco_oracle_select_to_budget_iterated(const double *s, const double *q, const int *n, int L, int B, int r,
                                          int mode, double delta, int *keep) {
  int n_near = 0;
  for (int j = 0; j < L; ++j) keep[j] = 1;
  if (L <= B) return 0;
  double *cs = (double *)malloc(sizeof(double) * (size_t)L), *cq = (double *)malloc(sizeof(double) * (size_t)L);
  int *cn = (int *)malloc(sizeof(int) * (size_t)L), *cp = (int *)malloc(sizeof(int) * (size_t)L);
  for (int alive = L; alive > B; --alive) {
    int k = 0;
    for (int j = 0; j < L; ++j)
      if (keep[j]) { cs[k] = s[j]; cq[k] = q[j]; cn[k] = n[j]; cp[k] = j; ++k; }
    int near = 0;
    int slot = roco_oracle_select(cs, cq, cn, cp, alive, r, mode, delta, &near, NULL);
    n_near += near;
    keep[cp[slot]] = 0;
  }
  free(cs); free(cq); free(cn); free(cp);
  return n_near;
}

/* Which tokens could be the victim if every statistic were off by at most the relative margin delta?
 * With var_j known only to +-delta*(Acc^square/Count + mean^2) (the uncancelled terms, as in roco_oracle_select)
 * and mean_j to +-delta*mean_j, token u is *admissible* when (a) it may lie in the scope: fewer than m tokens come
 * certainly before it in (variance, position) order, and (b) no token that lies in the scope whatever the errors
 * has a certainly lower mean.  Both conditions are necessary for u to be the rule's choice (Sec. 4.3) under some
 * error within the margin, so adm[] holds every such choice (and, for delta = 0, the choice alone).  "Certainly
 * before" between two exactly known, equal values falls to the position, like the rule's own ties.
 * adm: [live] 0/1.  Tokens with Count = 0 are never admissible (they are not evictable). */
void roco_oracle_admissible_victims(const double *s, const double *q, const int *n, const int *pos, int live, int r,
                                    int mode, double delta, int *adm) {
  double *vlo = (double *)malloc(sizeof(double) * (size_t)(live > 0 ? live : 1) * 4);
  double *vhi = vlo + live, *mlo = vhi + live, *mhi = mlo + live;
  int nc = 0;
  for (int j = 0; j < live; ++j) {
    adm[j] = 0;
    if (n[j] <= 0) { vlo[j] = vhi[j] = mlo[j] = mhi[j] = NAN; continue; }
    double mean = s[j] / n[j], a = q[j] / n[j];
    double var = a - mean * mean;
    if (var < 0.0) var = 0.0;
    double ev = delta * (a + mean * mean), em = delta * mean;
    vlo[j] = var - ev; vhi[j] = var + ev; mlo[j] = mean - em; mhi[j] = mean + em;
    ++nc;
  }
  if (nc == 0) { free(vlo); return; }
  int m = (mode == ROCO_ORACLE_EXCLUDE_TOP_R) ? nc - r : r;
  if (m < 1) m = 1;
  if (m > nc) m = nc;
#define CERTAINLY_BEFORE(lo, hi, k, u) \
  ((hi)[k] < (lo)[u] || ((hi)[k] == (lo)[u] && (lo)[k] == (hi)[k] && (lo)[u] == (hi)[u] && pos[k] < pos[u]))
  int *sure = (int *)malloc(sizeof(int) * (size_t)live); /* in the scope whatever the errors */
  for (int k = 0; k < live; ++k) {
    sure[k] = 0;
    if (n[k] <= 0) continue;
    int maybe_before = 0; /* tokens that are not certainly after k */
    for (int j = 0; j < live; ++j)
      if (j != k && n[j] > 0 && !CERTAINLY_BEFORE(vlo, vhi, k, j)) ++maybe_before;
    sure[k] = maybe_before < m;
  }
  for (int u = 0; u < live; ++u) {
    if (n[u] <= 0) continue;
    int before = 0;
    for (int k = 0; k < live; ++k)
      if (k != u && n[k] > 0 && CERTAINLY_BEFORE(vlo, vhi, k, u)) ++before;
    if (before >= m) continue; /* (a) fails */
    int beaten = 0;
    for (int k = 0; k < live && !beaten; ++k)
      if (k != u && sure[k] && CERTAINLY_BEFORE(mlo, mhi, k, u)) beaten = 1;
    adm[u] = !beaten;
  }
#undef CERTAINLY_BEFORE
  free(sure); free(vlo);
}

/* Select-to-budget (iterated form) replayed next to another implementation's survivor set guide_keep[L]: at every
 * iteration the rule's own victim is taken if the guide evicted it too; otherwise the iteration must be a decision
 * inside the margin delta, and the admissible victim (see above) first in (mean, position) order among those the
 * guide evicted is taken instead.  Returns the number of iterations where the guide's choice was followed
 * (0 = the guide's set is the rule's own), or -(iteration + 1) at the first iteration where the guide kept the
 * rule's victim and evicted no admissible one: a disagreement outside the margin.  keep[L] receives the replayed
 * survivor set, equal to guide_keep on success when that holds exactly B (or L, if L <= B) tokens. */
int roco_oracle_select_to_budget_guided(const double *s, const double *q, const int *n, int L, int B, int r,
                                        int mode, double delta, const int *guide_keep, int *keep) {
  for (int j = 0; j < L; ++j) keep[j] = 1;
  if (L <= B) return 0;
  double *cs = (double *)malloc(sizeof(double) * (size_t)L), *cq = (double *)malloc(sizeof(double) * (size_t)L);
  int *cn = (int *)malloc(sizeof(int) * (size_t)L), *cp = (int *)malloc(sizeof(int) * (size_t)L);
  int *adm = (int *)malloc(sizeof(int) * (size_t)L);
  int followed = 0, rc = 0;
  for (int alive = L, it = 0; alive > B; --alive, ++it) {
    int k = 0;
    for (int j = 0; j < L; ++j)
      if (keep[j]) { cs[k] = s[j]; cq[k] = q[j]; cn[k] = n[j]; cp[k] = j; ++k; }
    int c = roco_oracle_select(cs, cq, cn, cp, alive, r, mode, delta, NULL, NULL);
    if (guide_keep[cp[c]]) { /* the guide kept the rule's victim: look for the admissible one it evicted */
      roco_oracle_admissible_victims(cs, cq, cn, cp, alive, r, mode, delta, adm);
      int alt = -1;
      for (int i = 0; i < alive; ++i) {
        if (!adm[i] || guide_keep[cp[i]]) continue;
        double mi = cs[i] / cn[i];
        if (alt < 0 || mi < cs[alt] / cn[alt] || (mi == cs[alt] / cn[alt] && cp[i] < cp[alt])) alt = i;
      }
      if (alt < 0) { rc = -(it + 1); break; }
      c = alt;
      ++followed;
    }
    keep[cp[c]] = 0;
  }
  free(cs); free(cq); free(cn); free(cp); free(adm);
  return rc ? rc : followed;
}

typedef struct { double key; double eps; int pos; } rank_t;
static int cmp_key_pos(const void *a, const void *b) {
  const rank_t *x = (const rank_t *)a, *y = (const rank_t *)b;
  if (x->key < y->key) return -1;
  if (x->key > y->key) return 1;
  return (x->pos > y->pos) - (x->pos < y->pos);
}

/* Select-to-budget, one pass (EXCLUDE_TOP_R only, every Count > 0, r <= B): protect the r tokens last in
 * (variance, position) order; of the others evict the L-B first in (mean, position) order.  Equal to the
 * iterated form because a protected token is never in scope, so the protected set never changes.
 * uncertain[j] = 1 where token j's fate could flip within the relative margin delta (near either
 * boundary; if any token is near the protection boundary, the tokens around the eviction boundary that
 * a one-token shift per such token could reach are marked too).  Returns 0, or -1 on a precondition. */
int roco_oracle_select_to_budget_onepass(const double *s, const double *q, const int *n, int L, int B, int r,
                                         double delta, int *keep, int *uncertain) {
  for (int j = 0; j < L; ++j) { keep[j] = 1; if (uncertain) uncertain[j] = 0; }
  if (L <= B) return 0;
  if (r > B || r < 0) return -1;
  for (int j = 0; j < L; ++j) if (n[j] <= 0) return -1;
  rank_t *v = (rank_t *)malloc(sizeof(rank_t) * (size_t)L);
  for (int j = 0; j < L; ++j) {
    double mean = s[j] / n[j], a = q[j] / n[j];
    double var = a - mean * mean;
    if (var < 0.0) var = 0.0;
    v[j].key = var; v[j].eps = delta * (a + mean * mean); v[j].pos = j;
  }
  qsort(v, (size_t)L, sizeof(rank_t), cmp_key_pos);
  int nu = L - r; /* unprotected: v[0..nu) */
  int shaky = 0;  /* tokens that could cross the protection boundary */
  if (r > 0 && nu > 0 && uncertain) {
    double lo_prot = INFINITY, hi_unprot = -INFINITY;
    for (int k = nu; k < L; ++k) if (v[k].key - v[k].eps < lo_prot) lo_prot = v[k].key - v[k].eps;
    for (int k = 0; k < nu; ++k) if (v[k].key + v[k].eps > hi_unprot) hi_unprot = v[k].key + v[k].eps;
    for (int k = 0; k < L; ++k) {
      int crosses = (k < nu) ? (v[k].key + v[k].eps >= lo_prot) : (v[k].key - v[k].eps <= hi_unprot);
      if (crosses) { uncertain[v[k].pos] = 1; ++shaky; }
    }
  }
  rank_t *m = (rank_t *)malloc(sizeof(rank_t) * (size_t)(nu > 0 ? nu : 1));
  for (int k = 0; k < nu; ++k) {
    int j = v[k].pos;
    m[k].key = s[j] / n[j]; m[k].eps = delta * m[k].key; m[k].pos = j;
  }
  qsort(m, (size_t)nu, sizeof(rank_t), cmp_key_pos);
  int E = L - B;
  for (int k = 0; k < E; ++k) keep[m[k].pos] = 0;
  if (uncertain && E < nu) {
    double last_out = m[E - 1].key + m[E - 1].eps, first_in = m[E].key - m[E].eps;
    for (int k = 0; k < nu; ++k) {
      int near = (k < E) ? (m[k].key + m[k].eps >= first_in) : (m[k].key - m[k].eps <= last_out);
      if (near) uncertain[m[k].pos] = 1;
    }
    int lo = E - shaky, hi = E + shaky;
    if (lo < 0) lo = 0;
    if (hi > nu) hi = nu;
    for (int k = lo; k < hi; ++k) uncertain[m[k].pos] = 1;
  }
  free(v); free(m);
  return 0;
}

/* ------------------------------------------------------------ prefill ---- */

/* Whole prefill of one unit: statistics, select-to-budget, survivors copied in increasing position
 * order.  Q,K,V: [L][d].  Cache outputs: Kc,Vc [B][d]; sc,qc [B]; nc,posc [B] (pos = -1 for empty);
 * *live = min(L,B).  s_full,q_full,n_full: [L] pre-eviction statistics (required).  keep_io [L]:
 * if force_keep != 0 it is read as the survivor set to use; otherwise it receives the oracle's own.
 * uncertain [L] may be NULL.  LOWEST_R uses the iterated form; there every token is marked uncertain as
 * soon as one iteration was a near-tie. */
int roco_oracle_prefill_unit(const double *Q, const double *K, const double *V, int L, int d, int B, int r,
                             int mode, double scale, int count_self, double delta, double *Kc, double *Vc,
                             double *sc, double *qc, int *nc, int *posc, int *live, double *lse, double *s_full,
                             double *q_full, int *n_full, int *keep_io, int force_keep, int *uncertain) {
  roco_oracle_prefill_stats(Q, K, L, d, scale, count_self, lse, s_full, q_full, n_full, NULL);
  if (!force_keep) {
    int rc = 0;
    if (mode == ROCO_ORACLE_EXCLUDE_TOP_R && count_self)
      rc = roco_oracle_select_to_budget_onepass(s_full, q_full, n_full, L, B, r, delta, keep_io, uncertain);
    else {
      int n_near = roco_oracle_select_to_budget_iterated(s_full, q_full, n_full, L, B, r, mode, delta, keep_io);
      if (uncertain) for (int j = 0; j < L; ++j) uncertain[j] = n_near > 0; /* no finer analysis for this form */
    }
    if (rc) return rc;
  }
  int k = 0;
  for (int j = 0; j < L; ++j) {
    if (!keep_io[j]) continue;
    if (k >= B) return -2;
    memcpy(Kc + (size_t)k * d, K + (size_t)j * d, sizeof(double) * (size_t)d);
    memcpy(Vc + (size_t)k * d, V + (size_t)j * d, sizeof(double) * (size_t)d);
    sc[k] = s_full[j]; qc[k] = q_full[j]; nc[k] = n_full[j]; posc[k] = j;
    ++k;
  }
  *live = k;
  for (; k < B; ++k) {
    memset(Kc + (size_t)k * d, 0, sizeof(double) * (size_t)d);
    memset(Vc + (size_t)k * d, 0, sizeof(double) * (size_t)d);
    sc[k] = 0.0; qc[k] = 0.0; nc[k] = 0; posc[k] = -1;
  }
  return 0;
}

/* ------------------------------------------------------------- decode ---- */

static void insert_token(double *K, double *V, double *s, double *q, int *n, int *pos, int slot, int d,
                         const double *k_new, const double *v_new, int t) {
  memcpy(K + (size_t)slot * d, k_new, sizeof(double) * (size_t)d);
  memcpy(V + (size_t)slot * d, v_new, sizeof(double) * (size_t)d);
  s[slot] = 0.0; q[slot] = 0.0; n[slot] = 0; pos[slot] = t;
}

static double attend(const double *K, const double *V, double *s, double *q, int *n, int live, int d,
                     const double *qv, double scale, int skip_slot, double *out, double *p) {
  double lse = softmax_row(qv, K, live, d, scale, p);
  for (int c = 0; c < d; ++c) out[c] = 0.0;
  for (int j = 0; j < live; ++j) {
    for (int c = 0; c < d; ++c) out[c] += p[j] * V[(size_t)j * d + c];
    if (j == skip_slot) continue; /* count_self = 0: the new token's own query is not a "future" query */
    s[j] += p[j];
    q[j] += p[j] * p[j];
    n[j] += 1;
  }
  return lse;
}

/* One decode step of one unit.  Cache K,V [B][d]; s,q [B]; n,pos [B]; *live; *t_next = position of the
 * new token (incremented on return).  force_victim >= 0 replaces the policy's choice when the buffer is
 * full (used to continue from a common state after a logged near-tie); with force_only_near != 0 it does
 * so only at steps the margin analysis flags as near-ties.
 * Outputs: out [d]; *lse; *evicted_slot (-1 when nothing was evicted); *evicted_pos; *choice = the
 * policy's own victim (-1 if none); *near_tie.  p_out [B] may be NULL. */
void roco_oracle_decode_step_unit(double *K, double *V, double *s, double *q, int *n, int *pos, int *live,
                                  int *t_next, int B, int d, const double *qv, const double *k_new,
                                  const double *v_new, int r, int mode, int order, double scale,
                                  int count_self, double delta, int force_victim, int force_only_near,
                                  double *out, double *lse, int *evicted_slot, int *evicted_pos, int *choice,
                                  int *near_tie, double *p_out) {
  double *p = p_out ? p_out : (double *)malloc(sizeof(double) * (size_t)B);
  int t = *t_next, slot, near = 0, own = -1;
  *evicted_slot = -1;
  *evicted_pos = -1;
  if (order == ROCO_ORACLE_ATTEND_FIRST)
    *lse = attend(K, V, s, q, n, *live, d, qv, scale, -1, out, p); /* the new token is not in the cache yet */
  if (*live == B) { /* buffer full: run the policy (Sec. 4) */
    own = roco_oracle_select(s, q, n, pos, *live, r, mode, delta, &near, NULL);
    slot = (force_victim >= 0 && force_victim < B && (near || !force_only_near)) ? force_victim : own;
    *evicted_slot = slot;
    *evicted_pos = pos[slot];
  } else {
    slot = (*live)++;
  }
  insert_token(K, V, s, q, n, pos, slot, d, k_new, v_new, t);
  if (order == ROCO_ORACLE_EVICT_FIRST)
    *lse = attend(K, V, s, q, n, *live, d, qv, scale, count_self ? -1 : slot, out, p);
  *choice = own;
  *near_tie = near;
  *t_next = t + 1;
  if (!p_out) free(p);
}

/* ------------------------------------------------- batch drivers (OpenMP) -- */

void roco_oracle_decode_step_batch(int U, double *K, double *V, double *s, double *q, int *n, int *pos,
                                   int *live, int *t_next, int B, int d, const double *qv,
                                   const double *k_new, const double *v_new, int r, int mode, int order,
                                   double scale, int count_self, double delta, const int *force_victim,
                                   int force_only_near, double *out, double *lse, int *evicted_slot,
                                   int *evicted_pos, int *choice, int *near_tie) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    size_t kb = (size_t)u * B * d, sb = (size_t)u * B, vb = (size_t)u * d;
    roco_oracle_decode_step_unit(K + kb, V + kb, s + sb, q + sb, n + sb, pos + sb, live + u, t_next + u, B, d,
                                 qv + vb, k_new + vb, v_new + vb, r, mode, order, scale, count_self, delta,
                                 force_victim ? force_victim[u] : -1, force_only_near, out + vb, lse + u,
                                 evicted_slot + u, evicted_pos + u, choice + u, near_tie + u, NULL);
  }
}

/* Units may have different prompt lengths: unit u uses rows 0..lens[u]-1 of its [Lmax][d] block. */
int roco_oracle_prefill_batch(int U, const double *Q, const double *K, const double *V, const int *lens,
                              int Lmax, int d, int B, int r, int mode, double scale, int count_self,
                              double delta, double *Kc, double *Vc, double *sc, double *qc, int *nc, int *posc,
                              int *live, double *lse, double *s_full, double *q_full, int *n_full, int *keep_io,
                              int force_keep, int *uncertain) {
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    size_t ib = (size_t)u * Lmax * d, cb = (size_t)u * B * d, sb = (size_t)u * B, fb = (size_t)u * Lmax;
    int rc = roco_oracle_prefill_unit(Q + ib, K + ib, V + ib, lens[u], d, B, r, mode, scale, count_self, delta,
                                      Kc + cb, Vc + cb, sc + sb, qc + sb, nc + sb, posc + sb, live + u,
                                      lse + fb, s_full + fb, q_full + fb, n_full + fb, keep_io + fb, force_keep,
                                      uncertain ? uncertain + fb : NULL);
    if (rc) {
#pragma omp atomic write
      bad = rc;
    }
  }
  return bad;
}

/* ------------------------------------------------ block-wise evict-and-encode (Sec. 5.3 "Overhead", App. B) -- */

/* One eviction step that frees and encodes b tokens (Sec. 5.3: "The block size b controls the number of tokens
 * being freed and encoded within one eviction step").  Order as in Fig. 1: evict, insert, attend.
 *   1. need = live + b - B tokens (if positive) leave the cache: the per-step rule of Sec. 4.3 applied `need`
 *      times on the frozen statistics, each time on the tokens still alive.
 *   2. The b new tokens (positions t_next .. t_next+b-1) take, in order, the target slots sorted by slot index:
 *      the freed slots and, while the buffer is not full, slots live, live+1, ...
 *   3. Query i attends over the remaining old tokens and the new tokens 0..i (causal inside the block, Sec. 2.1);
 *      every attended token gets Count += 1, Acc += p, Acc^square += p^2 (Sec. 4.3).
 * Q, Kn, Vn: [b][d].  out: [b][d]; lse: [b].  evicted_slot / evicted_pos: [b], ascending slot order, -1 padded.
 * force_slots (may be NULL): [b] slots to evict instead of the policy's, -1 padded (used only when *near_tie).
 * *near_tie counts the eviction iterations inside the decision margin delta. */
void roco_oracle_block_step_unit(double *K, double *V, double *s, double *q, int *n, int *pos, int *live,
                                 int *t_next, int B, int d, int b, const double *Q, const double *Kn,
                                 const double *Vn, int r, int mode, double scale, double delta,
                                 const int *force_slots, double *out, double *lse, int *evicted_slot,
                                 int *evicted_pos, int *choice, int *near_tie) {
  const int live0 = *live, t0 = *t_next;
  int need = live0 + b - B;
  if (need < 0) need = 0;
  int *gone = (int *)calloc((size_t)B, sizeof(int));
  int n_near = 0;
  /* 1. policy on frozen statistics */
  double *cs = (double *)malloc(sizeof(double) * (size_t)B), *cq = (double *)malloc(sizeof(double) * (size_t)B);
  int *cn = (int *)malloc(sizeof(int) * (size_t)B), *cp = (int *)malloc(sizeof(int) * (size_t)B);
  int *cslot = (int *)malloc(sizeof(int) * (size_t)B);
  for (int it = 0; it < need; ++it) {
    int k = 0;
    for (int j = 0; j < live0; ++j)
      if (!gone[j]) { cs[k] = s[j]; cq[k] = q[j]; cn[k] = n[j]; cp[k] = pos[j]; cslot[k] = j; ++k; }
    int near = 0;
    int c = roco_oracle_select(cs, cq, cn, cp, k, r, mode, delta, &near, NULL);
    n_near += near;
    gone[cslot[c]] = 1;
  }
  for (int i = 0; i < b; ++i) { choice[i] = -1; evicted_slot[i] = -1; evicted_pos[i] = -1; }
  {
    int k = 0;
    for (int j = 0; j < live0; ++j) if (gone[j]) choice[k++] = j;
  }
  if (force_slots && n_near > 0) { /* continue from the other side's (in-margin) choice */
    memset(gone, 0, sizeof(int) * (size_t)B);
    for (int i = 0; i < b; ++i) if (force_slots[i] >= 0 && force_slots[i] < live0) gone[force_slots[i]] = 1;
  }
  {
    int k = 0;
    for (int j = 0; j < live0; ++j) if (gone[j]) { evicted_slot[k] = j; evicted_pos[k] = pos[j]; ++k; }
  }
  /* 2. insert: target slots in increasing slot order */
  int *slot_of_new = (int *)malloc(sizeof(int) * (size_t)b);
  {
    int k = 0;
    for (int j = 0; j < B && k < b; ++j)
      if (j >= live0 || gone[j]) slot_of_new[k++] = j;
  }
  int live1 = live0 - need + b;
  for (int i = 0; i < b; ++i)
    insert_token(K, V, s, q, n, pos, slot_of_new[i], d, Kn + (size_t)i * d, Vn + (size_t)i * d, t0 + i);
  /* 3. attention of query i over the old survivors and the new tokens 0..i */
  double *p = (double *)malloc(sizeof(double) * (size_t)B);
  double *Kc = (double *)malloc(sizeof(double) * (size_t)B * d);
  int *members = (int *)malloc(sizeof(int) * (size_t)B);
  for (int i = 0; i < b; ++i) {
    int m = 0;
    for (int j = 0; j < live1; ++j) {
      int newer = 0;
      for (int i2 = i + 1; i2 < b; ++i2) if (slot_of_new[i2] == j) newer = 1;
      if (!newer) members[m++] = j;
    }
    for (int k = 0; k < m; ++k) memcpy(Kc + (size_t)k * d, K + (size_t)members[k] * d, sizeof(double) * (size_t)d);
    lse[i] = softmax_row(Q + (size_t)i * d, Kc, m, d, scale, p);
    for (int c = 0; c < d; ++c) out[(size_t)i * d + c] = 0.0;
    for (int k = 0; k < m; ++k) {
      const int j = members[k];
      for (int c = 0; c < d; ++c) out[(size_t)i * d + c] += p[k] * V[(size_t)j * d + c];
      s[j] += p[k];
      q[j] += p[k] * p[k];
      n[j] += 1;
    }
  }
  *live = live1;
  *t_next = t0 + b;
  *near_tie = n_near;
  free(gone); free(cs); free(cq); free(cn); free(cp); free(cslot); free(slot_of_new); free(p); free(Kc); free(members);
}

/* --------------------------------------------------- grouped-query attention (Sec. 5.3, App. A "Extension") -- */

/* One decode step of a key-value head shared by `group` query heads (Sec. 5.3: the group-wise averaged attention
 * score updates the importance score).  Order as in Fig. 1 (evict, insert, attend).  Every query head g attends
 * over the same cache: p_g = Softmax(scale * q_g K^T), out_g = p_g V (Eq. 1); the statistics of Sec. 4.3 receive
 * the group mean pbar = (1/group) sum_g p_g: Count += 1, Acc += pbar, Acc^square += pbar^2.
 * Q: [group][d]; out: [group][d]; lse: [group]. */
void roco_oracle_gqa_step_unit(double *K, double *V, double *s, double *q, int *n, int *pos, int *live, int *t_next,
                               int B, int d, int group, const double *Q, const double *k_new, const double *v_new,
                               int r, int mode, double scale, double delta, int force_victim, double *out,
                               double *lse, int *evicted_slot, int *evicted_pos, int *choice, int *near_tie) {
  int t = *t_next, slot, near = 0, own = -1;
  *evicted_slot = -1;
  *evicted_pos = -1;
  if (*live == B) {
    own = roco_oracle_select(s, q, n, pos, *live, r, mode, delta, &near, NULL);
    slot = (force_victim >= 0 && force_victim < B && near) ? force_victim : own;
    *evicted_slot = slot;
    *evicted_pos = pos[slot];
  } else {
    slot = (*live)++;
  }
  insert_token(K, V, s, q, n, pos, slot, d, k_new, v_new, t);
  const int m = *live;
  double *p = (double *)malloc(sizeof(double) * (size_t)m), *pbar = (double *)calloc((size_t)m, sizeof(double));
  for (int g = 0; g < group; ++g) {
    lse[g] = softmax_row(Q + (size_t)g * d, K, m, d, scale, p);
    for (int c = 0; c < d; ++c) out[(size_t)g * d + c] = 0.0;
    for (int j = 0; j < m; ++j) {
      for (int c = 0; c < d; ++c) out[(size_t)g * d + c] += p[j] * V[(size_t)j * d + c];
      pbar[j] += p[j];
    }
  }
  for (int j = 0; j < m; ++j) {
    const double pb = pbar[j] / group;
    s[j] += pb;
    q[j] += pb * pb;
    n[j] += 1;
  }
  *choice = own;
  *near_tie = near;
  *t_next = t + 1;
  free(p); free(pbar);
}

/* --------- block-wise evict-and-encode on a grouped-query model (Sec. 5.3 "Extension to Grouped-Query Attention",
 * App. A; App. B / Table 9: block-wise eviction on Zephyr-7B, a grouped-query model) -- */

/* One eviction step that frees and encodes b tokens of a key-value head shared by `group` query heads.
 * Steps 1 and 2 as in roco_oracle_block_step_unit (rule applied on frozen statistics; new tokens to the freed /
 * free slots in increasing slot order).  Step 3: for token i of the block every query head g attends over the
 * remaining old tokens and the new tokens 0..i (Eq. 1, causal inside the block), out_{i,g} = p_{i,g} V; the
 * statistics of Sec. 4.3 receive, once per token of the block, the group-wise averaged probability
 * pbar_i = (1/group) sum_g p_{i,g}: Count += 1, Acc += pbar_i, Acc^square += pbar_i^2.
 * group = 1 is roco_oracle_block_step_unit; b = 1 is roco_oracle_gqa_step_unit.
 * Q: [b][group][d]; Kn, Vn: [b][d]; out: [b][group][d]; lse: [b][group].  Other arguments as the block step. */
void roco_oracle_gqa_block_step_unit(double *K, double *V, double *s, double *q, int *n, int *pos, int *live,
                                     int *t_next, int B, int d, int b, int group, const double *Q, const double *Kn,
                                     const double *Vn, int r, int mode, double scale, double delta,
                                     const int *force_slots, double *out, double *lse, int *evicted_slot,
                                     int *evicted_pos, int *choice, int *near_tie) {
  const int live0 = *live, t0 = *t_next;
  int need = live0 + b - B;
  if (need < 0) need = 0;
  int *gone = (int *)calloc((size_t)B, sizeof(int));
  int n_near = 0;
  double *cs = (double *)malloc(sizeof(double) * (size_t)B), *cq = (double *)malloc(sizeof(double) * (size_t)B);
  int *cn = (int *)malloc(sizeof(int) * (size_t)B), *cp = (int *)malloc(sizeof(int) * (size_t)B);
  int *cslot = (int *)malloc(sizeof(int) * (size_t)B);
  for (int it = 0; it < need; ++it) { /* 1. the rule, `need` times, on the statistics as they stand */
    int k = 0;
    for (int j = 0; j < live0; ++j)
      if (!gone[j]) { cs[k] = s[j]; cq[k] = q[j]; cn[k] = n[j]; cp[k] = pos[j]; cslot[k] = j; ++k; }
    int near = 0;
    int c = roco_oracle_select(cs, cq, cn, cp, k, r, mode, delta, &near, NULL);
    n_near += near;
    gone[cslot[c]] = 1;
  }
  for (int i = 0; i < b; ++i) { choice[i] = -1; evicted_slot[i] = -1; evicted_pos[i] = -1; }
  {
    int k = 0;
    for (int j = 0; j < live0; ++j) if (gone[j]) choice[k++] = j;
  }
  if (force_slots && n_near > 0) {
    memset(gone, 0, sizeof(int) * (size_t)B);
    for (int i = 0; i < b; ++i) if (force_slots[i] >= 0 && force_slots[i] < live0) gone[force_slots[i]] = 1;
  }
  {
    int k = 0;
    for (int j = 0; j < live0; ++j) if (gone[j]) { evicted_slot[k] = j; evicted_pos[k] = pos[j]; ++k; }
  }
  int *slot_of_new = (int *)malloc(sizeof(int) * (size_t)b); /* 2. insert */
  {
    int k = 0;
    for (int j = 0; j < B && k < b; ++j)
      if (j >= live0 || gone[j]) slot_of_new[k++] = j;
  }
  const int live1 = live0 - need + b;
  for (int i = 0; i < b; ++i)
    insert_token(K, V, s, q, n, pos, slot_of_new[i], d, Kn + (size_t)i * d, Vn + (size_t)i * d, t0 + i);
  double *p = (double *)malloc(sizeof(double) * (size_t)B), *pbar = (double *)malloc(sizeof(double) * (size_t)B);
  double *Kc = (double *)malloc(sizeof(double) * (size_t)B * d);
  int *members = (int *)malloc(sizeof(int) * (size_t)B);
  for (int i = 0; i < b; ++i) { /* 3. token i of the block: every head of the group, then the group mean */
    int m = 0;
    for (int j = 0; j < live1; ++j) {
      int newer = 0;
      for (int i2 = i + 1; i2 < b; ++i2) if (slot_of_new[i2] == j) newer = 1;
      if (!newer) members[m++] = j;
    }
    for (int k = 0; k < m; ++k) {
      memcpy(Kc + (size_t)k * d, K + (size_t)members[k] * d, sizeof(double) * (size_t)d);
      pbar[k] = 0.0;
    }
    for (int g = 0; g < group; ++g) {
      const size_t row = (size_t)i * group + g;
      lse[row] = softmax_row(Q + row * d, Kc, m, d, scale, p);
      for (int c = 0; c < d; ++c) out[row * d + c] = 0.0;
      for (int k = 0; k < m; ++k) {
        for (int c = 0; c < d; ++c) out[row * d + c] += p[k] * V[(size_t)members[k] * d + c];
        pbar[k] += p[k];
      }
    }
    for (int k = 0; k < m; ++k) {
      const int j = members[k];
      const double pb = pbar[k] / group;
      s[j] += pb;
      q[j] += pb * pb;
      n[j] += 1;
    }
  }
  *live = live1;
  *t_next = t0 + b;
  *near_tie = n_near;
  free(gone); free(cs); free(cq); free(cn); free(cp); free(cslot); free(slot_of_new); free(p); free(pbar); free(Kc);
  free(members);
}

void roco_oracle_gqa_block_step_batch(int U, double *K, double *V, double *s, double *q, int *n, int *pos, int *live,
                                      int *t_next, int B, int d, int b, int group, const double *Q, const double *Kn,
                                      const double *Vn, int r, int mode, double scale, double delta,
                                      const int *force_slots, double *out, double *lse, int *evicted_slot,
                                      int *evicted_pos, int *choice, int *near_tie) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    size_t kb = (size_t)u * B * d, sb = (size_t)u * B, qb = (size_t)u * b * group * d, vb = (size_t)u * b * d;
    size_t ib = (size_t)u * b;
    roco_oracle_gqa_block_step_unit(K + kb, V + kb, s + sb, q + sb, n + sb, pos + sb, live + u, t_next + u, B, d, b,
                                    group, Q + qb, Kn + vb, Vn + vb, r, mode, scale, delta,
                                    force_slots ? force_slots + ib : NULL, out + qb, lse + ib * group,
                                    evicted_slot + ib, evicted_pos + ib, choice + ib, near_tie + u);
  }
}

void roco_oracle_block_step_batch(int U, double *K, double *V, double *s, double *q, int *n, int *pos, int *live,
                                  int *t_next, int B, int d, int b, const double *Q, const double *Kn,
                                  const double *Vn, int r, int mode, double scale, double delta,
                                  const int *force_slots, double *out, double *lse, int *evicted_slot,
                                  int *evicted_pos, int *choice, int *near_tie) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    size_t kb = (size_t)u * B * d, sb = (size_t)u * B, vb = (size_t)u * b * d, ib = (size_t)u * b;
    roco_oracle_block_step_unit(K + kb, V + kb, s + sb, q + sb, n + sb, pos + sb, live + u, t_next + u, B, d, b,
                                Q + vb, Kn + vb, Vn + vb, r, mode, scale, delta,
                                force_slots ? force_slots + ib : NULL, out + vb, lse + ib, evicted_slot + ib,
                                evicted_pos + ib, choice + ib, near_tie + u);
  }
}

void roco_oracle_gqa_step_batch(int U, double *K, double *V, double *s, double *q, int *n, int *pos, int *live,
                                int *t_next, int B, int d, int group, const double *Q, const double *k_new,
                                const double *v_new, int r, int mode, double scale, double delta,
                                const int *force_victim, double *out, double *lse, int *evicted_slot,
                                int *evicted_pos, int *choice, int *near_tie) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    size_t kb = (size_t)u * B * d, sb = (size_t)u * B, qb = (size_t)u * group * d, vb = (size_t)u * d;
    roco_oracle_gqa_step_unit(K + kb, V + kb, s + sb, q + sb, n + sb, pos + sb, live + u, t_next + u, B, d, group,
                              Q + qb, k_new + vb, v_new + vb, r, mode, scale, delta,
                              force_victim ? force_victim[u] : -1, out + qb, lse + (size_t)u * group,
                              evicted_slot + u, evicted_pos + u, choice + u, near_tie + u);
  }
}

/* ---------------------------------------------- the other eviction policies of Table 1 (Sec. 4.1, 4.2, 5.1) -- */

enum {
  ROCO_ORACLE_POLICY_ROCO = 0,         /* MAS + standard-deviation scope (Sec. 4.3), EXCLUDE_TOP_R reading        */
  ROCO_ORACLE_POLICY_RANDOM = 1,       /* Sec. 4.1: a randomly chosen pair (the draw is an input)                  */
  ROCO_ORACLE_POLICY_RECENCY = 2,      /* Sec. 4.1: the farthest token                                             */
  ROCO_ORACLE_POLICY_STREAMLLM = 3,    /* Sec. 5.1: the first token after the 4 initial attention-sink tokens      */
  ROCO_ORACLE_POLICY_SCISSORHANDS = 4, /* Sec. 4.1 AQAS (1 = above-average probability) + local window of size r   */
  ROCO_ORACLE_POLICY_H2O = 5,          /* Sec. 4.1 AAS (accumulated probability) + local window of size r          */
  ROCO_ORACLE_POLICY_TOVA = 6,         /* Sec. 4.1 LTAS (the last query's probability), no scope restriction       */
  ROCO_ORACLE_POLICY_MAS_WINDOW = 7    /* Sec. 4.3 preliminary experiment: MAS + local window of size r            */
};

/* The token a policy evicts from a full buffer (Sec. 4.1, 4.2, 5.1), given the state arrays described at
 * roco_oracle_policy_step_unit and t, the position of the incoming token.  *near: the decision is inside the
 * margin delta. */
static int policy_pick(const double *s, const double *q, const int *n, const int *pos, int B, int policy, int r,
                       unsigned rnd, int t, double delta, int *near) {
  int own = -1;
  *near = 0;
  if (policy == ROCO_ORACLE_POLICY_ROCO) return roco_oracle_select(s, q, n, pos, B, r, ROCO_ORACLE_EXCLUDE_TOP_R, delta, near, NULL);
  if (policy == ROCO_ORACLE_POLICY_RANDOM) return (int)(rnd % (unsigned)B);
  const int windowed = policy == ROCO_ORACLE_POLICY_SCISSORHANDS || policy == ROCO_ORACLE_POLICY_H2O ||
                       policy == ROCO_ORACLE_POLICY_MAS_WINDOW;
  int any = 0;
  for (int j = 0; j < B; ++j) if (!windowed || pos[j] < t - r) any = 1;
  double best = 0.0, second = INFINITY;
  for (int j = 0; j < B; ++j) {
    if (windowed && any && !(pos[j] < t - r)) continue;
    if (policy == ROCO_ORACLE_POLICY_STREAMLLM && pos[j] < 4) continue;
    double sc = 0.0; /* RECENCY, STREAMLLM: position alone decides */
    if (policy == ROCO_ORACLE_POLICY_H2O) sc = s[j];
    if (policy == ROCO_ORACLE_POLICY_SCISSORHANDS || policy == ROCO_ORACLE_POLICY_TOVA) sc = q[j];
    if (policy == ROCO_ORACLE_POLICY_MAS_WINDOW) sc = s[j] / n[j];
    if (own < 0 || sc < best || (sc == best && pos[j] < pos[own])) {
      if (own >= 0) second = best < second ? best : second;
      best = sc; own = j;
    } else if (sc < second) {
      second = sc;
    }
  }
  if (own < 0) { own = 0; for (int j = 1; j < B; ++j) if (pos[j] < pos[own]) own = j; } /* all sinks */
  const int real_valued = policy == ROCO_ORACLE_POLICY_H2O || policy == ROCO_ORACLE_POLICY_TOVA ||
                          policy == ROCO_ORACLE_POLICY_MAS_WINDOW;
  if (real_valued && second - best <= delta * (second + best)) *near = 1;
  return own;
}

/* Eq. 1 over the m occupied slots and the policy's statistics update; returns the log-sum-exp. */
static double policy_attend(const double *K, const double *V, double *s, double *q, int *n, int m, int d,
                            const double *qv, double scale, int policy, double delta, double *out, int *quant_near) {
  double *p = (double *)malloc(sizeof(double) * (size_t)(m > 0 ? m : 1));
  const double lse = softmax_row(qv, K, m, d, scale, p);
  for (int c = 0; c < d; ++c) out[c] = 0.0;
  for (int j = 0; j < m; ++j) {
    for (int c = 0; c < d; ++c) out[c] += p[j] * V[(size_t)j * d + c];
    s[j] += p[j];
    n[j] += 1;
    if (quant_near) quant_near[j] = 0;
    if (policy == ROCO_ORACLE_POLICY_SCISSORHANDS) {
      q[j] += (p[j] * m > 1.0) ? 1.0 : 0.0;
      if (quant_near && fabs(p[j] * m - 1.0) <= delta) quant_near[j] = 1;
    } else if (policy == ROCO_ORACLE_POLICY_TOVA) {
      q[j] = p[j];
    } else {
      q[j] += p[j] * p[j];
    }
  }
  free(p);
  return lse;
}

/* One decode step under one of the policies above, in either order of Fig. 1 / its alternative: EVICT_FIRST
 * (evict, insert, attend) or ATTEND_FIRST (attend over the cache as it stands, update, then evict and insert).
 * State: s = accumulated probability (Acc), n = Count for every policy; q = Acc^square, except under
 * SCISSORHANDS, where it accumulates the quantised score (1 if the token's probability exceeds the average
 * 1/live of this query, else 0), and under TOVA, where it holds the last query's probability.
 * Local window (Sec. 4.2): tokens outside a window of the r most recent positions are evictable, i.e. pos < t - r
 * with t the position of the incoming token.  Ties: (score asc, position asc).
 * rnd: the random draw for RANDOM (victim = rnd mod live).  quant_near [B] (may be NULL): set to 1 where a
 * SCISSORHANDS quantisation falls within delta (relative) of the average. */
void roco_oracle_policy_step_unit(double *K, double *V, double *s, double *q, int *n, int *pos, int *live,
                                  int *t_next, int B, int d, const double *qv, const double *k_new,
                                  const double *v_new, int policy, int r, int order, unsigned rnd, double scale,
                                  double delta, int force_victim, double *out, double *lse, int *evicted_slot,
                                  int *evicted_pos, int *choice, int *near_tie, int *quant_near) {
  const int t = *t_next;
  int slot, own = -1, near = 0;
  *evicted_slot = -1;
  *evicted_pos = -1;
  if (order == ROCO_ORACLE_ATTEND_FIRST)
    *lse = policy_attend(K, V, s, q, n, *live, d, qv, scale, policy, delta, out, quant_near);
  if (*live == B) {
    own = policy_pick(s, q, n, pos, B, policy, r, rnd, t, delta, &near);
    slot = (force_victim >= 0 && force_victim < B && near) ? force_victim : own;
    *evicted_slot = slot;
    *evicted_pos = pos[slot];
  } else {
    slot = (*live)++;
  }
  insert_token(K, V, s, q, n, pos, slot, d, k_new, v_new, t);
  if (order == ROCO_ORACLE_EVICT_FIRST)
    *lse = policy_attend(K, V, s, q, n, *live, d, qv, scale, policy, delta, out, quant_near);
  *choice = own;
  *near_tie = near;
  *t_next = t + 1;
}

void roco_oracle_policy_step_batch(int U, double *K, double *V, double *s, double *q, int *n, int *pos, int *live,
                                   int *t_next, int B, int d, const double *qv, const double *k_new,
                                   const double *v_new, int policy, int r, int order, const unsigned *rnd,
                                   double scale, double delta, const int *force_victim, double *out, double *lse,
                                   int *evicted_slot,
                                   int *evicted_pos, int *choice, int *near_tie, int *quant_near) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    size_t kb = (size_t)u * B * d, sb = (size_t)u * B, vb = (size_t)u * d;
    roco_oracle_policy_step_unit(K + kb, V + kb, s + sb, q + sb, n + sb, pos + sb, live + u, t_next + u, B, d, qv + vb,
                                 k_new + vb, v_new + vb, policy, r, order, rnd ? rnd[u] : 0u, scale, delta,
                                 force_victim ? force_victim[u] : -1, out + vb, lse + u, evicted_slot + u,
                                 evicted_pos + u, choice + u, near_tie + u, quant_near ? quant_near + sb : NULL);
  }
}

/* ------------------------------ consistency with the full cache (Sec. 4.3 "Preliminary Experiments", set-up) -- */

/* The importance score a policy ranks the cached tokens by (Sec. 4.1; MAS: Sec. 4.3), from the statistics the
 * policy step keeps: AAS = Acc (H2O), AQAS = the accumulated quantised score (ScissorHands, kept in q), LTAS = the
 * last query's probability (TOVA, kept in q), MAS = Acc / Count (RoCo and MAS + window; 0 while Count = 0). */
double roco_oracle_policy_score(int policy, double s, double q, int n) {
  if (policy == ROCO_ORACLE_POLICY_H2O) return s;
  if (policy == ROCO_ORACLE_POLICY_SCISSORHANDS || policy == ROCO_ORACLE_POLICY_TOVA) return q;
  return n > 0 ? s / n : 0.0;
}

typedef struct { double score; int pos; } scored_t;
static int cmp_score_pos(const void *a, const void *b) {
  const scored_t *x = (const scored_t *)a, *y = (const scored_t *)b;
  if (x->score < y->score) return -1;
  if (x->score > y->score) return 1;
  return (x->pos > y->pos) - (x->pos < y->pos);
}

/* The B most important tokens of a full cache are the ones left when the policy's eviction order -- (score asc,
 * position asc) -- has removed live - B tokens: the last B in that order.  Returns how many of them are among
 * kept_pos[B] (the positions a budgeted cache retains); the Jaccard similarity of the two B-sized sets is
 * overlap / (2B - overlap).  *slack (may be NULL) bounds by how much that count can move if every score is off by
 * at most the relative margin delta: the smaller of the number of top-B tokens within the margin of the best
 * excluded score and the number of excluded tokens within the margin of the worst included score (scores exactly
 * equal to the other side's boundary count as within the margin unless exact_ties_firm, for integer-valued
 * scores, where equal values are ordered by position on every implementation alike).  live >= B >= 1. */
int roco_oracle_topb_overlap(const double *score, const int *pos, int live, const int *kept_pos, int B, double delta,
                             int exact_ties_firm, int *slack) {
  scored_t *c = (scored_t *)malloc(sizeof(scored_t) * (size_t)live);
  for (int j = 0; j < live; ++j) { c[j].score = score[j]; c[j].pos = pos[j]; }
  qsort(c, (size_t)live, sizeof(scored_t), cmp_score_pos);
  const int cut = live - B; /* c[cut..live) is the top-B set */
  int overlap = 0;
  for (int k = cut; k < live; ++k)
    for (int i = 0; i < B; ++i)
      if (kept_pos[i] == c[k].pos) { ++overlap; break; }
  if (slack) {
    *slack = 0;
    if (cut > 0) {
      const double best_out = c[cut - 1].score, worst_in = c[cut].score;
      int near_in = 0, near_out = 0;
      for (int k = cut; k < live; ++k) {
        const double gap = c[k].score - best_out;
        if (gap <= delta * (fabs(c[k].score) + fabs(best_out)) && !(exact_ties_firm && gap == 0.0)) ++near_in;
      }
      for (int k = 0; k < cut; ++k) {
        const double gap = worst_in - c[k].score;
        if (gap <= delta * (fabs(c[k].score) + fabs(worst_in)) && !(exact_ties_firm && gap == 0.0)) ++near_out;
      }
      *slack = near_in < near_out ? near_in : near_out;
    }
  }
  free(c);
  return overlap;
}

/* Jaccard similarity |X and Y| / |X or Y| of two sets of B elements each that share `overlap` elements. */
double roco_oracle_jaccard_equal_sets(int overlap, int B) { return (double)overlap / (double)(2 * B - overlap); }

