"""fp64 CPU oracle for RoCo KV-constrained inference (test infrastructure only).

Thin ctypes/numpy marshalling around ``roco_oracle.c``; all arithmetic is in the C file.
Only the test suite, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library never does.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from typing import Optional

import numpy as np

from .build import build as build_library

EXCLUDE_TOP_R, LOWEST_R = 0, 1
EVICT_FIRST, ATTEND_FIRST = 0, 1
(POLICY_ROCO, POLICY_RANDOM, POLICY_RECENCY, POLICY_STREAMLLM, POLICY_SCISSORHANDS, POLICY_H2O, POLICY_TOVA,
 POLICY_MAS_WINDOW) = range(8)

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build_library())
        _lib.roco_oracle_threads.restype = C.c_int
        _lib.roco_oracle_select.restype = C.c_int
        _lib.roco_oracle_select_to_budget_iterated.restype = C.c_int
        _lib.roco_oracle_attention_row.restype = C.c_double
        _lib.roco_oracle_select_to_budget_onepass.restype = C.c_int
        _lib.roco_oracle_select_to_budget_guided.restype = C.c_int
        _lib.roco_oracle_policy_score.restype = C.c_double
        _lib.roco_oracle_policy_score.argtypes = [C.c_int, C.c_double, C.c_double, C.c_int]
        _lib.roco_oracle_topb_overlap.restype = C.c_int
        _lib.roco_oracle_jaccard_equal_sets.restype = C.c_double
        _lib.roco_oracle_prefill_unit.restype = C.c_int
        _lib.roco_oracle_prefill_batch.restype = C.c_int
    return _lib


def threads() -> int:
    return int(lib().roco_oracle_threads())


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def prefill_stats(Q, K, scale, count_self=1, want_P=False):
    """Column statistics of the causal softmax of one unit.  Q, K: [L][d].
    Returns lse [L], s [L], q [L], n [L] (and P [L][L] if asked)."""
    Q, K = _f64(Q), _f64(K)
    L, d = Q.shape
    lse = np.zeros(L); s = np.zeros(L); q = np.zeros(L); n = np.zeros(L, np.int32)
    P = np.zeros((L, L)) if want_P else None
    lib().roco_oracle_prefill_stats(_p(Q), _p(K), C.c_int(L), C.c_int(d), C.c_double(scale),
                                    C.c_int(count_self), _p(lse), _p(s), _p(q), _p(n), _p(P))
    return (lse, s, q, n, P) if want_P else (lse, s, q, n)


def attention_row(qv, K, scale):
    """Eq. 1 for one query over the rows of K: returns (p [count], lse)."""
    qv, K = _f64(qv), _f64(K)
    p = np.zeros(K.shape[0])
    lse = lib().roco_oracle_attention_row(_p(qv), _p(K), C.c_int(K.shape[0]), C.c_int(K.shape[1]), C.c_double(scale),
                                          _p(p))
    return p, float(lse)


def prompt_attention_rows(Q, K, V, rows, scale):
    """Causal attention output of a prompt (Eq. 1 with the mask of Sec. 2.1) for the query rows listed:
    out_i = sum_{j<=i} p_ij V_j.  Q, K, V: [L][d].  Returns (out [len(rows)][d], lse [len(rows)])."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    out = np.zeros((len(rows), V.shape[1]))
    lse = np.zeros(len(rows))
    for t, i in enumerate(rows):
        p, lse[t] = attention_row(Q[i], K[: i + 1], scale)
        for j in range(i + 1):
            out[t] += p[j] * V[j]
    return out, lse


def select(s, q, n, pos, r, mode, delta=1e-5):
    """Victim slot among slots 0..len-1.  Returns (slot, near_tie, scope_size)."""
    s, q, n, pos = _f64(s), _f64(q), _i32(n), _i32(pos)
    near, m = C.c_int(0), C.c_int(0)
    slot = lib().roco_oracle_select(_p(s), _p(q), _p(n), _p(pos), C.c_int(len(s)), C.c_int(r), C.c_int(mode),
                                    C.c_double(delta), C.byref(near), C.byref(m))
    return int(slot), bool(near.value), int(m.value)


def select_to_budget_iterated(s, q, n, B, r, mode, delta=0.0):
    s, q, n = _f64(s), _f64(q), _i32(n)
    keep = np.zeros(len(s), np.int32)
    lib().roco_oracle_select_to_budget_iterated(_p(s), _p(q), _p(n), C.c_int(len(s)), C.c_int(B), C.c_int(r),
                                                C.c_int(mode), C.c_double(delta), _p(keep))
    return keep.astype(bool)


def admissible_victims(s, q, n, pos, r, mode, delta=1e-5):
    """Tokens that could be the victim if every statistic were off by at most the relative margin delta: [len] bool."""
    s, q, n, pos = _f64(s), _f64(q), _i32(n), _i32(pos)
    adm = np.zeros(len(s), np.int32)
    lib().roco_oracle_admissible_victims(_p(s), _p(q), _p(n), _p(pos), C.c_int(len(s)), C.c_int(r), C.c_int(mode),
                                         C.c_double(delta), _p(adm))
    return adm.astype(bool)


def select_to_budget_guided(s, q, n, B, r, mode, guide_keep, delta=1e-5):
    """The iterated select-to-budget replayed next to another implementation's survivor set.  Returns
    (followed, keep): followed = number of in-margin iterations where the guide's choice was taken, or
    -(iteration + 1) at the first disagreement outside the margin; keep = the replayed survivor set."""
    s, q, n = _f64(s), _f64(q), _i32(n)
    guide = _i32(np.asarray(guide_keep).astype(np.int32))
    keep = np.zeros(len(s), np.int32)
    rc = lib().roco_oracle_select_to_budget_guided(_p(s), _p(q), _p(n), C.c_int(len(s)), C.c_int(B), C.c_int(r),
                                                   C.c_int(mode), C.c_double(delta), _p(guide), _p(keep))
    return int(rc), keep.astype(bool)


def select_to_budget_onepass(s, q, n, B, r, delta=1e-5):
    s, q, n = _f64(s), _f64(q), _i32(n)
    keep = np.zeros(len(s), np.int32); unc = np.zeros(len(s), np.int32)
    rc = lib().roco_oracle_select_to_budget_onepass(_p(s), _p(q), _p(n), C.c_int(len(s)), C.c_int(B), C.c_int(r),
                                                    C.c_double(delta), _p(keep), _p(unc))
    if rc:
        raise ValueError(f"one-pass select-to-budget precondition failed ({rc})")
    return keep.astype(bool), unc.astype(bool)


@dataclass
class State:
    """Budgeted cache of U units, everything fp64/int32 numpy, unit-major."""
    K: np.ndarray      # [U][B][d]
    V: np.ndarray      # [U][B][d]
    s: np.ndarray      # [U][B]
    q: np.ndarray      # [U][B]
    n: np.ndarray      # [U][B] int32
    pos: np.ndarray    # [U][B] int32, -1 = empty
    live: np.ndarray   # [U] int32
    t_next: np.ndarray  # [U] int32

    @property
    def U(self): return self.K.shape[0]
    @property
    def B(self): return self.K.shape[1]
    @property
    def d(self): return self.K.shape[2]

    def copy(self) -> "State":
        return State(*(a.copy() for a in (self.K, self.V, self.s, self.q, self.n, self.pos, self.live, self.t_next)))


def empty_state(U, B, d) -> State:
    return State(np.zeros((U, B, d)), np.zeros((U, B, d)), np.zeros((U, B)), np.zeros((U, B)),
                 np.zeros((U, B), np.int32), np.full((U, B), -1, np.int32), np.zeros(U, np.int32),
                 np.zeros(U, np.int32))


@dataclass
class PrefillResult:
    state: State
    lse: np.ndarray        # [U][Lmax]
    s_full: np.ndarray     # [U][Lmax]
    q_full: np.ndarray
    n_full: np.ndarray
    keep: np.ndarray       # [U][Lmax] bool
    uncertain: np.ndarray  # [U][Lmax] bool


def prefill(Q, K, V, lens, B, r, mode, scale, count_self=1, delta=1e-5, force_keep=None) -> PrefillResult:
    """Q, K, V: [U][Lmax][d]; lens: [U] per-unit prompt length."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    U, Lmax, d = Q.shape
    lens = _i32(lens)
    st = empty_state(U, B, d)
    lse = np.zeros((U, Lmax)); sf = np.zeros((U, Lmax)); qf = np.zeros((U, Lmax)); nf = np.zeros((U, Lmax), np.int32)
    keep = np.zeros((U, Lmax), np.int32) if force_keep is None else _i32(force_keep).copy()
    unc = np.zeros((U, Lmax), np.int32)
    rc = lib().roco_oracle_prefill_batch(C.c_int(U), _p(Q), _p(K), _p(V), _p(lens), C.c_int(Lmax), C.c_int(d),
                                         C.c_int(B), C.c_int(r), C.c_int(mode), C.c_double(scale),
                                         C.c_int(count_self), C.c_double(delta), _p(st.K), _p(st.V), _p(st.s),
                                         _p(st.q), _p(st.n), _p(st.pos), _p(st.live), _p(lse), _p(sf), _p(qf),
                                         _p(nf), _p(keep), C.c_int(0 if force_keep is None else 1), _p(unc))
    if rc:
        raise ValueError(f"oracle prefill failed ({rc})")
    st.t_next[:] = lens
    return PrefillResult(st, lse, sf, qf, nf, keep.astype(bool), unc.astype(bool))


@dataclass
class StepResult:
    out: np.ndarray           # [U][d]
    lse: np.ndarray           # [U]
    evicted_slot: np.ndarray  # [U], -1 = nothing evicted
    evicted_pos: np.ndarray   # [U]
    choice: np.ndarray        # [U] the policy's own victim (differs from evicted_slot only when forced)
    near_tie: np.ndarray      # [U] bool


def decode_step(st: State, qv, k_new, v_new, r, mode, order, scale, count_self=1, delta=1e-5,
                force_victim: Optional[np.ndarray] = None, force_only_near: bool = False) -> StepResult:
    """One decode step of every unit, in place on `st`.  qv, k_new, v_new: [U][d].
    force_victim[u] >= 0 replaces the policy's victim (only at near-ties if force_only_near)."""
    qv, k_new, v_new = _f64(qv), _f64(k_new), _f64(v_new)
    U, B, d = st.U, st.B, st.d
    out = np.zeros((U, d)); lse = np.zeros(U)
    es = np.zeros(U, np.int32); ep = np.zeros(U, np.int32); ch = np.zeros(U, np.int32); nt = np.zeros(U, np.int32)
    fv = None if force_victim is None else _i32(force_victim)
    lib().roco_oracle_decode_step_batch(C.c_int(U), _p(st.K), _p(st.V), _p(st.s), _p(st.q), _p(st.n), _p(st.pos),
                                        _p(st.live), _p(st.t_next), C.c_int(B), C.c_int(d), _p(qv), _p(k_new),
                                        _p(v_new), C.c_int(r), C.c_int(mode), C.c_int(order), C.c_double(scale),
                                        C.c_int(count_self), C.c_double(delta), _p(fv), C.c_int(int(force_only_near)), _p(out), _p(lse), _p(es),
                                        _p(ep), _p(ch), _p(nt))
    return StepResult(out, lse, es, ep, ch, nt.astype(bool))


@dataclass
class BlockResult:
    out: np.ndarray           # [U][b][d]
    lse: np.ndarray           # [U][b]
    evicted_slot: np.ndarray  # [U][b] ascending slots, -1 padded
    evicted_pos: np.ndarray   # [U][b]
    choice: np.ndarray        # [U][b] the policy's own set (differs from evicted_slot only when forced)
    near_tie: np.ndarray      # [U] number of eviction iterations inside the decision margin


def block_step(st: State, Q, K_new, V_new, r, mode, scale, delta=1e-5, force_slots=None) -> BlockResult:
    """Block-wise evict-and-encode of b tokens per unit, in place on `st`.  Q, K_new, V_new: [U][b][d]."""
    Q, K_new, V_new = _f64(Q), _f64(K_new), _f64(V_new)
    U, b, d = Q.shape
    out = np.zeros((U, b, d)); lse = np.zeros((U, b))
    es = np.zeros((U, b), np.int32); ep = np.zeros((U, b), np.int32); ch = np.zeros((U, b), np.int32)
    nt = np.zeros(U, np.int32)
    fs = None if force_slots is None else _i32(force_slots)
    lib().roco_oracle_block_step_batch(C.c_int(U), _p(st.K), _p(st.V), _p(st.s), _p(st.q), _p(st.n), _p(st.pos),
                                       _p(st.live), _p(st.t_next), C.c_int(st.B), C.c_int(d), C.c_int(b), _p(Q),
                                       _p(K_new), _p(V_new), C.c_int(r), C.c_int(mode), C.c_double(scale),
                                       C.c_double(delta), _p(fs), _p(out), _p(lse), _p(es), _p(ep), _p(ch), _p(nt))
    return BlockResult(out, lse, es, ep, ch, nt)


def gqa_block_step(st: State, Q, K_new, V_new, r, mode, scale, delta=1e-5, force_slots=None) -> BlockResult:
    """Block-wise evict-and-encode of b tokens per key-value head shared by `group` query heads, in place on `st`.
    Q: [U][b][group][d]; K_new, V_new: [U][b][d].  Returns out [U][b][group][d], lse [U][b][group]."""
    Q, K_new, V_new = _f64(Q), _f64(K_new), _f64(V_new)
    U, b, group, d = Q.shape
    out = np.zeros((U, b, group, d)); lse = np.zeros((U, b, group))
    es = np.zeros((U, b), np.int32); ep = np.zeros((U, b), np.int32); ch = np.zeros((U, b), np.int32)
    nt = np.zeros(U, np.int32)
    fs = None if force_slots is None else _i32(force_slots)
    lib().roco_oracle_gqa_block_step_batch(C.c_int(U), _p(st.K), _p(st.V), _p(st.s), _p(st.q), _p(st.n), _p(st.pos),
                                           _p(st.live), _p(st.t_next), C.c_int(st.B), C.c_int(d), C.c_int(b),
                                           C.c_int(group), _p(Q), _p(K_new), _p(V_new), C.c_int(r), C.c_int(mode),
                                           C.c_double(scale), C.c_double(delta), _p(fs), _p(out), _p(lse), _p(es),
                                           _p(ep), _p(ch), _p(nt))
    return BlockResult(out, lse, es, ep, ch, nt)


def gqa_step(st: State, Q, k_new, v_new, r, mode, scale, delta=1e-5, force_victim=None) -> StepResult:
    """One decode step of U key-value heads, each shared by `group` query heads.  Q: [U][group][d];
    k_new, v_new: [U][d].  Returns out [U][group][d], lse [U][group]."""
    Q, k_new, v_new = _f64(Q), _f64(k_new), _f64(v_new)
    U, group, d = Q.shape
    out = np.zeros((U, group, d)); lse = np.zeros((U, group))
    es = np.zeros(U, np.int32); ep = np.zeros(U, np.int32); ch = np.zeros(U, np.int32); nt = np.zeros(U, np.int32)
    fv = None if force_victim is None else _i32(force_victim)
    lib().roco_oracle_gqa_step_batch(C.c_int(U), _p(st.K), _p(st.V), _p(st.s), _p(st.q), _p(st.n), _p(st.pos),
                                     _p(st.live), _p(st.t_next), C.c_int(st.B), C.c_int(d), C.c_int(group), _p(Q),
                                     _p(k_new), _p(v_new), C.c_int(r), C.c_int(mode), C.c_double(scale),
                                     C.c_double(delta), _p(fv), _p(out), _p(lse), _p(es), _p(ep), _p(ch), _p(nt))
    return StepResult(out, lse, es, ep, ch, nt.astype(bool))


def policy_step(st: State, qv, k_new, v_new, policy, r, scale, rnd=None, delta=1e-5, force_victim=None,
                order=EVICT_FIRST):
    """One decode step under one of the Table 1 policies, in place on `st`; order: EVICT_FIRST (evict, insert,
    attend) or ATTEND_FIRST (attend and update, then evict and insert).
    Returns (StepResult, quant_near [U][B] bool).  rnd: [U] uint32 draws for POLICY_RANDOM."""
    qv, k_new, v_new = _f64(qv), _f64(k_new), _f64(v_new)
    U, B, d = st.U, st.B, st.d
    out = np.zeros((U, d)); lse = np.zeros(U)
    es = np.zeros(U, np.int32); ep = np.zeros(U, np.int32); ch = np.zeros(U, np.int32); nt = np.zeros(U, np.int32)
    qn = np.zeros((U, B), np.int32)
    fv = None if force_victim is None else _i32(force_victim)
    rn = None if rnd is None else np.ascontiguousarray(rnd, dtype=np.uint32)
    lib().roco_oracle_policy_step_batch(C.c_int(U), _p(st.K), _p(st.V), _p(st.s), _p(st.q), _p(st.n), _p(st.pos),
                                        _p(st.live), _p(st.t_next), C.c_int(B), C.c_int(d), _p(qv), _p(k_new),
                                        _p(v_new), C.c_int(policy), C.c_int(r), C.c_int(order), _p(rn), C.c_double(scale),
                                        C.c_double(delta), _p(fv), _p(out), _p(lse), _p(es), _p(ep), _p(ch), _p(nt),
                                        _p(qn))
    return StepResult(out, lse, es, ep, ch, nt.astype(bool)), qn.astype(bool)


def policy_score(policy, s, q, n) -> np.ndarray:
    """Importance score of every token under a Table 1 policy, from the statistics its steps keep."""
    s, q, n = np.asarray(s, np.float64), np.asarray(q, np.float64), np.asarray(n, np.int32)
    out = np.zeros(s.shape)
    for idx in np.ndindex(s.shape):
        out[idx] = lib().roco_oracle_policy_score(int(policy), float(s[idx]), float(q[idx]), int(n[idx]))
    return out


def topb_overlap(score, pos, kept_pos, delta=1e-5, exact_ties_firm=False):
    """How many of the B = len(kept_pos) most important tokens (by `score`, ties as the eviction order has them)
    are among kept_pos.  Returns (overlap, slack): slack bounds the change under score errors within delta."""
    score, pos, kept = _f64(score), _i32(pos), _i32(kept_pos)
    slack = C.c_int(0)
    ov = lib().roco_oracle_topb_overlap(_p(score), _p(pos), C.c_int(len(score)), _p(kept), C.c_int(len(kept)),
                                        C.c_double(delta), C.c_int(int(exact_ties_firm)), C.byref(slack))
    return int(ov), int(slack.value)


def jaccard_from_overlap(overlap: int, B: int) -> float:
    """Jaccard similarity of two B-sized sets that share `overlap` elements."""
    return float(lib().roco_oracle_jaccard_equal_sets(int(overlap), int(B)))

