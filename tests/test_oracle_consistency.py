"""Pins for the oracle's consistency diagnostic (Sec. 4.3, preliminary experiments: Jaccard similarity between the
top-B tokens of a budgeted cache and those of a full cache).  Expected values are hand cases, Python brute force
and a bound that follows from the set sizes."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
import workloads as W
from oracle import POLICY_H2O, POLICY_MAS_WINDOW, POLICY_ROCO, POLICY_SCISSORHANDS, POLICY_TOVA


def test_policy_scores_hand_values():
    s, q, n = 0.75, 0.3125, 2
    assert oracle.policy_score(POLICY_H2O, [s], [q], [n])[0] == 0.75            # accumulated probability
    assert oracle.policy_score(POLICY_SCISSORHANDS, [s], [3.0], [n])[0] == 3.0  # quantised count, kept in q
    assert oracle.policy_score(POLICY_TOVA, [s], [0.125], [n])[0] == 0.125      # last probability, kept in q
    assert oracle.policy_score(POLICY_MAS_WINDOW, [s], [q], [n])[0] == 0.375    # mean attention score
    assert oracle.policy_score(POLICY_ROCO, [s], [q], [n])[0] == 0.375
    assert oracle.policy_score(POLICY_MAS_WINDOW, [0.0], [0.0], [0])[0] == 0.0  # never attended yet


def test_topb_hand_case_with_a_tied_pair():
    score, pos = [0.1, 0.5, 0.3, 0.5], [0, 1, 2, 3]
    # eviction order (score, position): 0, 2, 1, 3 -> top-2 = {1, 3}, top-1 = {3}
    assert oracle.topb_overlap(score, pos, [1, 3])[0] == 2
    assert oracle.topb_overlap(score, pos, [3, 0])[0] == 1
    assert oracle.topb_overlap(score, pos, [3])[0] == 1
    assert oracle.topb_overlap(score, pos, [1])[0] == 0
    assert oracle.topb_overlap(score, pos, [0, 1, 2, 3])[0] == 4


def test_identical_scores_leave_the_latest_positions():
    pos = np.array([5, 2, 9, 7, 1, 8], np.int32)
    score = np.full(6, 0.25)
    for B in (1, 2, 3, 5):
        top = sorted(pos)[-B:]
        assert oracle.topb_overlap(score, pos, top)[0] == B
        others = sorted(pos)[:B]
        assert oracle.topb_overlap(score, pos, others)[0] == len(set(top) & set(others))


def test_topb_against_python_sorting():
    rng = np.random.default_rng(5)
    for _ in range(50):
        live, B = 40, int(rng.integers(1, 40))
        score = rng.integers(0, 6, live).astype(float) if rng.random() < 0.5 else rng.random(live)
        pos = rng.permutation(100)[:live].astype(np.int32)
        kept = rng.permutation(pos)[:B]
        order = sorted(range(live), key=lambda j: (score[j], pos[j]))
        top = {int(pos[j]) for j in order[live - B:]}
        assert oracle.topb_overlap(score, pos, kept)[0] == len(top & {int(x) for x in kept})


def test_slack_counts_tokens_that_may_cross_the_boundary():
    pos = np.arange(6, dtype=np.int32)
    score = np.array([0.10, 0.2000000, 0.2000001, 0.30, 0.40, 0.50])
    # B = 4: boundary between tokens 1 (out) and 2 (in), 5e-7 relative apart
    assert oracle.topb_overlap(score, pos, [2, 3, 4, 5], delta=1e-5) == (4, 1)
    assert oracle.topb_overlap(score, pos, [2, 3, 4, 5], delta=1e-8) == (4, 0)
    # B = 3: boundary between 0.2000001 and 0.30: firm
    assert oracle.topb_overlap(score, pos, [3, 4, 5], delta=1e-5) == (3, 0)
    # an exact tie across the boundary is inside any margin, unless the scores are integer counts
    tied = np.array([1.0, 2.0, 2.0, 2.0, 3.0, 4.0])
    assert oracle.topb_overlap(tied, pos, [2, 3, 4, 5], delta=1e-5) == (4, 1)
    assert oracle.topb_overlap(tied, pos, [2, 3, 4, 5], delta=1e-5, exact_ties_firm=True) == (4, 0)
    assert oracle.topb_overlap(tied, pos, [3, 4, 5], delta=1e-5) == (3, 1)        # 1 in, 2 out on the tie


def test_jaccard_of_equal_sized_sets():
    assert oracle.jaccard_from_overlap(7, 7) == 1.0
    assert oracle.jaccard_from_overlap(0, 7) == 0.0
    assert oracle.jaccard_from_overlap(1, 3) == float(Fraction(1, 5))
    assert oracle.jaccard_from_overlap(2, 3) == 0.5


@pytest.mark.parametrize("policy", [POLICY_MAS_WINDOW, POLICY_H2O, POLICY_SCISSORHANDS, POLICY_TOVA])
def test_budget_one_short_of_the_sequence(policy):
    """A budgeted cache of T - 1 slots has evicted exactly one of T tokens: its retained set and the full cache's
    top-(T-1) can differ by at most one token, so the Jaccard similarity is at least (B - 1) / (B + 1); and a
    budget that holds everything gives exactly 1."""
    w = W.scaled(W.TOY, heads=2)
    T, d = 24, w.d
    for B in (T - 1, T):
        full, small = oracle.empty_state(w.U, T, d), oracle.empty_state(w.U, B, d)
        for t in range(T):
            q, k, v = (x[0].double().numpy() for x in W.decode_tokens(w, t, [t], "cpu"))
            for st in (full, small):
                oracle.policy_step(st, q, k, v, policy, 0, w.scale)
        for u in range(w.U):
            sc = oracle.policy_score(policy, full.s[u], full.q[u], full.n[u])
            ov, _ = oracle.topb_overlap(sc, full.pos[u], small.pos[u, :B])
            j = oracle.jaccard_from_overlap(ov, B)
            assert j == 1.0 if B == T else j >= (B - 1) / (B + 1) - 1e-12
