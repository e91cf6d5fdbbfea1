"""Pins for the oracle's other Table 1 policies: each is re-derived from the full probability history with plain
Python (library softmax, exhaustive min), plus structural facts (recency keeps the last B tokens, StreamLLM keeps
the four sinks, the RoCo policy is the already pinned step)."""
import numpy as np
import pytest
from scipy.special import softmax

import oracle as O


def brute_policy_run(policy, r, B, d, T, scale, seed, order=O.EVICT_FIRST):
    """Replays T steps from the full probability history: hist[p] = [(probability, cache size)] of every query that
    attended token p.  EVICT_FIRST: decide on the history so far, insert, attend.  ATTEND_FIRST: attend over the
    cache as it stands (the new token is not in it), extend the history, decide on that, insert."""
    rng = np.random.default_rng(seed)
    st = O.empty_state(1, B, d)
    hist, slots, Ks, Vs = {}, [], {}, {}

    def attend(qv):
        z = np.array([scale * Ks[p] @ qv[0] for p in slots])
        pr = softmax(z) if len(slots) else np.zeros(0)
        for i, p in enumerate(slots):
            hist[p].append((float(pr[i]), len(slots)))
        return sum((pr[i] * Vs[p] for i, p in enumerate(slots)), np.zeros(d))

    def victim(t, rnd):
        def score(j):
            h = hist[slots[j]]
            if policy == O.POLICY_H2O: return sum(x for x, _ in h)
            if policy == O.POLICY_SCISSORHANDS: return float(sum(1 for x, m in h if x * m > 1.0))
            if policy == O.POLICY_TOVA: return h[-1][0]
            if policy == O.POLICY_MAS_WINDOW: return sum(x for x, _ in h) / len(h)
            return 0.0
        cand = list(range(B))
        if policy in (O.POLICY_H2O, O.POLICY_SCISSORHANDS, O.POLICY_MAS_WINDOW):
            cand = [j for j in cand if slots[j] < t - r]
        if policy == O.POLICY_STREAMLLM:
            cand = [j for j in cand if slots[j] >= 4]
        if policy == O.POLICY_RANDOM:
            return int(rnd[0]) % B
        return min(cand, key=lambda j: (score(j), slots[j]))

    for t in range(T):
        qv, kn, vn = rng.normal(size=(3, 1, d))
        rnd = rng.integers(0, 2 ** 32, 1, dtype=np.uint64).astype(np.uint32)
        want_out = attend(qv) if order == O.ATTEND_FIRST else None
        Ks[t], Vs[t] = kn[0], vn[0]
        ev = -1
        if len(slots) == B:
            ev = victim(t, rnd)
            slots[ev] = t
        else:
            slots.append(t)
        hist[t] = []
        if order == O.EVICT_FIRST:
            want_out = attend(qv)
        res, _ = O.policy_step(st, qv, kn, vn, policy, r, scale, rnd=rnd, delta=1e-12, order=order)
        assert res.evicted_slot[0] == ev, (t, policy)
        np.testing.assert_allclose(res.out[0], want_out, rtol=1e-12, atol=1e-300)
        np.testing.assert_array_equal(st.pos[0, :len(slots)], slots)
        for j, p in enumerate(slots):
            h = hist[p]
            assert st.n[0, j] == len(h)
            assert st.s[0, j] == pytest.approx(sum(x for x, _ in h), rel=1e-12)
            if policy == O.POLICY_SCISSORHANDS:
                assert st.q[0, j] == sum(1 for x, m in h if x * m > 1.0)
            elif policy == O.POLICY_TOVA:
                assert st.q[0, j] == pytest.approx(h[-1][0] if h else 0.0, rel=1e-12)
            else:
                assert st.q[0, j] == pytest.approx(sum(x * x for x, _ in h), rel=1e-12)
    return st


@pytest.mark.parametrize("policy", [O.POLICY_RANDOM, O.POLICY_RECENCY, O.POLICY_STREAMLLM, O.POLICY_SCISSORHANDS,
                                    O.POLICY_H2O, O.POLICY_TOVA, O.POLICY_MAS_WINDOW])
@pytest.mark.parametrize("order", [O.EVICT_FIRST, O.ATTEND_FIRST])
def test_policy_brute_force(policy, order):
    brute_policy_run(policy, r=3, B=8, d=5, T=40, scale=0.6, seed=policy, order=order)


def test_roco_policy_in_the_other_order_is_the_pinned_decode_step():
    rng = np.random.default_rng(7)
    a, b = O.empty_state(2, 7, 4), O.empty_state(2, 7, 4)
    for _ in range(20):
        qv, kn, vn = rng.normal(size=(3, 2, 4))
        ra = O.decode_step(a, qv, kn, vn, 2, O.EXCLUDE_TOP_R, O.ATTEND_FIRST, 0.5)
        rb, _ = O.policy_step(b, qv, kn, vn, O.POLICY_ROCO, 2, 0.5, order=O.ATTEND_FIRST)
        np.testing.assert_array_equal(ra.evicted_slot, rb.evicted_slot)
        np.testing.assert_array_equal(ra.out, rb.out)
        np.testing.assert_array_equal(a.s, b.s)
        np.testing.assert_array_equal(a.q, b.q)


def test_recency_keeps_the_last_B_and_streamllm_keeps_the_sinks():
    st = brute_policy_run(O.POLICY_RECENCY, 0, 6, 4, 25, 0.5, 1)
    assert sorted(st.pos[0]) == list(range(19, 25))
    st = brute_policy_run(O.POLICY_STREAMLLM, 0, 8, 4, 30, 0.5, 2)
    assert sorted(st.pos[0]) == [0, 1, 2, 3] + list(range(26, 30))


def test_roco_policy_is_the_pinned_decode_step():
    rng = np.random.default_rng(5)
    a, b = O.empty_state(2, 7, 4), O.empty_state(2, 7, 4)
    for _ in range(20):
        qv, kn, vn = rng.normal(size=(3, 2, 4))
        ra = O.decode_step(a, qv, kn, vn, 2, O.EXCLUDE_TOP_R, O.EVICT_FIRST, 0.5)
        rb, _ = O.policy_step(b, qv, kn, vn, O.POLICY_ROCO, 2, 0.5)
        np.testing.assert_array_equal(ra.evicted_slot, rb.evicted_slot)
        np.testing.assert_array_equal(a.s, b.s)
        np.testing.assert_array_equal(a.q, b.q)


def test_local_window_protects_the_recent_tokens():
    """H2O with r = B - 1: only the single token outside the window is evictable, whatever its score."""
    rng = np.random.default_rng(6)
    B = 6
    st = O.empty_state(1, B, 4)
    for t in range(20):
        res, _ = O.policy_step(st, *rng.normal(size=(3, 1, 4)), O.POLICY_H2O, B - 1, 0.5)
        if t >= B:
            assert res.evicted_pos[0] == t - B          # the oldest one is the only candidate


def test_quantisation_near_flag():
    st = O.empty_state(1, 4, 2)
    for _ in range(3):
        O.policy_step(st, np.zeros((1, 2)), np.ones((1, 2)), np.ones((1, 2)), O.POLICY_SCISSORHANDS, 1, 0.5)
    # zero query: every probability equals the average exactly -> all flagged, none counted as above average
    res, qn = O.policy_step(st, np.zeros((1, 2)), np.ones((1, 2)), np.ones((1, 2)), O.POLICY_SCISSORHANDS, 1, 0.5)
    assert qn[0].all() and np.all(st.q[0] == 0)
