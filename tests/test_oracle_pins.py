"""Pins for the fp64 CPU oracle: every expected value here comes from somewhere other than the oracle
(hand-worked rationals, closed forms, library softmax/logsumexp, brute-force history recomputation,
invariants), chosen so that a dropped term, a wrong sign or index, or a transposed operand fails."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

import oracle
from oracle import ATTEND_FIRST, EVICT_FIRST, EXCLUDE_TOP_R, LOWEST_R

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_example_4tok.txt")


def load_golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, vals = line.split(":")
        out[key.strip()] = [Fraction(v) for v in vals.split()]
    return out


def hand_inputs():
    g = load_golden()
    W = [g[f"W{i}"] for i in range(4)]
    Q = np.zeros((4, 4))
    for i, row in enumerate(W):
        for j, w in enumerate(row):
            Q[i, j] = 2.0 * math.log(float(w))
    K = np.eye(4)
    V = np.arange(16, dtype=np.float64).reshape(4, 4) + 1.0
    return g, Q, K, V


def fl(xs):
    return np.array([float(x) for x in xs])


# ------------------------------------------------------------------ hand-worked example


def test_hand_example_stats():
    g, Q, K, _ = hand_inputs()
    lse, s, q, n, P = oracle.prefill_stats(Q, K, 0.5, count_self=1, want_P=True)
    for i in range(4):
        np.testing.assert_allclose(P[i, : i + 1], fl(g[f"P{i}"]), rtol=0, atol=1e-15)
        assert np.all(P[i, i + 1:] == 0)
        assert lse[i] == pytest.approx(math.log(float(sum(g[f"W{i}"]))), abs=1e-14)
    np.testing.assert_array_equal(n, [int(x) for x in g["n"]])
    np.testing.assert_allclose(s, fl(g["s"]), rtol=1e-15)
    np.testing.assert_allclose(q, fl(g["q"]), rtol=1e-15)
    mean = s / n
    np.testing.assert_allclose(mean, fl(g["mean"]), rtol=1e-15)
    np.testing.assert_allclose(q / n - mean ** 2, fl(g["var"]), atol=1e-16)


def test_hand_example_stats_noself():
    g, Q, K, _ = hand_inputs()
    _, s, q, n = oracle.prefill_stats(Q, K, 0.5, count_self=0)
    np.testing.assert_array_equal(n, [int(x) for x in g["n_noself"]])
    np.testing.assert_allclose(s, fl(g["s_noself"]), rtol=1e-15)
    np.testing.assert_allclose(q, fl(g["q_noself"]), rtol=1e-15)


def test_hand_example_prefill_eviction():
    g, Q, K, V = hand_inputs()
    res = oracle.prefill(Q[None], K[None], V[None], [4], 3, 1, EXCLUDE_TOP_R, 0.5)
    assert list(np.nonzero(~res.keep[0])[0]) == [int(g["evict_B3_exclude_r1"][0])]
    np.testing.assert_array_equal(res.state.pos[0], [0, 1, 2])
    np.testing.assert_array_equal(res.state.K[0], K[:3])
    np.testing.assert_array_equal(res.state.V[0], V[:3])
    np.testing.assert_allclose(res.state.s[0], fl(g["s"])[:3], rtol=1e-15)
    assert res.state.live[0] == 3 and res.state.t_next[0] == 4
    res = oracle.prefill(Q[None], K[None], V[None], [4], 3, 2, LOWEST_R, 0.5)
    assert list(np.nonzero(~res.keep[0])[0]) == [int(g["evict_B3_lowest_r2"][0])]
    res = oracle.prefill(Q[None], K[None], V[None], [4], 2, 1, EXCLUDE_TOP_R, 0.5)
    assert list(np.nonzero(res.keep[0])[0]) == [int(x) for x in g["keep_B2_exclude_r1"]]
    np.testing.assert_array_equal(res.state.V[0], V[[0, 2]])


def _hand_decode(order):
    g, Q, K, V = hand_inputs()
    res = oracle.prefill(Q[None], K[None], V[None], [4], 3, 1, EXCLUDE_TOP_R, 0.5)
    st = res.state
    qv = np.array([[2 * math.log(2.0), 0.0, 0.0, 0.0]])
    k_new = np.array([[0.0, 1.0, 0.0, 0.0]])
    v_new = np.array([[100.0, 200.0, 300.0, 400.0]])
    step = oracle.decode_step(st, qv, k_new, v_new, 1, EXCLUDE_TOP_R, order, 0.5)
    return g, V, v_new, st, step


def test_hand_example_decode_evict_first():
    g, V, v_new, st, step = _hand_decode(EVICT_FIRST)
    assert step.evicted_pos[0] == int(g["ef_victim_pos"][0]) and step.evicted_slot[0] == 1
    np.testing.assert_array_equal(st.pos[0], [int(x) for x in g["ef_pos"]])
    np.testing.assert_array_equal(st.n[0], [int(x) for x in g["ef_n"]])
    np.testing.assert_allclose(st.s[0], fl(g["ef_s"]), rtol=1e-15)
    np.testing.assert_allclose(st.q[0], fl(g["ef_q"]), rtol=1e-15)
    p = fl(g["ef_p"])
    np.testing.assert_allclose(step.out[0], p[0] * V[0] + p[1] * v_new[0] + p[2] * V[2], rtol=1e-14)
    assert step.lse[0] == pytest.approx(math.log(4.0), abs=1e-14)
    assert st.t_next[0] == 5 and st.live[0] == 3


def test_hand_example_decode_attend_first():
    g, V, v_new, st, step = _hand_decode(ATTEND_FIRST)
    assert step.evicted_pos[0] == int(g["af_victim_pos"][0]) and step.evicted_slot[0] == 1
    np.testing.assert_array_equal(st.pos[0], [int(x) for x in g["af_pos"]])
    np.testing.assert_array_equal(st.n[0], [int(x) for x in g["af_n"]])
    np.testing.assert_allclose(st.s[0], fl(g["af_s"]), rtol=1e-15)
    np.testing.assert_allclose(st.q[0], fl(g["af_q"]), rtol=1e-15)
    np.testing.assert_allclose(step.out[0], 0.5 * V[0] + 0.25 * V[1] + 0.25 * V[2], rtol=1e-14)
    np.testing.assert_array_equal(st.V[0, 1], v_new[0])
    # the variances the policy saw, recomputed from the golden pre-eviction statistics
    nb, sb, qb = fl(g["af_n_before_evict"]), fl(g["af_s_before_evict"]), fl(g["af_q_before_evict"])
    np.testing.assert_allclose(qb / nb - (sb / nb) ** 2, fl(g["af_var_before_evict"]), rtol=1e-13)


# ------------------------------------------------------------------ closed forms


@pytest.mark.parametrize("L", [1, 2, 7, 64])
def test_uniform_attention_harmonic_closed_form(L):
    """All keys equal => P_ij = 1/(i+1): n_j = L-j, s_j = H_L - H_j, q_j = sum_{i=j+1..L} 1/i^2."""
    rng = np.random.default_rng(L)
    K = np.tile(rng.normal(size=(1, 8)), (L, 1))
    Q = rng.normal(size=(L, 8))
    lse, s, q, n = oracle.prefill_stats(Q, K, 0.3)
    H = [Fraction(0)]
    H2 = [Fraction(0)]
    for i in range(1, L + 1):
        H.append(H[-1] + Fraction(1, i))
        H2.append(H2[-1] + Fraction(1, i * i))
    np.testing.assert_array_equal(n, [L - j for j in range(L)])
    np.testing.assert_allclose(s, [float(H[L] - H[j]) for j in range(L)], rtol=1e-13)
    np.testing.assert_allclose(q, [float(H2[L] - H2[j]) for j in range(L)], rtol=1e-13)
    z = 0.3 * Q @ K[0]
    np.testing.assert_allclose(lse, z + np.log(np.arange(1, L + 1)), rtol=1e-13, atol=1e-13)


def test_zero_query_decode_gains_one_over_live():
    U, B, d = 1, 6, 4
    rng = np.random.default_rng(0)
    st = oracle.empty_state(U, B, d)
    for t in range(10):
        before = st.s.copy()
        live_before = int(st.live[0])
        step = oracle.decode_step(st, np.zeros((U, d)), rng.normal(size=(U, d)), rng.normal(size=(U, d)),
                                  2, EXCLUDE_TOP_R, EVICT_FIRST, 0.5)
        live = int(st.live[0])
        assert live == min(live_before + 1, B)
        gain = st.s[0, :live] - np.where(np.arange(live) == (step.evicted_slot[0] if step.evicted_slot[0] >= 0
                                                              else live - 1), 0.0, before[0, :live])
        np.testing.assert_allclose(gain, 1.0 / live, rtol=1e-14)
        np.testing.assert_allclose(step.out[0], st.V[0, :live].mean(0), rtol=1e-13)


def test_uniform_attention_ties_go_to_lowest_position():
    """Bit-identical statistics: the position rule alone decides (scope boundary and victim)."""
    n = np.array([3, 3, 3, 3, 3], np.int32)
    s = np.full(5, 0.6); q = np.full(5, 0.2)
    pos = np.array([40, 10, 30, 20, 50], np.int32)
    # EXCLUDE r=2: order by (var,pos) = positions 10,20,30,40,50 -> scope {10,20,30}; victim: lowest pos = 10
    slot, _, m = oracle.select(s, q, n, pos, 2, EXCLUDE_TOP_R, delta=0.0)
    assert m == 3 and pos[slot] == 10
    # make token at position 10 the highest mean: victim is now the next lowest position in scope
    s2 = s.copy(); s2[1] = 0.9; q2 = q.copy(); q2[1] = 0.9 ** 2 / 3 + 0.2 - 0.6 ** 2 / 3
    slot, _, _ = oracle.select(s2, q2, n, pos, 2, EXCLUDE_TOP_R, delta=0.0)
    assert pos[slot] == 20
    # LOWEST r=1: scope is only the lowest (var,pos) = position 10
    slot, _, m = oracle.select(s, q, n, pos, 1, LOWEST_R, delta=0.0)
    assert m == 1 and pos[slot] == 10


# ------------------------------------------------------------------ textbook special cases


def test_budget_not_binding_is_plain_causal_attention():
    rng = np.random.default_rng(1)
    L, d, scale = 33, 16, 0.25
    Q, K, V = rng.normal(size=(3, L, d))
    res = oracle.prefill(Q[None], K[None], V[None], [L], L + 5, 4, EXCLUDE_TOP_R, scale)
    Z = scale * Q @ K.T
    Z[np.triu_indices(L, 1)] = -np.inf
    P = softmax(Z, axis=1)
    np.testing.assert_allclose(res.s_full[0], P.sum(0), rtol=1e-13)
    np.testing.assert_allclose(res.q_full[0], (P ** 2).sum(0), rtol=1e-13)
    np.testing.assert_array_equal(res.n_full[0], L - np.arange(L))
    np.testing.assert_allclose(res.lse[0], logsumexp(Z, axis=1), rtol=1e-13)
    assert res.keep[0].all() and res.state.live[0] == L
    np.testing.assert_array_equal(res.state.K[0, :L], K)
    np.testing.assert_array_equal(res.state.pos[0, :L], np.arange(L))
    assert np.all(res.state.pos[0, L:] == -1)
    # decode on the unbounded cache = ordinary attention over L+1 keys (EVICT_FIRST) or L keys (ATTEND_FIRST)
    qv, kn, vn = rng.normal(size=(3, 1, d))
    for order, Kx, Vx in ((EVICT_FIRST, np.vstack([K, kn]), np.vstack([V, vn])), (ATTEND_FIRST, K, V)):
        st = res.state.copy()
        step = oracle.decode_step(st, qv, kn, vn, 4, EXCLUDE_TOP_R, order, scale)
        z = scale * Kx @ qv[0]
        np.testing.assert_allclose(step.out[0], softmax(z) @ Vx, rtol=1e-13)
        assert step.lse[0] == pytest.approx(logsumexp(z), rel=1e-13)
        assert step.evicted_slot[0] == -1 and st.live[0] == L + 1
        expect_s = np.concatenate([P.sum(0), np.zeros(len(z) - L)]) + softmax(z)
        np.testing.assert_allclose(st.s[0, : len(z)], expect_s, rtol=1e-13)


def test_transposed_operands_would_fail():
    """Asymmetric Q/K: the statistics of (Q,K) and (K,Q) differ, and the oracle matches the former."""
    rng = np.random.default_rng(5)
    L, d = 9, 4
    Q, K = rng.normal(size=(2, L, d))
    _, s, _, _ = oracle.prefill_stats(Q, K, 0.5)
    Z = 0.5 * Q @ K.T
    Z[np.triu_indices(L, 1)] = -np.inf
    Zt = 0.5 * K @ Q.T
    Zt[np.triu_indices(L, 1)] = -np.inf
    np.testing.assert_allclose(s, softmax(Z, axis=1).sum(0), rtol=1e-13)
    assert np.abs(s - softmax(Zt, axis=1).sum(0)).max() > 1e-2


def test_prefill_equals_streamed_decode():
    """Column reduction of the causal matrix = running accumulation over decode steps (budget not binding)."""
    rng = np.random.default_rng(2)
    U, L, d, scale = 3, 20, 8, 0.35
    Q, K, V = rng.normal(size=(3, U, L, d))
    res = oracle.prefill(Q, K, V, [L] * U, L, 3, EXCLUDE_TOP_R, scale)
    st = oracle.empty_state(U, L, d)
    lses = []
    for t in range(L):
        step = oracle.decode_step(st, Q[:, t], K[:, t], V[:, t], 3, EXCLUDE_TOP_R, EVICT_FIRST, scale)
        lses.append(step.lse)
        assert np.all(step.evicted_slot == -1)
    np.testing.assert_allclose(st.s, res.state.s, rtol=1e-13)
    np.testing.assert_allclose(st.q, res.state.q, rtol=1e-13)
    np.testing.assert_array_equal(st.n, res.state.n)
    np.testing.assert_array_equal(st.pos, res.state.pos)
    np.testing.assert_allclose(np.stack(lses, 1), res.lse, rtol=1e-13)


def test_scope_modes_coincide_and_r0_is_pure_mas():
    rng = np.random.default_rng(3)
    live = 37
    n = rng.integers(1, 30, live).astype(np.int32)
    p = rng.uniform(0.01, 0.5, live)
    s = p * n
    q = (p ** 2 + rng.uniform(0, 0.01, live)) * n
    pos = rng.permutation(1000)[:live].astype(np.int32)
    for r in (0, 1, 5, 36):
        a, _, ma = oracle.select(s, q, n, pos, r, EXCLUDE_TOP_R)
        b, _, mb = oracle.select(s, q, n, pos, live - r, LOWEST_R)
        assert a == b and ma == mb == max(1, live - r)
    a, _, _ = oracle.select(s, q, n, pos, 0, EXCLUDE_TOP_R)
    assert a == int(np.argmin(s / n))


# ------------------------------------------------------------------ brute force on tiny inputs


def brute_select(hist, pos_of_slot, live, r, mode):
    """Exhaustive re-derivation from the full probability history (own code, Python floats/sorted())."""
    toks = []
    for slot in range(live):
        ps = hist[pos_of_slot[slot]]
        if not ps:
            continue
        mean = math.fsum(ps) / len(ps)
        var = max(0.0, math.fsum(x * x for x in ps) / len(ps) - mean * mean)
        toks.append((var, pos_of_slot[slot], mean, slot))
    toks.sort(key=lambda t: (t[0], t[1]))
    m = len(toks) - r if mode == EXCLUDE_TOP_R else r
    m = min(max(m, 1), len(toks))
    scope = toks[:m]
    return min(scope, key=lambda t: (t[2], t[1]))[3]


@pytest.mark.parametrize("mode,r", [(EXCLUDE_TOP_R, 2), (EXCLUDE_TOP_R, 0), (LOWEST_R, 3), (LOWEST_R, 1)])
@pytest.mark.parametrize("order", [EVICT_FIRST, ATTEND_FIRST])
@pytest.mark.parametrize("count_self", [1, 0])
def test_brute_force_history(mode, r, order, count_self):
    if order == ATTEND_FIRST and count_self == 0:
        pytest.skip("count_self only matters when the query sees its own key")
    rng = np.random.default_rng(100 * mode + 10 * r + order)
    B, d, T, scale = 6, 5, 40, 0.6
    st = oracle.empty_state(1, B, d)
    hist = {}          # token position -> list of probabilities it has received so far
    slots = []         # slot -> position
    Ks, Vs = {}, {}
    total_mass = 0.0
    for t in range(T):
        qv, kn, vn = rng.normal(size=(3, 1, d))
        Ks[t], Vs[t] = kn[0], vn[0]
        # --- brute force side
        def attend_bf(members):
            z = np.array([scale * Ks[p] @ qv[0] for p in members])
            pr = softmax(z)
            o = sum(pr[i] * Vs[p] for i, p in enumerate(members))
            for i, p in enumerate(members):
                if p == t and not count_self:
                    continue
                hist[p].append(float(pr[i]))
            return o, logsumexp(z)
        ev_bf = -1
        if order == ATTEND_FIRST and slots:
            out_bf, lse_bf = attend_bf(list(slots))
        if len(slots) == B:
            ev_bf = brute_select(hist, slots, B, r, mode)
            slots[ev_bf] = t
        else:
            slots.append(t)
        hist[t] = []
        if order == EVICT_FIRST:
            out_bf, lse_bf = attend_bf(list(slots))
        # --- oracle side
        step = oracle.decode_step(st, qv, kn, vn, r, mode, order, scale, count_self=count_self, delta=1e-9)
        assert not step.near_tie[0]
        assert step.evicted_slot[0] == ev_bf
        live = int(st.live[0])
        assert live == len(slots) <= B
        np.testing.assert_array_equal(st.pos[0, :live], slots)
        if order == EVICT_FIRST or t > 0:
            np.testing.assert_allclose(step.out[0], out_bf, rtol=1e-12, atol=1e-14)
            assert step.lse[0] == pytest.approx(lse_bf, rel=1e-12)
        for slot, p in enumerate(slots):
            assert st.n[0, slot] == len(hist[p])
            assert st.s[0, slot] == pytest.approx(math.fsum(hist[p]), rel=1e-12, abs=1e-300)
            assert st.q[0, slot] == pytest.approx(math.fsum(x * x for x in hist[p]), rel=1e-12, abs=1e-300)
            np.testing.assert_array_equal(st.K[0, slot], Ks[p])
            np.testing.assert_array_equal(st.V[0, slot], Vs[p])


# ------------------------------------------------------------------ invariants


@pytest.mark.parametrize("mode,r", [(EXCLUDE_TOP_R, 4), (LOWEST_R, 4)])
@pytest.mark.parametrize("order", [EVICT_FIRST, ATTEND_FIRST])
def test_invariants_over_a_run(mode, r, order):
    rng = np.random.default_rng(7)
    U, L, B, d, scale, T = 4, 24, 12, 8, 0.35, 30
    Q, K, V = rng.normal(size=(3, U, L, d))
    res = oracle.prefill(Q, K, V, [L] * U, B, r, mode, scale)
    st = res.state
    np.testing.assert_allclose(res.s_full.sum(1), L, rtol=1e-13)          # every query's row sums to 1
    assert np.all(res.keep.sum(1) == B) and np.all(st.live == B)
    evicted_mass = (res.s_full * ~res.keep).sum(1)
    for step_i in range(T):
        before = st.copy()
        qv, kn, vn = rng.normal(size=(3, U, d))
        step = oracle.decode_step(st, qv, kn, vn, r, mode, order, scale)
        t = L + step_i
        assert np.all(st.live <= B)                                        # Sec. 3: n <= B at every step
        for u in range(U):
            e = step.evicted_slot[u]
            assert e >= 0 and step.evicted_pos[u] == before.pos[u, e]
            # the victim lies in the scope and has the lowest mean there (checked on the stats the policy saw)
            ref = st if order == ATTEND_FIRST else before
            s_seen = before.s[u].copy(); q_seen = before.q[u].copy(); n_seen = before.n[u].copy()
            if order == ATTEND_FIRST:
                z = scale * before.K[u] @ qv[u]
                p = softmax(z)
                s_seen += p; q_seen += p * p; n_seen += 1
            mean = s_seen / n_seen
            var = np.maximum(0, q_seen / n_seen - mean ** 2)
            order_v = sorted(range(B), key=lambda j: (var[j], before.pos[u, j]))
            m = B - r if mode == EXCLUDE_TOP_R else r
            scope = order_v[:m]
            assert e in scope and mean[e] == min(mean[j] for j in scope)
            evicted_mass[u] += s_seen[e]
            assert len(set(st.pos[u])) == B                                # live positions are distinct
            assert st.pos[u, e] == t
        np.testing.assert_allclose(st.s.sum(1) + evicted_mass, t + 1, rtol=1e-12)   # mass grows by 1 per step
        assert np.all(st.q <= st.s + 1e-15) and np.all(st.s <= st.n + 1e-12) and np.all(st.q >= 0)
        nn = np.maximum(st.n, 1)
        mean = st.s / nn
        var = st.q / nn - mean ** 2
        assert np.all(var >= -1e-15) and np.all(var <= mean * (1 - mean) + 1e-15)
        # Count is redundant with position
        expect_n = t - st.pos + 1
        if order == ATTEND_FIRST:
            expect_n = np.where(st.pos >= L, t - st.pos, expect_n)
        np.testing.assert_array_equal(st.n, expect_n)


# ------------------------------------------------------------------ select-to-budget


@pytest.mark.parametrize("seed", range(5))
def test_onepass_equals_iterated(seed):
    rng = np.random.default_rng(seed)
    L, d = 48, 8
    Q, K = rng.normal(size=(2, L, d))
    _, s, q, n = oracle.prefill_stats(Q, K, 0.5)
    for B, r in ((20, 6), (47, 1), (10, 10), (30, 0)):
        it = oracle.select_to_budget_iterated(s, q, n, B, r, EXCLUDE_TOP_R)
        op, unc = oracle.select_to_budget_onepass(s, q, n, B, r, delta=1e-12)
        np.testing.assert_array_equal(it, op)
        assert it.sum() == B
        # brute force: protect top-r (var,pos), evict L-B lowest (mean,pos) of the rest
        mean = s / n; var = np.maximum(0, q / n - mean ** 2)
        by_var = sorted(range(L), key=lambda j: (var[j], j))
        rest = by_var[: L - r]
        gone = sorted(rest, key=lambda j: (mean[j], j))[: L - B]
        assert set(np.nonzero(~it)[0]) == set(gone)


def test_iterated_lowest_r_matches_bruteforce():
    rng = np.random.default_rng(11)
    L, d, B, r = 30, 6, 12, 5
    Q, K = rng.normal(size=(2, L, d))
    _, s, q, n = oracle.prefill_stats(Q, K, 0.5)
    keep = oracle.select_to_budget_iterated(s, q, n, B, r, LOWEST_R)
    mean = s / n; var = np.maximum(0, q / n - mean ** 2)
    alive = list(range(L))
    while len(alive) > B:
        scope = sorted(alive, key=lambda j: (var[j], j))[:r]
        alive.remove(min(scope, key=lambda j: (mean[j], j)))
    assert sorted(np.nonzero(keep)[0]) == alive


def test_uncertain_flags_mark_near_boundary_tokens():
    n = np.full(6, 4, np.int32)
    mean = np.array([0.10, 0.20, 0.2000001, 0.30, 0.40, 0.50])
    var = np.array([0.01, 0.02, 0.03, 0.04, 0.05, 0.9])
    s = mean * 4; q = (var + mean ** 2) * 4
    keep, unc = oracle.select_to_budget_onepass(s, q, n, 4, 1, delta=1e-5)   # evict 2 of the 5 unprotected
    assert list(np.nonzero(~keep)[0]) == [0, 1]
    assert list(np.nonzero(unc)[0]) == [1, 2]                                # the eviction boundary is a near-tie
    keep, unc = oracle.select_to_budget_onepass(s, q, n, 4, 1, delta=1e-9)
    assert not unc.any()


def test_near_tie_flags():
    n = np.full(4, 10, np.int32)
    pos = np.arange(4, dtype=np.int32)
    mean = np.array([0.2, 0.2 * (1 + 1e-7), 0.3, 0.4])
    var = np.array([0.01, 0.02, 0.03, 0.5])
    s = mean * 10; q = (var + mean ** 2) * 10
    slot, near, _ = oracle.select(s, q, n, pos, 1, EXCLUDE_TOP_R, delta=1e-5)
    assert slot == 0 and near                                   # runner-up within the margin
    slot, near, _ = oracle.select(s, q, n, pos, 1, EXCLUDE_TOP_R, delta=1e-9)
    assert slot == 0 and not near
    # victim on the scope boundary: two variances a hair apart, scope of 1
    var2 = np.array([0.02, 0.02 * (1 + 1e-7), 0.03, 0.5])
    q2 = (var2 + mean ** 2) * 10
    slot, near, m = oracle.select(s, q2, n, pos, 1, LOWEST_R, delta=1e-5)
    assert m == 1 and slot == 0 and near
    # an outsider with lower mean sits just outside the scope
    mean3 = np.array([0.3, 0.1, 0.35, 0.4]); var3 = np.array([0.01, 0.0100000001, 0.2, 0.5])
    slot, near, _ = oracle.select(mean3 * 10, (var3 + mean3 ** 2) * 10, n, pos, 1, LOWEST_R, delta=1e-5)
    assert slot == 0 and near
    slot, near, _ = oracle.select(mean3 * 10, (var3 + mean3 ** 2) * 10, n, pos, 1, LOWEST_R, delta=1e-12)
    assert slot == 0 and not near


def test_force_victim_and_empty_cases():
    rng = np.random.default_rng(4)
    U, B, d = 2, 3, 4
    st = oracle.empty_state(U, B, d)
    step = oracle.decode_step(st, *rng.normal(size=(3, U, d)), 1, EXCLUDE_TOP_R, ATTEND_FIRST, 0.5)
    assert np.all(step.out == 0) and np.all(np.isneginf(step.lse))     # nothing cached yet
    for _ in range(3):
        oracle.decode_step(st, *rng.normal(size=(3, U, d)), 1, EXCLUDE_TOP_R, EVICT_FIRST, 0.5)
    own = oracle.decode_step(st.copy(), *rng.normal(size=(3, U, d)), 1, EXCLUDE_TOP_R, EVICT_FIRST, 0.5).choice
    forced = (own + 1) % B
    step = oracle.decode_step(st, *rng.normal(size=(3, U, d)), 1, EXCLUDE_TOP_R, EVICT_FIRST, 0.5,
                              force_victim=forced)
    np.testing.assert_array_equal(step.evicted_slot, forced)


def test_ragged_prompts_in_one_batch():
    rng = np.random.default_rng(9)
    U, Lmax, d, B = 3, 16, 4, 6
    lens = [16, 5, 9]
    Q, K, V = rng.normal(size=(3, U, Lmax, d))
    res = oracle.prefill(Q, K, V, lens, B, 2, EXCLUDE_TOP_R, 0.5)
    for u, L in enumerate(lens):
        solo = oracle.prefill(Q[u:u + 1, :L], K[u:u + 1, :L], V[u:u + 1, :L], [L], B, 2, EXCLUDE_TOP_R, 0.5)
        np.testing.assert_array_equal(res.state.pos[u], solo.state.pos[0])
        np.testing.assert_array_equal(res.state.s[u], solo.state.s[0])
        assert res.state.live[u] == min(L, B) and res.state.t_next[u] == L


def test_attention_row_is_library_softmax():
    rng = np.random.default_rng(21)
    K = rng.normal(size=(37, 8)); qv = rng.normal(size=8)
    p, lse = oracle.attention_row(qv, K, 0.4)
    np.testing.assert_allclose(p, softmax(0.4 * K @ qv), rtol=1e-13)
    assert lse == pytest.approx(logsumexp(0.4 * K @ qv), rel=1e-13)


# ---------------------------------------------------------------- prompt attention output (Eq. 1, causal)

def test_prompt_attention_constant_values_pass_through():
    """Probabilities of a row sum to one, so identical value rows come back unchanged."""
    rng = np.random.default_rng(31)
    L, d = 23, 8
    Q, K = rng.normal(size=(L, d)), rng.normal(size=(L, d))
    v = rng.normal(size=d)
    out, _ = oracle.prompt_attention_rows(Q, K, np.tile(v, (L, 1)), list(range(L)), 0.3)
    np.testing.assert_allclose(out, np.tile(v, (L, 1)), rtol=1e-12, atol=1e-14)


def test_prompt_attention_zero_queries_give_running_mean():
    """Q = 0 makes every causal row uniform: out_i is the mean of V_0..V_i (a closed form that also pins the mask)."""
    rng = np.random.default_rng(32)
    L, d = 19, 4
    K, V = rng.normal(size=(L, d)), rng.normal(size=(L, d))
    out, lse = oracle.prompt_attention_rows(np.zeros((L, d)), K, V, list(range(L)), 1.0)
    want = np.cumsum(V, axis=0) / np.arange(1, L + 1)[:, None]
    np.testing.assert_allclose(out, want, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse, np.log(np.arange(1, L + 1)), rtol=1e-12, atol=1e-14)


def test_prompt_attention_dominant_key_selects_its_value_and_future_is_masked():
    """One key aligned with every query and far larger than the rest takes all the probability -- but only for
    the rows at or after its position; earlier rows must not see it."""
    L, d, hot = 12, 4, 5
    Q = np.tile(np.array([1.0, 0, 0, 0]), (L, 1))
    K = np.zeros((L, d)); K[hot, 0] = 60.0
    V = np.arange(L * d, dtype=float).reshape(L, d)
    out, _ = oracle.prompt_attention_rows(Q, K, V, list(range(L)), 1.0)
    for i in range(L):
        if i >= hot:
            np.testing.assert_allclose(out[i], V[hot], rtol=1e-12)
        else:
            np.testing.assert_allclose(out[i], V[: i + 1].mean(axis=0), rtol=1e-12)


def test_prompt_attention_last_row_equals_decode_attention_over_the_prompt():
    """The last prompt row attends over the whole prompt: same output as one ATTEND_FIRST-style read of a cache
    that holds every prompt token (cross-check against the decode-step oracle's attention)."""
    rng = np.random.default_rng(33)
    L, d = 17, 8
    Q, K, V = rng.normal(size=(L, d)), rng.normal(size=(L, d)), rng.normal(size=(L, d))
    out, lse = oracle.prompt_attention_rows(Q, K, V, [L - 1], 0.35)
    p, l2 = oracle.attention_row(Q[L - 1], K, 0.35)
    np.testing.assert_allclose(out[0], p @ V, rtol=1e-12)
    assert lse[0] == pytest.approx(l2, rel=1e-14)
