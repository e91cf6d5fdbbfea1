"""Pins for the oracle's block-wise evict-and-encode step (Sec. 5.3, App. B) and grouped-query step (Sec. 5.3,
App. A): special cases that reduce to the already pinned single-token step, brute force with library softmax
and exhaustive sorting, and invariants."""
import math

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

import oracle
from oracle import EVICT_FIRST, EXCLUDE_TOP_R, LOWEST_R


def filled_state(rng, U, B, d, live, scale=0.4):
    st = oracle.empty_state(U, B, d)
    for _ in range(live):
        oracle.decode_step(st, *rng.normal(size=(3, U, d)), 2, EXCLUDE_TOP_R, EVICT_FIRST, scale)
    return st


def brute_victims(s, q, n, pos, live, need, r, mode):
    alive = list(range(live))
    gone = []
    for _ in range(need):
        mean = {j: s[j] / n[j] for j in alive}
        var = {j: max(0.0, q[j] / n[j] - mean[j] ** 2) for j in alive}
        order = sorted(alive, key=lambda j: (var[j], pos[j]))
        m = len(alive) - r if mode == EXCLUDE_TOP_R else r
        m = min(max(m, 1), len(alive))
        v = min(order[:m], key=lambda j: (mean[j], pos[j]))
        alive.remove(v)
        gone.append(v)
    return sorted(gone)


@pytest.mark.parametrize("mode,r", [(EXCLUDE_TOP_R, 2), (LOWEST_R, 4)])
def test_block_of_one_is_the_single_token_step(mode, r):
    rng = np.random.default_rng(0)
    U, B, d = 3, 9, 6
    a = filled_state(rng, U, B, d, 12)
    b = a.copy()
    for _ in range(6):
        qv, kn, vn = rng.normal(size=(3, U, d))
        ra = oracle.decode_step(a, qv, kn, vn, r, mode, EVICT_FIRST, 0.4)
        rb = oracle.block_step(b, qv[:, None], kn[:, None], vn[:, None], r, mode, 0.4)
        np.testing.assert_array_equal(ra.evicted_slot, rb.evicted_slot[:, 0])
        np.testing.assert_allclose(ra.out, rb.out[:, 0], rtol=1e-14)
        np.testing.assert_allclose(ra.lse, rb.lse[:, 0], rtol=1e-14)
        for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
            np.testing.assert_allclose(getattr(a, name), getattr(b, name), rtol=1e-14)


def test_block_without_eviction_is_sequential_decoding():
    """While the buffer has room nothing is evicted, and causal attention inside the block is exactly what
    b single-token steps compute."""
    rng = np.random.default_rng(1)
    U, B, d, b = 2, 40, 5, 7
    a = filled_state(rng, U, B, d, 10)
    c = a.copy()
    Q, Kn, Vn = rng.normal(size=(3, U, b, d))
    rb = oracle.block_step(c, Q, Kn, Vn, 3, EXCLUDE_TOP_R, 0.4)
    assert np.all(rb.evicted_slot == -1)
    for i in range(b):
        ra = oracle.decode_step(a, Q[:, i], Kn[:, i], Vn[:, i], 3, EXCLUDE_TOP_R, EVICT_FIRST, 0.4)
        np.testing.assert_allclose(ra.out, rb.out[:, i], rtol=1e-13)
        np.testing.assert_allclose(ra.lse, rb.lse[:, i], rtol=1e-13)
    for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
        np.testing.assert_allclose(getattr(a, name), getattr(c, name), rtol=1e-13)


@pytest.mark.parametrize("mode,r", [(EXCLUDE_TOP_R, 3), (EXCLUDE_TOP_R, 0), (LOWEST_R, 5)])
@pytest.mark.parametrize("b", [2, 4, 5])
def test_block_step_brute_force(mode, r, b):
    rng = np.random.default_rng(10 * b + r)
    U, B, d, scale = 1, 12, 6, 0.5
    st = filled_state(rng, U, B, d, B - 1, scale)          # one free slot: need = b - 1 evictions, then b
    for step in range(3):
        before = st.copy()
        Q, Kn, Vn = rng.normal(size=(3, U, b, d))
        res = oracle.block_step(st, Q, Kn, Vn, r, mode, scale, delta=1e-9)
        live0, t0 = int(before.live[0]), int(before.t_next[0])
        need = max(0, live0 + b - B)
        gone = brute_victims(before.s[0], before.q[0], before.n[0], before.pos[0], live0, need, r, mode)
        assert list(res.evicted_slot[0][:need]) == gone and np.all(res.evicted_slot[0][need:] == -1)
        assert list(res.evicted_pos[0][:need]) == [before.pos[0][j] for j in gone]
        targets = sorted(gone + list(range(live0, live0 + b - need)))
        live1 = live0 - need + b
        assert st.live[0] == live1 and st.t_next[0] == t0 + b
        Kc, Vc = before.K[0].copy(), before.V[0].copy()
        s, q, n = before.s[0].copy(), before.q[0].copy(), before.n[0].copy()
        for i, slot in enumerate(targets):
            Kc[slot], Vc[slot] = Kn[0, i], Vn[0, i]
            s[slot] = q[slot] = 0.0
            n[slot] = 0
            assert st.pos[0, slot] == t0 + i
        for i in range(b):
            members = [j for j in range(live1) if j not in targets[i + 1:]]
            z = scale * Kc[members] @ Q[0, i]
            p = softmax(z)
            np.testing.assert_allclose(res.out[0, i], p @ Vc[members], rtol=1e-12)
            assert res.lse[0, i] == pytest.approx(logsumexp(z), rel=1e-12)
            s[members] += p; q[members] += p * p; n[members] += 1
        np.testing.assert_allclose(st.s[0, :live1], s[:live1], rtol=1e-12)
        np.testing.assert_allclose(st.q[0, :live1], q[:live1], rtol=1e-12)
        np.testing.assert_array_equal(st.n[0, :live1], n[:live1])
        np.testing.assert_array_equal(st.K[0, :live1], Kc[:live1])
        # every query's probabilities sum to 1: the mass that left with the victims plus the mass kept grows by b
        lost = before.s[0][gone].sum()
        assert st.s[0, :live1].sum() + lost == pytest.approx(before.s[0, :live0].sum() + b, rel=1e-12)


def test_gqa_group_of_one_and_identical_heads_reduce_to_the_single_head_step():
    rng = np.random.default_rng(3)
    U, B, d = 2, 8, 6
    a = filled_state(rng, U, B, d, 11)
    b1, b4 = a.copy(), a.copy()
    for _ in range(5):
        qv, kn, vn = rng.normal(size=(3, U, d))
        ra = oracle.decode_step(a, qv, kn, vn, 2, EXCLUDE_TOP_R, EVICT_FIRST, 0.4)
        r1 = oracle.gqa_step(b1, qv[:, None], kn, vn, 2, EXCLUDE_TOP_R, 0.4)
        r4 = oracle.gqa_step(b4, np.repeat(qv[:, None], 4, 1), kn, vn, 2, EXCLUDE_TOP_R, 0.4)
        np.testing.assert_array_equal(ra.evicted_slot, r1.evicted_slot)
        np.testing.assert_array_equal(ra.evicted_slot, r4.evicted_slot)
        np.testing.assert_allclose(r1.out[:, 0], ra.out, rtol=1e-14)
        for g in range(4):
            np.testing.assert_allclose(r4.out[:, g], ra.out, rtol=1e-14)
        for name in ("s", "q", "n", "pos"):
            np.testing.assert_allclose(getattr(b1, name), getattr(a, name), rtol=1e-14)
            np.testing.assert_allclose(getattr(b4, name), getattr(a, name), rtol=1e-13)


@pytest.mark.parametrize("group", [2, 4, 8])
def test_gqa_brute_force_group_mean(group):
    rng = np.random.default_rng(group)
    U, B, d, scale = 1, 10, 5, 0.5
    st = filled_state(rng, U, B, d, B + 3, scale)
    for _ in range(4):
        before = st.copy()
        Q = rng.normal(size=(U, group, d)); kn, vn = rng.normal(size=(2, U, d))
        res = oracle.gqa_step(st, Q, kn, vn, 3, EXCLUDE_TOP_R, scale, delta=1e-9)
        e = brute_victims(before.s[0], before.q[0], before.n[0], before.pos[0], B, 1, 3, EXCLUDE_TOP_R)[0]
        assert res.evicted_slot[0] == e
        Kc, Vc = before.K[0].copy(), before.V[0].copy()
        Kc[e], Vc[e] = kn[0], vn[0]
        P = softmax(scale * Q[0] @ Kc.T, axis=1)                      # [group][B]
        np.testing.assert_allclose(res.out[0], P @ Vc, rtol=1e-12)
        np.testing.assert_allclose(res.lse[0], logsumexp(scale * Q[0] @ Kc.T, axis=1), rtol=1e-12)
        pbar = P.mean(0)
        s, q, n = before.s[0].copy(), before.q[0].copy(), before.n[0].copy()
        s[e] = q[e] = 0.0; n[e] = 0
        np.testing.assert_allclose(st.s[0], s + pbar, rtol=1e-12)
        np.testing.assert_allclose(st.q[0], q + pbar ** 2, rtol=1e-12)
        np.testing.assert_array_equal(st.n[0], n + 1)
        assert pbar.sum() == pytest.approx(1.0, rel=1e-13)            # the group mean is still a distribution


# ------------------------------------------------ block-wise eviction on a grouped-query model (App. B, Table 9)

def test_grouped_block_with_one_head_is_the_block_step_and_with_one_token_the_gqa_step():
    rng = np.random.default_rng(21)
    U, B, d = 2, 12, 5
    base = filled_state(rng, U, B, d, 14)
    # group = 1  ==  block step
    a, b_ = base.copy(), base.copy()
    for _ in range(3):
        Q, Kn, Vn = rng.normal(size=(3, U, 3, d))
        ra = oracle.block_step(a, Q, Kn, Vn, 2, EXCLUDE_TOP_R, 0.4)
        rb = oracle.gqa_block_step(b_, Q[:, :, None], Kn, Vn, 2, EXCLUDE_TOP_R, 0.4)
        np.testing.assert_array_equal(ra.evicted_slot, rb.evicted_slot)
        np.testing.assert_array_equal(ra.out, rb.out[:, :, 0])
        np.testing.assert_array_equal(ra.lse, rb.lse[:, :, 0])
        for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
            np.testing.assert_array_equal(getattr(a, name), getattr(b_, name))
    # b = 1  ==  grouped-query decode step
    a, b_ = base.copy(), base.copy()
    for _ in range(3):
        Q = rng.normal(size=(U, 4, d))
        kn, vn = rng.normal(size=(2, U, d))
        ra = oracle.gqa_step(a, Q, kn, vn, 2, EXCLUDE_TOP_R, 0.4)
        rb = oracle.gqa_block_step(b_, Q[:, None], kn[:, None], vn[:, None], 2, EXCLUDE_TOP_R, 0.4)
        np.testing.assert_array_equal(ra.evicted_slot, rb.evicted_slot[:, 0])
        np.testing.assert_array_equal(ra.out, rb.out[:, 0])
        for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
            np.testing.assert_array_equal(getattr(a, name), getattr(b_, name))


def test_grouped_block_identical_heads_equal_the_single_head_block_step():
    rng = np.random.default_rng(22)
    U, B, d, b = 2, 10, 6, 4
    a = filled_state(rng, U, B, d, 13)
    c = a.copy()
    for _ in range(3):
        Q, Kn, Vn = rng.normal(size=(3, U, b, d))
        ra = oracle.block_step(a, Q, Kn, Vn, 3, EXCLUDE_TOP_R, 0.4)
        rc = oracle.gqa_block_step(c, np.repeat(Q[:, :, None], 3, 2), Kn, Vn, 3, EXCLUDE_TOP_R, 0.4)
        np.testing.assert_array_equal(ra.evicted_slot, rc.evicted_slot)
        for g in range(3):
            np.testing.assert_allclose(rc.out[:, :, g], ra.out, rtol=1e-13)
        for name in ("s", "q"):
            np.testing.assert_allclose(getattr(c, name), getattr(a, name), rtol=1e-12)
        np.testing.assert_array_equal(c.n, a.n)


@pytest.mark.parametrize("b,group", [(2, 2), (3, 4), (4, 2)])
def test_grouped_block_brute_force(b, group):
    """Definitions written out with library softmax: victims by exhaustive sorting on the frozen statistics, new
    tokens to the freed / free slots in increasing slot order, token i's heads see the survivors and new tokens
    0..i, statistics from the mean over the heads, once per token."""
    rng = np.random.default_rng(100 * b + group)
    U, B, d, scale, r = 1, 9, 4, 0.5, 2
    for live_start in (6, 12):
        st = filled_state(rng, U, B, d, live_start, scale)
        before = st.copy()
        live0 = int(before.live[0])
        need = max(0, live0 + b - B)
        Q = rng.normal(size=(U, b, group, d))
        Kn, Vn = rng.normal(size=(2, U, b, d))
        res = oracle.gqa_block_step(st, Q, Kn, Vn, r, EXCLUDE_TOP_R, scale)
        gone = brute_victims(before.s[0], before.q[0], before.n[0], before.pos[0], live0, need, r, EXCLUDE_TOP_R)
        assert list(res.evicted_slot[0][:need]) == gone and all(x == -1 for x in res.evicted_slot[0][need:])
        targets = sorted(gone + list(range(live0, live0 + b - need)))
        Kc, Vc = before.K[0].copy(), before.V[0].copy()
        s, q, n = before.s[0].copy(), before.q[0].copy(), before.n[0].copy()
        for i, t in enumerate(targets):
            Kc[t], Vc[t], s[t], q[t], n[t] = Kn[0, i], Vn[0, i], 0.0, 0.0, 0
        live1 = live0 - need + b
        for i in range(b):
            members = [j for j in range(live1) if j not in targets[i + 1:]]
            pbar = np.zeros(len(members))
            for g in range(group):
                z = scale * Kc[members] @ Q[0, i, g]
                p = softmax(z)
                np.testing.assert_allclose(res.out[0, i, g], p @ Vc[members], rtol=1e-12, atol=1e-15)
                assert res.lse[0, i, g] == pytest.approx(logsumexp(z), rel=1e-12)
                pbar += p
            pbar /= group
            s[members] += pbar; q[members] += pbar * pbar; n[members] += 1
        np.testing.assert_allclose(st.s[0, :live1], s[:live1], rtol=1e-12)
        np.testing.assert_allclose(st.q[0, :live1], q[:live1], rtol=1e-12)
        np.testing.assert_array_equal(st.n[0, :live1], n[:live1])
        # the group mean of probability rows still sums to 1 per token of the block
        lost = before.s[0][gone].sum()
        assert st.s[0, :live1].sum() + lost == pytest.approx(before.s[0, :live0].sum() + b, rel=1e-12)
