"""Pins for the oracle's margin analysis: the set of admissible victims (Sec. 4.3 rule under errors of at most a
relative margin) and the select-to-budget replay guided by another implementation's survivor set.  Expected values
come from exact hand cases and from brute force in Python (sorted()), never from the functions under test."""
import numpy as np
import pytest

import oracle
from oracle import EXCLUDE_TOP_R, LOWEST_R


def py_victim(s, q, n, pos, r, mode):
    """The rule by exhaustive sorting: m lowest (variance, position); of those the lowest (mean, position)."""
    live = len(s)
    mean = [s[j] / n[j] for j in range(live)]
    var = [max(0.0, q[j] / n[j] - mean[j] ** 2) for j in range(live)]
    order = sorted(range(live), key=lambda j: (var[j], pos[j]))
    m = min(max((live - r) if mode == EXCLUDE_TOP_R else r, 1), live)
    return min(order[:m], key=lambda j: (mean[j], pos[j]))


def random_stats(rng, live):
    n = rng.integers(1, 40, live).astype(np.int32)
    p = rng.uniform(1e-3, 0.2, live)
    s = p * n
    q = s * p * rng.uniform(1.0, 1.8, live)
    return s, q, n, rng.permutation(live).astype(np.int32)


@pytest.mark.parametrize("mode,r", [(EXCLUDE_TOP_R, 0), (EXCLUDE_TOP_R, 5), (LOWEST_R, 1), (LOWEST_R, 6), (LOWEST_R, 24)])
def test_zero_margin_admits_the_victim_alone(mode, r):
    rng = np.random.default_rng(3)
    for _ in range(40):
        s, q, n, pos = random_stats(rng, 24)
        adm = oracle.admissible_victims(s, q, n, pos, r, mode, delta=0.0)
        assert adm.sum() == 1 and adm[py_victim(s, q, n, pos, r, mode)]


def test_exact_ties_at_zero_margin_fall_to_the_position():
    # four tokens with identical statistics: the rule's choice is the lowest position, and nothing else is admissible
    s, q, n = np.full(4, 0.5), np.full(4, 0.2), np.full(4, 2, np.int32)
    pos = np.array([7, 3, 9, 5], np.int32)
    for mode, r in ((EXCLUDE_TOP_R, 1), (LOWEST_R, 2)):
        adm = oracle.admissible_victims(s, q, n, pos, r, mode, delta=0.0)
        assert adm.tolist() == [False, True, False, False]


def test_hand_case_two_means_inside_the_margin():
    # variances 0, 0, 0.09, 0 (tokens 0, 1, 3 seen once: Acc^square = Acc^2); means 0.1000, 0.1001, 0.05, 0.3
    n = np.array([1, 1, 2, 1], np.int32)
    s = np.array([0.1, 0.1001, 0.1, 0.3])
    q = np.array([0.01, 0.1001 ** 2, 2 * (0.05 ** 2 + 0.09), 0.09])
    pos = np.arange(4, dtype=np.int32)
    # scope = all but the highest variance (token 2, whose mean is the lowest of all): tokens 0 and 1 are 0.1 % apart
    assert oracle.admissible_victims(s, q, n, pos, 1, EXCLUDE_TOP_R, 1e-5).tolist() == [True, False, False, False]
    assert oracle.admissible_victims(s, q, n, pos, 1, EXCLUDE_TOP_R, 1e-3).tolist() == [True, True, False, False]
    # scope = everything: token 2 wins on the mean by a factor of two, margin or not
    assert oracle.admissible_victims(s, q, n, pos, 0, EXCLUDE_TOP_R, 1e-3).tolist() == [False, False, True, False]


@pytest.mark.parametrize("mode,r", [(EXCLUDE_TOP_R, 4), (LOWEST_R, 5)])
def test_every_victim_reachable_inside_the_margin_is_admitted(mode, r):
    """Monte Carlo: statistics moved by up to delta/4 relative (which moves the variance by less than
    delta x its uncancelled terms and the mean by less than delta x mean) never produce a victim outside
    the admissible set; and the set stays small."""
    rng = np.random.default_rng(9)
    delta = 0.02
    sizes = []
    for _ in range(12):
        s, q, n, pos = random_stats(rng, 20)
        s[3] = s[5] / n[5] * n[3] * 1.004          # two means 0.4 % apart
        adm = oracle.admissible_victims(s, q, n, pos, r, mode, delta)
        sizes.append(int(adm.sum()))
        for _ in range(200):
            e1, e2 = rng.uniform(-delta / 4, delta / 4, (2, 20))
            v = py_victim(s * (1 + e1), q * (1 + e2), n, pos, r, mode)
            assert adm[v], (v, adm)
        assert adm[py_victim(s, q, n, pos, r, mode)]
    assert np.mean(sizes) < 6


def test_guided_replay_with_the_rules_own_set_follows_nothing():
    rng = np.random.default_rng(1)
    for mode, r in ((EXCLUDE_TOP_R, 3), (LOWEST_R, 4), (LOWEST_R, 1)):
        s, q, n, _ = random_stats(rng, 30)
        own = oracle.select_to_budget_iterated(s, q, n, 12, r, mode)
        followed, keep = oracle.select_to_budget_guided(s, q, n, 12, r, mode, own, delta=1e-5)
        assert followed == 0 and np.array_equal(keep, own) and keep.sum() == 12


def test_guided_replay_follows_a_swap_inside_the_margin_and_rejects_one_outside():
    # 6 tokens seen once (variance 0), budget 4, scope = everything: the two lowest means leave.
    n = np.ones(6, np.int32)
    s = np.array([0.30, 0.1000000, 0.25, 0.1000001, 0.05, 0.40])
    q = s * s
    own = oracle.select_to_budget_iterated(s, q, n, 4, 0, EXCLUDE_TOP_R)
    assert own.tolist() == [True, False, True, True, False, True]           # tokens 4 and 1 leave
    swapped = np.array([True, True, True, False, False, True])             # token 3 instead of 1: 1e-6 apart
    followed, keep = oracle.select_to_budget_guided(s, q, n, 4, 0, EXCLUDE_TOP_R, swapped, delta=1e-5)
    assert followed == 1 and np.array_equal(keep, swapped)
    wrong = np.array([True, True, False, True, False, True])               # token 2 (mean 0.25) instead of 1
    followed, _ = oracle.select_to_budget_guided(s, q, n, 4, 0, EXCLUDE_TOP_R, wrong, delta=1e-5)
    assert followed == -2                                                   # second iteration, outside the margin
    followed, _ = oracle.select_to_budget_guided(s, q, n, 4, 0, EXCLUDE_TOP_R, swapped, delta=1e-8)
    assert followed == -2                                                   # the same swap, margin too small
