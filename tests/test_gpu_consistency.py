"""The consistency diagnostic (Sec. 4.3 preliminary experiment, on synthetic inputs) against the oracle: a budgeted
cache and a cache that never evicts are fed the same tokens under one policy; at every step the library's overlap
count (budgeted cache's tokens among the full cache's top-B by the policy's score) must equal the oracle's, up to
the tokens whose score lies within the 1e-5 margin of the top-B boundary."""
import numpy as np
import pytest
import torch

import oracle
import paper_2402_06262_b200 as R
import workloads as W
from harness import PolicyParity, Tally, unit_view, widen

pytestmark = pytest.mark.gpu
DEV = "cuda"
SCORED = {"MAS": R.ROCO_POLICY_MAS_WINDOW, "AAS": R.ROCO_POLICY_H2O, "AQAS": R.ROCO_POLICY_SCISSORHANDS,
          "LTAS": R.ROCO_POLICY_TOVA}


def run(w, policy, budget, total):
    """Feeds `total` tokens through both caches on the GPU and in the oracle; returns the per-step comparison."""
    full = R.Cache(w.S, w.G, total, w.d, w.torch_dtype, DEV)
    small = R.Cache(w.S, w.G, budget, w.d, w.torch_dtype, DEV)
    units = range(w.U)
    par_f = PolicyParity(full, oracle.empty_state(w.U, total, w.d), units, policy, 0, Tally(), scale=w.scale)
    par_s = PolicyParity(small, oracle.empty_state(w.U, budget, w.d), units, policy, 0, Tally(), scale=w.scale)
    ov = torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV)
    jsum = torch.zeros(w.S, w.G, dtype=torch.float32, device=DEV)
    cnt = torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV)
    firm = slack_total = 0
    want_sum = np.zeros(w.U)
    for t in range(total):
        q, k, v = W.decode_tokens(w, t, [t] * w.S, DEV)
        par_f.step(q, k, v)
        par_s.step(q, k, v)
        R.roco_consistency_step(full, small, policy, ov, jsum, cnt)
        torch.cuda.synchronize()
        g = ov.flatten().cpu().numpy()
        B = min(t + 1, budget)
        for u in range(w.U):
            fs, ss = par_f.st, par_s.st
            sc = oracle.policy_score(policy, fs.s[u, :t + 1], fs.q[u, :t + 1], fs.n[u, :t + 1])
            want, slack = oracle.topb_overlap(sc, fs.pos[u, :t + 1], ss.pos[u, :B], delta=1e-5,
                                              exact_ties_firm=(policy == R.ROCO_POLICY_SCISSORHANDS))
            assert abs(int(g[u]) - want) <= slack, (t, u, int(g[u]), want, slack)
            firm += slack == 0
            slack_total += slack
            want_sum[u] += oracle.jaccard_from_overlap(int(g[u]), B)
    assert R.roco_device_status(full) == 0 and R.roco_device_status(small) == 0
    assert bool((cnt == total).all())
    np.testing.assert_allclose(jsum.flatten().cpu().numpy(), want_sum, rtol=1e-5)
    return firm, slack_total, float(jsum.sum() / cnt.sum())


@pytest.mark.parametrize("name", sorted(SCORED))
def test_overlap_counts_match_the_oracle(name):
    w = W.scaled(W.LLAMA7B_DECODE, S=2, layers=1, heads=3, prompt_lo=0, prompt_hi=0)
    total, budget = 120, 48
    firm, slack_total, mean_j = run(w, SCORED[name], budget, total)
    assert firm >= 0.9 * total * w.U, (firm, slack_total)     # nearly every comparison is exact
    assert 0.0 < mean_j <= 1.0


def test_budget_one_short_and_budget_that_holds_everything():
    w = W.scaled(W.TOY, heads=2)
    _, _, j = run(w, R.ROCO_POLICY_MAS_WINDOW, 39, 40)
    assert j >= (39 - 1) / (39 + 1) - 1e-6
    _, _, j = run(w, R.ROCO_POLICY_H2O, 40, 40)
    assert j == 1.0


def test_argument_checks():
    a = R.Cache(1, 2, 16, 64, torch.float32, DEV)
    b = R.Cache(1, 2, 32, 64, torch.float32, DEV)
    z = torch.zeros(1, 2, dtype=torch.int32, device=DEV)
    f = torch.zeros(1, 2, dtype=torch.float32, device=DEV)
    with pytest.raises(R.RocoError) as e:
        R.roco_consistency_step(a, b, R.ROCO_POLICY_H2O, z, f, z.clone())          # full smaller than budgeted
    assert e.value.code == 1
    with pytest.raises(R.RocoError) as e:
        R.roco_consistency_step(b, a, R.ROCO_POLICY_RECENCY, z, f, z.clone())      # no attention-based score
    assert e.value.code == 1
