"""The synthetic consistency diagnostic (Sec. 4.3 preliminary experiment on synthetic inputs)."""
import pytest

import workloads as W
from paper_2402_06262_b200.consistency import SCORED, jaccard_consistency

pytestmark = pytest.mark.gpu


def test_jaccard_is_one_when_the_budget_holds_everything_and_in_range_otherwise():
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=4, prompt_lo=96, prompt_hi=96)
    for name in SCORED:
        j = jaccard_consistency(w, name, budget=48, steps=32)
        assert 0.0 < j <= 1.0, (name, j)
    # budget one short of the whole sequence: the two sets can differ by at most one token
    j = jaccard_consistency(w, "MAS", budget=127, steps=32)
    assert j >= (127 - 1) / (127 + 1) - 1e-6
