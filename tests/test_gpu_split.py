"""GPU parity of the decode step split over the cache slots (few units per call)."""
import pytest
import torch

import oracle
import paper_2402_06262_b200 as R
import workloads as W
from harness import DecodeParity, Tally

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("order", [R.ROCO_EVICT_FIRST, R.ROCO_ATTEND_FIRST])
@pytest.mark.parametrize("splits", [1, 2, 3, 8])
@pytest.mark.parametrize("mode", [R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_SCOPE_LOWEST_R])
@pytest.mark.parametrize("dtype,d,B", [("bf16", 128, 300), ("f32", 64, 100)])
def test_split_decode_from_empty_cache(splits, mode, dtype, d, B, order):
    """Fill from empty (ranges that are still empty for some CTAs), then evict; B is not a multiple of the tile."""
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=5, d=d, dtype=dtype, B=B, r=11)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    st = oracle.empty_state(w.U, B, d)
    tally = Tally()
    par = DecodeParity(cache, st, range(w.U), w.r, mode, order, tally, scale=w.scale, splits=splits)
    for i in range(B + 40):
        par.step(*W.decode_tokens(w, i, [i], DEV), check_state=(i % 25 == 24) or i == B + 39)
    assert R.roco_device_status(cache) == 0 and tally.decisions == 40 * w.U


def test_split_workspace_is_checked():
    w = W.scaled(W.TOY, B=32, r=4)
    cache = R.Cache(w.S, w.G, w.B, w.d, torch.float32, DEV)
    x = torch.zeros(w.S, w.G, w.d, device=DEV)
    ev = torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV)
    small = torch.empty(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(R.RocoError) as e:
        R.roco_decode_step_split(cache, x, x, x, 4, 4, x.clone(), ev, small)
    assert e.value.code == 3
    with pytest.raises(R.RocoError) as e:
        R.roco_decode_step_split(cache, x, x, x, 4, 0, x.clone(), ev, small)
    assert e.value.code == 1
