"""Device-side anomalies are reported through the status word and the kernel returns normally (nothing traps):
a corrupt occupancy count is clamped and flagged; statistics that are all NaN leave no victim and are flagged."""
import pytest
import torch

import paper_2402_06262_b200 as R
import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def filled_cache(w):
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    out = torch.zeros(w.S, w.G, w.d, dtype=w.torch_dtype, device=DEV)
    ev = torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV)
    for i in range(w.B + 3):
        R.roco_decode_step(cache, *W.decode_tokens(w, i, [i] * w.S, DEV), w.r, out, ev, scale=w.scale)
    torch.cuda.synchronize()
    assert R.roco_device_status(cache) == 0
    return cache, out, ev


def test_corrupt_live_is_clamped_and_flagged():
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=3, B=80, r=8)
    cache, out, ev = filled_cache(w)
    cache.live[0, 1] = w.B + 7                       # impossible: more occupied slots than the budget
    R.roco_decode_step(cache, *W.decode_tokens(w, 999, [w.B + 3], DEV), w.r, out, ev, scale=w.scale)
    torch.cuda.synchronize()
    assert R.roco_device_status(cache) & 2           # ROCO_DEV_BAD_LIVE
    assert int(cache.live.max()) == w.B              # the unit was treated as full
    assert torch.isfinite(out.float()).all()
    # the flag is sticky until the caller clears the word; after clearing, the next step is clean
    cache.status.zero_()
    R.roco_decode_step(cache, *W.decode_tokens(w, 1000, [w.B + 4], DEV), w.r, out, ev, scale=w.scale)
    assert R.roco_device_status(cache) == 0


def test_nan_statistics_are_flagged_not_fatal():
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=2, B=64, r=8)
    cache, out, ev = filled_cache(w)
    cache.s[0, 0] = float("nan")                     # every mean of unit 0 is NaN: no slot can win the argmin
    R.roco_decode_step(cache, *W.decode_tokens(w, 999, [w.B + 3], DEV), w.r, out, ev, scale=w.scale)
    torch.cuda.synchronize()
    assert R.roco_device_status(cache) & 4           # ROCO_DEV_BAD_VICTIM
    assert 0 <= int(ev[0, 0]) < w.B and 0 <= int(ev[0, 1]) < w.B
    assert torch.isfinite(out.float()).all()         # the attention itself does not read the statistics


def test_a_wait_that_nothing_ends_runs_out_and_is_reported():
    """The self-test kernel waits on a barrier that nothing completes: the bounded wait gives up after about two
    seconds, sets the time-out bit and the kernel returns; the context stays usable (a decode step runs after)."""
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    waited = torch.zeros(1, dtype=torch.int32, device=DEV)
    R.roco_selftest_wait_timeout(status, waited)
    torch.cuda.synchronize()
    assert int(status.item()) & 1, "ROCO_DEV_WAIT_TIMEOUT must be set"
    assert 1500 <= int(waited.item()) <= 4000, waited.item()
    probe = torch.arange(8, device=DEV).sum().item()   # the device still answers
    assert probe == 28
