"""GPU parity of both scope readings and both step orders at the budgets of the Llama-7B-shape decode workload
(B = 1024) and the long-context workload (B = 4096), in the launch configurations the benchmark times, plus the
case the order ATTEND_FIRST is most exposed to: a victim whose value row lies in the last tile the kernel streams.
"""
import numpy as np
import pytest
import torch

import paper_2402_06262_b200 as R
import workloads as W
from harness import DecodeParity, Tally, state_from_cache

pytestmark = pytest.mark.gpu
DEV = "cuda"

MODES = [(R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_EVICT_FIRST), (R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_ATTEND_FIRST),
         (R.ROCO_SCOPE_LOWEST_R, R.ROCO_EVICT_FIRST), (R.ROCO_SCOPE_LOWEST_R, R.ROCO_ATTEND_FIRST)]
ROWS_PER_TILE = 64            # a 16 KiB tile of bf16 rows with d = 128


def build_cache(w, scope_mode, L):
    """The whole workload's cache, built by the library's prefill chunk by chunk (prompts of L tokens)."""
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    chunk = min(w.G, 256)
    for b in range(w.S):
        for g0 in range(0, w.G, chunk):
            Q, K, V = (t[None] for t in W.prompt_chunk(w, b, g0, g0 + chunk, L, DEV))
            sub = R.Cache(1, chunk, w.B, w.d, w.torch_dtype, DEV)
            R.roco_prefill(Q, K, V, [L], w.B, w.r, sub, scope_mode=scope_mode, scale=w.scale)
            for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
                getattr(cache, name)[b, g0:g0 + chunk].copy_(getattr(sub, name)[0])
            assert R.roco_device_status(sub) == 0
    return cache


_CACHES = {}


def cached_cache(key, w, scope_mode, L):
    """One prefill per (workload, scope reading) and test session; every test steps a copy."""
    if (key, scope_mode) not in _CACHES:
        _CACHES.clear()                      # at most one full-size cache is kept alive
        _CACHES[(key, scope_mode)] = build_cache(w, scope_mode, L)
    src = _CACHES[(key, scope_mode)]
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
        getattr(cache, name).copy_(getattr(src, name))
    return cache


def step_and_compare(w, cache, units, mode, order, L, steps):
    tally = Tally()
    par = DecodeParity(cache, state_from_cache(cache, units), units, w.r, mode, order, tally, scale=w.scale)
    last_tile = 0
    t_pos = [L] * w.S
    for i in range(steps):
        res = par.step(*W.decode_tokens(w, i, t_pos, DEV), check_state=(i in (0, steps - 1)))
        last_tile += int((res.evicted_slot >= w.B - ROWS_PER_TILE).sum())
        t_pos = [t + 1 for t in t_pos]
    assert R.roco_device_status(cache) == 0
    assert tally.decisions == steps * len(units)
    # steps inside the margin are few, and even there the two sides almost always agree
    assert tally.near_ties <= tally.decisions // 5 and tally.near_tie_disagreements <= 2, tally
    return tally, last_tile


@pytest.mark.parametrize("mode,order", MODES)
def test_llama7b_decode_shape_both_readings(mode, order):
    """8192 units, B = 1024, r = 64: 96 sampled units through 8 steps under each reading of scope and order."""
    w = W.LLAMA7B_DECODE
    cache = cached_cache("7b", w, mode, w.prompt_lo)
    units = sorted(np.random.default_rng(11).choice(w.U, 96, replace=False).tolist())
    _, last_tile = step_and_compare(w, cache, units, mode, order, w.prompt_lo, 8)
    assert last_tile >= 1, "no sampled victim lay in the last value tile"
    assert int(cache.live.min()) == w.B == int(cache.live.max())
    srt = cache.pos.sort(dim=-1).values
    assert bool((srt[..., 1:] > srt[..., :-1]).all())


@pytest.mark.parametrize("mode,order", MODES)
def test_long_context_decode_shape_both_readings(mode, order):
    """4096 units, B = 4096, r = 64 (the long-context decode launch; prompts of 8192 tokens fill the budget):
    24 sampled units through 8 steps under each reading."""
    w = W.scaled(W.LONG_CONTEXT, prompt_lo=8192, prompt_hi=8192)
    cache = cached_cache("long", w, mode, 8192)
    units = sorted(np.random.default_rng(12).choice(w.U, 24, replace=False).tolist())
    step_and_compare(w, cache, units, mode, order, 8192, 8)
    assert int(cache.live.min()) == w.B == int(cache.live.max())


@pytest.mark.parametrize("mode,r", [(R.ROCO_SCOPE_EXCLUDE_TOP_R, 0), (R.ROCO_SCOPE_LOWEST_R, 1024)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_attend_first_victim_in_last_value_tile(mode, r, dtype):
    """ATTEND_FIRST attends over the cache as it stood before the step.  Every unit's victim is planted in the
    last tile of the value stream and receives about half of the query's probability, and the new value differs
    from the old one by 10 per component: an overwrite that lands before the value pass has read the row would
    move the output by ~5, far outside the tolerance.  296 units (two per SM) keep the SMs busy with several CTAs
    each, and three steps in a row move the victim inside the last tile."""
    S, G, B, d = 1, 296, 1024, 128
    g = torch.Generator(device=DEV); g.manual_seed(5)
    cache = R.Cache(S, G, B, d, dtype, DEV)
    cache.K.copy_(torch.randn(S, G, B, d, device=DEV, generator=g).to(dtype))
    cache.V.copy_(torch.randn(S, G, B, d, device=DEV, generator=g).to(dtype))
    p0 = torch.rand(S, G, B, device=DEV, generator=g) * 2e-3 + 5e-4     # per-token mean probability so far
    cache.n.fill_(50)
    cache.s.copy_(p0 * 50)
    cache.q.copy_(p0 * p0 * 50 * (1 + torch.rand(S, G, B, device=DEV, generator=g)))
    cache.pos.copy_(torch.arange(B, device=DEV, dtype=torch.int32).expand(S, G, B))
    cache.live.fill_(B)
    cache.t_next.fill_(B)
    scale = d ** -0.5
    units = list(range(0, G, 7))
    tally = Tally()
    par = DecodeParity(cache, None, units, r, mode, R.ROCO_ATTEND_FIRST, tally, scale=scale)
    for step in range(3):
        victim = B - 1 - ((torch.arange(G, device=DEV) * 5 + 17 * step) % ROWS_PER_TILE)      # last tile
        q = torch.randn(S, G, d, device=DEV, generator=g).to(dtype)
        # the planted victim: seen so often that its mean stays the lowest even after this query's share, and a
        # key along the query so that this query gives it about half of the probability mass
        qf = q.float()
        beta = (np.log(B) + 0.5) / (scale * (qf * qf).sum(-1, keepdim=True))
        idx = victim.view(1, G, 1, 1).expand(S, G, 1, d)
        cache.K.scatter_(2, idx, (beta * qf).to(dtype).unsqueeze(2))
        cache.n.scatter_(2, victim.view(1, G, 1), torch.full((S, G, 1), 1 << 20, dtype=torch.int32, device=DEV))
        v_old = torch.gather(cache.V, 2, idx).squeeze(2)
        v_new = (v_old.float() + 10.0).to(dtype)
        k_new = torch.randn(S, G, d, device=DEV, generator=g).to(dtype)
        par.st = state_from_cache(cache, units)
        res = par.step(q, k_new, v_new, check_state=True)
        np.testing.assert_array_equal(res.evicted_slot, victim[units].cpu().numpy())
        assert not res.near_tie.any()
    assert R.roco_device_status(cache) == 0
