"""GPU parity of the one-launch decode step for calls with few units (persistent CTAs that divide the cache rows
of all units among themselves; partial results merged by whoever draws a unit's last ticket): both step orders
and both scope readings, caches that fill from empty, pieces that span several units and units cut into many
pieces, the shapes the benchmark times, and a victim that dominates the softmax (the exact second pass)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2402_06262_b200 as R
import workloads as W
from harness import DecodeParity, Tally, state_from_cache

pytestmark = pytest.mark.gpu
DEV = "cuda"

MODES = [(R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_EVICT_FIRST), (R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_ATTEND_FIRST),
         (R.ROCO_SCOPE_LOWEST_R, R.ROCO_EVICT_FIRST), (R.ROCO_SCOPE_LOWEST_R, R.ROCO_ATTEND_FIRST)]


def tickets_are_clear(par):
    """Every completed call leaves the ticket counters (the head of the workspace) at zero."""
    U = par.cache.U
    return bool((par.pws[: 4 * U].view(torch.int32) == 0).all())


@pytest.mark.parametrize("mode,order", MODES)
@pytest.mark.parametrize("dtype,d,B,heads", [("bf16", 128, 300, 5), ("f32", 64, 100, 700), ("f32", 128, 77, 3),
                                               ("bf16", 64, 200, 40)])
def test_fill_from_empty_then_evict(mode, order, dtype, d, B, heads):
    """Fill from empty (pieces that hold no occupied row yet), then evict; B is not a multiple of the tile.  Five
    units are cut into one-tile pieces; 700 small units give every CTA several whole units and two halves."""
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=heads, d=d, dtype=dtype, B=B, r=11)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    units = list(range(w.U)) if w.U <= 8 else sorted(np.random.default_rng(3).choice(w.U, 8, replace=False).tolist())
    st = oracle.empty_state(len(units), B, d)
    tally = Tally()
    par = DecodeParity(cache, st, units, w.r, mode, order, tally, scale=w.scale, persistent=True)
    n_steps = B + 24
    for i in range(n_steps):
        par.step(*W.decode_tokens(w, i, [i], DEV), check_state=(i % 25 == 24) or i == n_steps - 1)
    assert R.roco_device_status(cache) == 0 and tally.decisions == 24 * len(units)
    assert tickets_are_clear(par)


def seeded_full_cache(S, G, B, d, dtype, seed):
    """A full cache with plausible statistics (each token seen 50 times), positions 0..B-1."""
    g = torch.Generator(device=DEV); g.manual_seed(seed)
    cache = R.Cache(S, G, B, d, dtype, DEV)
    cache.K.copy_(torch.randn(S, G, B, d, device=DEV, generator=g).to(dtype))
    cache.V.copy_(torch.randn(S, G, B, d, device=DEV, generator=g).to(dtype))
    p0 = torch.rand(S, G, B, device=DEV, generator=g) * 2e-3 + 5e-4
    cache.n.fill_(50)
    cache.s.copy_(p0 * 50)
    cache.q.copy_(p0 * p0 * 50 * (1 + torch.rand(S, G, B, device=DEV, generator=g)))
    cache.pos.copy_(torch.arange(B, device=DEV, dtype=torch.int32).expand(S, G, B))
    cache.live.fill_(B)
    cache.t_next.fill_(B)
    return cache, g


@pytest.mark.parametrize("mode,order", MODES)
@pytest.mark.parametrize("G,B,n_units", [(256, 1024, 24), (32, 8192, 6)])
def test_shapes_the_benchmark_times(mode, order, G, B, n_units):
    """One layer of the Llama-7B-shape decode workload (256 units, B = 1024) and one layer of one long sequence
    (32 units, B = 8192), bf16, d = 128: sampled units through 6 steps under each reading."""
    cache, g = seeded_full_cache(1, G, B, 128, torch.bfloat16, 17)
    units = sorted(np.random.default_rng(5).choice(G, n_units, replace=False).tolist())
    tally = Tally()
    par = DecodeParity(cache, state_from_cache(cache, units), units, 64, mode, order, tally, scale=128 ** -0.5,
                       persistent=True)
    for i in range(6):
        q, k, v = (torch.randn(1, G, 128, device=DEV, generator=g).to(torch.bfloat16) for _ in range(3))
        par.step(q, k, v, check_state=(i in (0, 5)))
    assert R.roco_device_status(cache) == 0 and tally.decisions == 6 * n_units
    assert tally.near_ties <= tally.decisions // 5, tally
    assert tickets_are_clear(par)
    srt = cache.pos.sort(dim=-1).values
    assert bool((srt[..., 1:] > srt[..., :-1]).all())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_victim_that_dominates_the_softmax(dtype):
    """EVICT_FIRST takes the victim's stale row out of sums that already contain it.  Here the victim (planted by a
    huge Count: the lowest mean) has a key along the query and holds about 90 % of the probability mass before it
    is removed, and its value row is 100 per component away from the others: a plain subtraction would lose the
    answer to cancellation, so the exact second pass has to run.  Checked against the oracle at the usual bounds
    (1e-5 for fp32)."""
    S, G, B, d = 1, 40, 512, 128
    cache, g = seeded_full_cache(S, G, B, d, dtype, 23)
    scale = d ** -0.5
    units = list(range(0, G, 3))
    tally = Tally()
    par = DecodeParity(cache, None, units, 0, R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_EVICT_FIRST, tally, scale=scale,
                       persistent=True)
    for step in range(3):
        victim = (torch.arange(G, device=DEV) * 37 + 101 * step) % B
        q = torch.randn(S, G, d, device=DEV, generator=g).to(dtype)
        qf = q.float()
        beta = (np.log(B) + 2.2) / (scale * (qf * qf).sum(-1, keepdim=True))     # e^2.2 ~ 9 times the rest
        idx = victim.view(1, G, 1, 1).expand(S, G, 1, d)
        cache.K.scatter_(2, idx, (beta * qf).to(dtype).unsqueeze(2))
        cache.V.scatter_(2, idx, torch.full((S, G, 1, d), 100.0, device=DEV).to(dtype))
        cache.n.scatter_(2, victim.view(1, G, 1), torch.full((S, G, 1), 1 << 20, dtype=torch.int32, device=DEV))
        k_new, v_new = (torch.randn(S, G, d, device=DEV, generator=g).to(dtype) for _ in range(2))
        par.st = state_from_cache(cache, units)
        # the victim's share of the softmax over the cache as it stands (what the kernel's guard looks at)
        z = scale * np.einsum("ud,ubd->ub", qf[0, units].double().cpu().numpy(), par.st.K)
        share = np.exp(z - z.max(1, keepdims=True))
        share /= share.sum(1, keepdims=True)
        assert (share[np.arange(len(units)), victim[units].cpu().numpy()] > 0.6).all()
        res = par.step(q, k_new, v_new, check_state=True)
        np.testing.assert_array_equal(res.evicted_slot, victim[units].cpu().numpy())
        assert not res.near_tie.any()
    assert R.roco_device_status(cache) == 0 and tickets_are_clear(par)


def test_matches_the_one_cta_per_unit_kernel():
    """Same inputs through roco_decode_step and the persistent path: identical decisions and integer state, outputs
    and statistics equal to fp32 rounding of the merge."""
    S, G, B, d = 2, 48, 640, 128
    a, g = seeded_full_cache(S, G, B, d, torch.bfloat16, 31)
    b = R.Cache(S, G, B, d, torch.bfloat16, DEV)
    for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
        getattr(b, name).copy_(getattr(a, name))
    ws = torch.empty(R.roco_decode_persistent_workspace_bytes(b), dtype=torch.uint8, device=DEV)
    R.roco_decode_persistent_workspace_init(b, ws)
    outs = [torch.zeros(S, G, d, dtype=torch.bfloat16, device=DEV) for _ in range(2)]
    evs = [torch.zeros(S, G, dtype=torch.int32, device=DEV) for _ in range(2)]
    for i in range(5):
        q, k, v = (torch.randn(S, G, d, device=DEV, generator=g).to(torch.bfloat16) for _ in range(3))
        R.roco_decode_step(a, q, k, v, 48, outs[0], evs[0])
        R.roco_decode_step_persistent(b, q, k, v, 48, outs[1], evs[1], ws)
        torch.cuda.synchronize()
        assert torch.equal(evs[0], evs[1])
        assert float((outs[0].float() - outs[1].float()).abs().max()) <= 2e-2
    for name in ("K", "V", "n", "pos", "live", "t_next"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    for name in ("s", "q"):
        np.testing.assert_allclose(getattr(b, name).cpu().numpy(), getattr(a, name).cpu().numpy(), rtol=1e-4, atol=1e-30)


def test_workspace_is_checked():
    w = W.scaled(W.TOY, B=32, r=4)
    cache = R.Cache(w.S, w.G, w.B, w.d, torch.float32, DEV)
    x = torch.zeros(w.S, w.G, w.d, device=DEV)
    ev = torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV)
    small = torch.empty(256, dtype=torch.uint8, device=DEV)
    assert R.roco_decode_persistent_workspace_bytes(cache) > 256
    with pytest.raises(R.RocoError) as e:
        R.roco_decode_step_persistent(cache, x, x, x, 4, x.clone(), ev, small)
    assert e.value.code == 3
    with pytest.raises(R.RocoError) as e:
        R.roco_decode_persistent_workspace_init(cache, small)
    assert e.value.code == 3
    ws = torch.empty(R.roco_decode_persistent_workspace_bytes(cache), dtype=torch.uint8, device=DEV)
    with pytest.raises(R.RocoError) as e:
        R.roco_decode_step_persistent(cache, x, x, x, 4, x.clone(), ev, ws, step_order=7)
    assert e.value.code == 1
