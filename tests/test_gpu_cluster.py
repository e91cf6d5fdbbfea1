"""GPU parity of the decode step with a thread-block cluster of CTAs per unit (calls with few units; partial
results exchanged through distributed shared memory): both step orders and both scope readings, 2, 4 and 8 CTAs
per unit, caches that fill from empty (ranks whose slot range is still empty, ranks that own no slot at all),
exact ties resolved by position across ranks, and the shapes the benchmark times."""
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


@pytest.mark.parametrize("mode,order", MODES)
@pytest.mark.parametrize("dtype,d,B,heads,ranks", [("bf16", 128, 300, 5, 2), ("bf16", 128, 300, 3, 8),
                                                     ("f32", 64, 100, 7, 2), ("f32", 128, 76, 3, 4),
                                                     ("bf16", 64, 520, 6, 4)])
def test_fill_from_empty_then_evict(mode, order, dtype, d, B, heads, ranks):
    """Fill from empty, then evict; B is not a multiple of the tile.  With 8 ranks on 5 tiles, three ranks own no
    slot at all and still take part in every exchange."""
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=heads, d=d, dtype=dtype, B=B, r=11)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    st = oracle.empty_state(w.U, B, d)
    tally = Tally()
    par = DecodeParity(cache, st, range(w.U), w.r, mode, order, tally, scale=w.scale, ranks=ranks)
    n_steps = B + 24
    for i in range(n_steps):
        par.step(*W.decode_tokens(w, i, [i], DEV), check_state=(i % 25 == 24) or i == n_steps - 1)
    assert R.roco_device_status(cache) == 0 and tally.decisions == 24 * w.U


@pytest.mark.parametrize("mode,order", MODES)
@pytest.mark.parametrize("ranks", [2, 4])
def test_uniform_attention_position_ties(mode, order, ranks):
    """q = 0 everywhere: all probabilities are exactly 1/live, statistics of same-age tokens are bit-identical,
    and only the position rule decides -- for the scope threshold and for the victim, across ranks.  No near-tie
    exclusions (strict)."""
    S, G, B, d, r = 1, 3, 160, 64, 5
    cache = R.Cache(S, G, B, d, torch.float32, DEV)
    st = oracle.empty_state(S * G, B, d)
    par = DecodeParity(cache, st, range(S * G), r, mode, order, Tally(), strict=True, ranks=ranks)
    g = torch.Generator(device=DEV); g.manual_seed(1)
    for i in range(B + 30):
        q = torch.zeros(S, G, d, device=DEV)
        k = torch.randn(S, G, d, device=DEV, generator=g)
        v = torch.randn(S, G, d, device=DEV, generator=g)
        par.step(q, k, v, check_state=(i % 10 == 9))
    assert R.roco_device_status(cache) == 0


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
@pytest.mark.parametrize("G,B,ranks,n_units", [(32, 8192, 8, 6), (64, 4096, 4, 8), (128, 1024, 2, 16)])
def test_shapes_the_benchmark_times(mode, order, G, B, ranks, n_units):
    """One layer of one long sequence (32 units, B = 8192, 8 CTAs per unit) and two shapes in between, bf16,
    d = 128: sampled units through 6 steps under each reading."""
    cache, g = seeded_full_cache(1, G, B, 128, torch.bfloat16, 17)
    assert R.roco_decode_cluster_ranks(cache) == ranks
    units = sorted(np.random.default_rng(5).choice(G, n_units, replace=False).tolist())
    tally = Tally()
    par = DecodeParity(cache, state_from_cache(cache, units), units, 64, mode, order, tally, scale=128 ** -0.5,
                       ranks=ranks)
    for i in range(6):
        q, k, v = (torch.randn(1, G, 128, device=DEV, generator=g).to(torch.bfloat16) for _ in range(3))
        par.step(q, k, v, check_state=(i in (0, 5)))
    assert R.roco_device_status(cache) == 0 and tally.decisions == 6 * n_units
    assert tally.near_ties <= tally.decisions // 5, tally
    srt = cache.pos.sort(dim=-1).values
    assert bool((srt[..., 1:] > srt[..., :-1]).all())


def test_matches_the_one_cta_per_unit_kernel():
    """Same inputs through roco_decode_step and the cluster path: identical decisions and integer state, outputs
    and statistics equal to fp32 rounding of the merge."""
    S, G, B, d = 2, 20, 640, 128
    a, g = seeded_full_cache(S, G, B, d, torch.bfloat16, 31)
    b = R.Cache(S, G, B, d, torch.bfloat16, DEV)
    for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
        getattr(b, name).copy_(getattr(a, name))
    outs = [torch.zeros(S, G, d, dtype=torch.bfloat16, device=DEV) for _ in range(2)]
    evs = [torch.zeros(S, G, dtype=torch.int32, device=DEV) for _ in range(2)]
    for i in range(5):
        q, k, v = (torch.randn(S, G, d, device=DEV, generator=g).to(torch.bfloat16) for _ in range(3))
        R.roco_decode_step(a, q, k, v, 48, outs[0], evs[0])
        R.roco_decode_step_cluster(b, q, k, v, 48, outs[1], evs[1], ranks=4)
        torch.cuda.synchronize()
        assert torch.equal(evs[0], evs[1])
        assert float((outs[0].float() - outs[1].float()).abs().max()) <= 2e-2
    for name in ("K", "V", "n", "pos", "live", "t_next"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    for name in ("s", "q"):
        np.testing.assert_allclose(getattr(b, name).cpu().numpy(), getattr(a, name).cpu().numpy(), rtol=1e-4, atol=1e-30)


def test_arguments_are_checked():
    w = W.scaled(W.TOY, B=32, r=4)
    cache = R.Cache(w.S, w.G, w.B, w.d, torch.float32, DEV)
    x = torch.zeros(w.S, w.G, w.d, device=DEV)
    ev = torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV)
    with pytest.raises(R.RocoError) as e:
        R.roco_decode_step_cluster(cache, x, x, x, 4, x.clone(), ev, ranks=3)
    assert e.value.code == 1
    odd = R.Cache(1, 2, 30, 64, torch.float32, DEV)        # B not a multiple of 4: no cluster path
    assert R.roco_decode_cluster_ranks(odd) == 1
    x2 = torch.zeros(1, 2, 64, device=DEV); ev2 = torch.zeros(1, 2, dtype=torch.int32, device=DEV)
    with pytest.raises(R.RocoError) as e:
        R.roco_decode_step_cluster(odd, x2, x2, x2, 4, x2.clone(), ev2, ranks=2)
    assert e.value.code == 2
    R.roco_decode_step_cluster(odd, x2, x2, x2, 4, x2.clone(), ev2, ranks=0)       # falls back to one CTA per unit
    torch.cuda.synchronize()
    assert R.roco_device_status(odd) == 0
