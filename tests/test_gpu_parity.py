"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle, element by element, on the same
seeded inputs.  Sizes span several 16 KiB tiles and a ragged tail; the full-size case runs the benchmark's
launch configuration and compares sampled units."""
import numpy as np
import pytest
import torch

import oracle
import paper_2402_06262_b200 as R
import workloads as W
from harness import DecodeParity, Tally, compare_state, prefill_parity, unit_view, widen, state_from_cache

pytestmark = pytest.mark.gpu

MODES = [(R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_EVICT_FIRST), (R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_ATTEND_FIRST),
         (R.ROCO_SCOPE_LOWEST_R, R.ROCO_EVICT_FIRST), (R.ROCO_SCOPE_LOWEST_R, R.ROCO_ATTEND_FIRST)]
DEV = "cuda"


def prompt_tensors(w, L, device=DEV):
    qs, ks, vs = zip(*[W.prompt_chunk(w, b, 0, w.G, L, device) for b in range(w.S)])
    return torch.stack(qs), torch.stack(ks), torch.stack(vs)


def run_workload(w, units, mode, order, steps, lens=None, check_every=8, Lmax=None, ranks=0):
    """prefill + `steps` decode steps of workload w on the GPU, compared with the oracle on `units`."""
    tally = Tally()
    lens = W.prompt_lens(w) if lens is None else lens
    Lmax = max(lens) if Lmax is None else Lmax
    Q, K, V = prompt_tensors(w, Lmax)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    st = prefill_parity(cache, Q, K, V, lens, w.r, mode, units, tally, scale=w.scale)
    par = DecodeParity(cache, st, units, w.r, mode, order, tally, scale=w.scale, ranks=ranks)
    t_pos = list(lens)
    for i in range(steps):
        q, k, v = W.decode_tokens(w, i, t_pos, DEV)
        par.step(q, k, v, check_state=(i % check_every == check_every - 1) or i == steps - 1)
        t_pos = [t + 1 for t in t_pos]
    assert R.roco_device_status(cache) == 0
    return tally


@pytest.mark.parametrize("mode,order", MODES)
def test_toy_config_whole(mode, order):
    """fp32, 4 heads, d=64: prompt 256 -> B=128, then 64 decode steps with r=16; every unit, every step."""
    w = W.TOY
    t = run_workload(w, range(w.U), mode, order, w.steps, check_every=4)
    assert t.steps == 64 and t.decisions == 64 * 4
    assert t.near_ties <= 4, t


@pytest.mark.parametrize("mode,order", MODES)
@pytest.mark.parametrize("dtype,d,B", [("bf16", 128, 300), ("bf16", 64, 333), ("f32", 128, 100)])
@pytest.mark.parametrize("ranks", [0, 1])     # the shape roco_decode_step picks for so few units, and one CTA per unit
def test_fill_then_evict_ragged_tiles(mode, order, dtype, d, B, ranks):
    """Short prompts (cache not full): slots are appended until the buffer fills, then eviction starts.
    B is not a multiple of the tile height, and the live count crosses tile boundaries on the way."""
    w = W.scaled(W.LLAMA7B_DECODE, S=2, layers=1, heads=5, d=d, dtype=dtype, prompt_lo=B - 40, prompt_hi=B - 40,
                 B=B, r=7, steps=60)
    t = run_workload(w, range(w.U), mode, order, w.steps, lens=[B - 40, B - 55], check_every=10, Lmax=B - 40,
                     ranks=ranks)
    assert t.decisions >= 2 * 5 * 5


@pytest.mark.parametrize("scale", [0.0, -0.07])
@pytest.mark.parametrize("ranks,splits", [(1, 0), (2, 0), (0, 3)])   # one CTA per unit, a cluster of two, the split
@pytest.mark.parametrize("order", [R.ROCO_EVICT_FIRST, R.ROCO_ATTEND_FIRST])
def test_decode_with_a_scale_that_is_not_positive(scale, ranks, splits, order):
    """Eq. 1 with scale 0 (uniform attention) and with a negative scale: masks and maxima must act on the scaled
    scores."""
    B = 200
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=3, B=B, r=7)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    st = oracle.empty_state(w.U, B, w.d)
    tally = Tally()
    par = DecodeParity(cache, st, range(w.U), w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, order, tally, scale=scale,
                       ranks=ranks, splits=splits)
    for i in range(B + 12):
        par.step(*W.decode_tokens(w, i, [i], DEV), check_state=(i == B + 11))
    assert R.roco_device_status(cache) == 0


@pytest.mark.parametrize("ranks,splits", [(1, 0), (2, 0), (0, 3)])   # one CTA per unit, a cluster of two, the split
@pytest.mark.parametrize("order", [R.ROCO_EVICT_FIRST, R.ROCO_ATTEND_FIRST])
def test_free_slots_may_hold_anything(ranks, splits, order):
    """Slots past `live` are not part of the cache: NaN in their K, V and statistics changes nothing."""
    B, fill = 400, 170
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=3, B=B, r=7)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    st = oracle.empty_state(w.U, B, w.d)
    tally = Tally()
    par = DecodeParity(cache, st, range(w.U), w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, order, tally, scale=w.scale,
                       ranks=ranks, splits=splits)
    for i in range(fill):
        par.step(*W.decode_tokens(w, i, [i], DEV))
    cache.K[:, :, fill:] = float("nan"); cache.V[:, :, fill:] = float("nan")
    cache.s[:, :, fill:] = float("nan"); cache.q[:, :, fill:] = float("nan"); cache.n[:, :, fill:] = -7
    for i in range(fill, fill + 40):
        par.step(*W.decode_tokens(w, i, [i], DEV), check_state=(i == fill + 39))
    assert R.roco_device_status(cache) == 0 and bool(torch.isfinite(par.out.float()).all())


@pytest.mark.parametrize("ranks,splits", [(1, 0), (2, 0), (0, 3)])   # one CTA per unit, a cluster of two, the split
def test_evicted_token_would_have_held_the_maximum(ranks, splits):
    """The token that leaves in this step (lowest mean, no variance) has a key 30 times the query: under
    EVICT_FIRST its score is no part of the row, and a maximum that still saw it would wipe out the row."""
    B, L = 300, 330
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=3, prompt_lo=L, prompt_hi=L, B=B, r=9)
    Q, K, V = (torch.stack(x) for x in zip(*[W.prompt_chunk(w, b, 0, w.G, L, DEV) for b in range(w.S)]))
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    R.roco_prefill(Q, K, V, [L], w.B, w.r, cache, scale=w.scale)
    q, k, v = W.decode_tokens(w, 0, [L], DEV)
    for u in range(w.U):
        sl = 40 + 50 * u
        cache.s[0, u, sl] = 1e-6
        cache.q[0, u, sl] = 1e-12 / float(cache.n[0, u, sl])
        cache.K[0, u, sl] = (30.0 * q[0, u].float()).to(cache.K.dtype)
    tally = Tally()
    par = DecodeParity(cache, state_from_cache(cache, range(w.U)), range(w.U), w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R,
                       R.ROCO_EVICT_FIRST, tally, scale=w.scale, ranks=ranks, splits=splits)
    par.step(q, k, v, check_state=True)
    assert par.ev_slot[0].tolist() == [40, 90, 140]
    assert bool(torch.isfinite(par.out.float()).all()) and R.roco_device_status(cache) == 0


@pytest.mark.parametrize("kind", ["sink", "lowrank", "burst"])
def test_prefill_eviction_structured(kind):
    """Prefill with eviction to budget on the structured generators, ragged lengths, several column tiles."""
    w = W.scaled(W.LLAMA7B_PREFILL, S=3, layers=1, heads=3, prompt_lo=700, prompt_hi=700, B=200, r=31, kind=kind)
    t = run_workload(w, range(w.U), R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_EVICT_FIRST, 12, lens=[700, 333, 65],
                     check_every=4)
    assert t.prefill_swapped <= 4, t


@pytest.mark.parametrize("r", [1, 31, 200])
def test_prefill_eviction_lowest_r(r):
    """LOWEST_R at prefill: the evictions are replayed one by one on frozen statistics (sorted scope order)."""
    w = W.scaled(W.LLAMA7B_PREFILL, S=3, layers=1, heads=3, prompt_lo=700, prompt_hi=700, B=200, r=r, kind="sink")
    t = run_workload(w, range(w.U), R.ROCO_SCOPE_LOWEST_R, R.ROCO_EVICT_FIRST, 6, lens=[700, 333, 65], check_every=3)
    # six units evict (prompts of 700 and 333 tokens); most survivor sets equal the oracle's token for token, and
    # where they do not, each differing eviction was replayed inside the margin
    assert t.prefill_units_evicting == 6 and t.prefill_units_firm >= 4 and t.prefill_swapped <= 4, t


def test_prefill_keeps_everything_when_budget_not_binding():
    w = W.scaled(W.TOY, prompt_lo=90, prompt_hi=90, B=128, r=16)
    run_workload(w, range(w.U), R.ROCO_SCOPE_LOWEST_R, R.ROCO_EVICT_FIRST, 50, check_every=5)


def test_prefill_r_zero_and_r_equal_budget():
    for r in (0, 64):
        w = W.scaled(W.TOY, prompt_lo=200, prompt_hi=200, B=64, r=r)
        run_workload(w, range(w.U), R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_EVICT_FIRST, 0)


@pytest.mark.parametrize("mode,order", MODES)
def test_uniform_attention_position_ties(mode, order):
    """q = 0 everywhere: all probabilities are exactly 1/live, statistics of same-age tokens are bit-identical,
    and only the position rule decides.  No near-tie exclusions (strict)."""
    S, G, B, d, r = 1, 3, 40, 64, 5
    cache = R.Cache(S, G, B, d, torch.float32, DEV)
    st = oracle.empty_state(S * G, B, d)
    par = DecodeParity(cache, st, range(S * G), r, mode, order, Tally(), strict=True)
    g = torch.Generator(device=DEV); g.manual_seed(1)
    for i in range(B + 30):
        q = torch.zeros(S, G, d, device=DEV)
        k = torch.randn(S, G, d, device=DEV, generator=g)
        v = torch.randn(S, G, d, device=DEV, generator=g)
        par.step(q, k, v, check_state=(i % 10 == 9))
    assert R.roco_device_status(cache) == 0


def test_budget_of_one_and_scope_extremes():
    for mode, r, B in ((R.ROCO_SCOPE_EXCLUDE_TOP_R, 0, 1), (R.ROCO_SCOPE_LOWEST_R, 1, 1),
                       (R.ROCO_SCOPE_LOWEST_R, 1, 9), (R.ROCO_SCOPE_LOWEST_R, 9, 9), (R.ROCO_SCOPE_EXCLUDE_TOP_R, 8, 9)):
        for order in (R.ROCO_EVICT_FIRST, R.ROCO_ATTEND_FIRST):
            w = W.scaled(W.TOY, B=B, r=r)
            cache = R.Cache(w.S, w.G, B, w.d, torch.float32, DEV)
            st = oracle.empty_state(w.U, B, w.d)
            par = DecodeParity(cache, st, range(w.U), r, mode, order, Tally(), scale=w.scale)
            for i in range(B + 6):
                par.step(*W.decode_tokens(w, i, [i], DEV), check_state=True)


def test_maximum_budget():
    """B = 8192 (largest supported), one CTA per SM: fill by prefill, then evict for a few steps."""
    w = W.scaled(W.LONG_CONTEXT, S=1, layers=1, heads=2, prompt_lo=8192, prompt_hi=8192, B=8192, r=64, steps=3)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    # the state is built by streaming 8192 tokens through the oracle-free path: prefill with B >= L
    Q, K, V = prompt_tensors(w, 8192)
    R.roco_prefill(Q, K, V, [8192], w.B, w.r, cache, scale=w.scale)
    torch.cuda.synchronize()
    st = oracle.State(widen(unit_view(cache.K, range(2))), widen(unit_view(cache.V, range(2))),
                      widen(unit_view(cache.s, range(2))), widen(unit_view(cache.q, range(2))),
                      unit_view(cache.n, range(2)).cpu().numpy().copy(), unit_view(cache.pos, range(2)).cpu().numpy().copy(),
                      unit_view(cache.live, range(2)).cpu().numpy().copy(), unit_view(cache.t_next, range(2)).cpu().numpy().copy())
    assert np.all(st.live == 8192)
    par = DecodeParity(cache, st, range(2), w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_EVICT_FIRST, Tally(), scale=w.scale)
    for i in range(w.steps):
        par.step(*W.decode_tokens(w, i, [8192 + i], DEV), check_state=(i == w.steps - 1))
    assert R.roco_device_status(cache) == 0


def test_checkpoint_resume_is_bit_exact():
    """The whole state is {K,V,s,q,n,pos,live,t_next}: 12 steps == 6 steps, copy to fresh buffers, 6 steps."""
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=6, prompt_lo=100, prompt_hi=100, B=80, r=9)
    Q, K, V = prompt_tensors(w, 100)
    outs = []
    for split in (False, True):
        cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
        R.roco_prefill(Q, K, V, [100], w.B, w.r, cache, scale=w.scale)
        out = torch.zeros(w.S, w.G, w.d, dtype=w.torch_dtype, device=DEV)
        ev = torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV)
        for i in range(12):
            if split and i == 6:
                fresh = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
                for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
                    getattr(fresh, name).copy_(getattr(cache, name))
                cache = fresh
            R.roco_decode_step(cache, *W.decode_tokens(w, i, [100 + i], DEV), w.r, out, ev, scale=w.scale)
        torch.cuda.synchronize()
        outs.append([getattr(cache, n).clone() for n in ("K", "V", "s", "q", "n", "pos", "live", "t_next")] + [out.clone()])
    for a, b in zip(*outs):
        assert torch.equal(a, b)


@pytest.mark.parametrize("layers,heads,B", [(1, 4, 128), (32, 33, 32)])
def test_host_buffer_variant_matches_device_variant(layers, heads, B):
    """Host-buffer step against the device-buffer step, bit for bit: 8 units (one launch) and 2112 units (the
    step is cut into four unit ranges whose copies overlap the kernels; 2112 is not a multiple of four ranges of
    equal size times anything convenient, and 33 heads make the ranges straddle sequences)."""
    w = W.scaled(W.LLAMA7B_DECODE, S=2, layers=layers, heads=heads, prompt_lo=150, prompt_hi=150, B=B, r=8)
    Q, K, V = prompt_tensors(w, 150)
    caches = [R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV) for _ in range(2)]
    for c in caches:
        R.roco_prefill(Q, K, V, [150, 150], w.B, w.r, c, scale=w.scale)
    out = torch.zeros(w.S, w.G, w.d, dtype=w.torch_dtype, device=DEV)
    ev = torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV)
    evp = torch.zeros_like(ev)
    staging = torch.empty(R.roco_decode_host_staging_bytes(caches[1]), dtype=torch.uint8, device=DEV)
    h_out = torch.zeros(w.S, w.G, w.d, dtype=w.torch_dtype).pin_memory()
    h_ev = torch.zeros(w.S, w.G, dtype=torch.int32).pin_memory()
    h_evp = torch.zeros(w.S, w.G, dtype=torch.int32).pin_memory()
    for i in range(5):
        q, k, v = W.decode_tokens(w, i, [150 + i] * 2, DEV)
        R.roco_decode_step(caches[0], q, k, v, w.r, out, ev, evp, scale=w.scale)
        R.roco_decode_step_host(caches[1], q.cpu().pin_memory(), k.cpu().pin_memory(), v.cpu().pin_memory(), w.r,
                                h_out, h_ev, h_evp, staging, scale=w.scale)
        torch.cuda.synchronize()
        assert torch.equal(out.cpu(), h_out) and torch.equal(ev.cpu(), h_ev) and torch.equal(evp.cpu(), h_evp)
    assert torch.equal(caches[0].s, caches[1].s) and torch.equal(caches[0].K, caches[1].K)


def test_pipelined_host_buffer_steps_match_device_steps():
    """begin/end form of the host-buffer step (two steps in flight, copies of one under the kernel of the other)
    against the device-buffer step, bit for bit, over 7 steps; and the in-flight rules."""
    w = W.scaled(W.LLAMA7B_DECODE, S=2, layers=4, heads=8, prompt_lo=150, prompt_hi=150, B=96, r=8)
    Q, K, V = prompt_tensors(w, 150)
    caches = [R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV) for _ in range(2)]
    for c in caches:
        R.roco_prefill(Q, K, V, [150, 150], w.B, w.r, c, scale=w.scale)
    n = 7
    toks = [W.decode_tokens(w, i, [150 + i] * 2, DEV) for i in range(n)]
    want = []
    out = torch.zeros(w.S, w.G, w.d, dtype=w.torch_dtype, device=DEV)
    ev = torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV)
    evp = torch.zeros_like(ev)
    for q, k, v in toks:
        R.roco_decode_step(caches[0], q, k, v, w.r, out, ev, evp, scale=w.scale)
        want.append((out.cpu().clone(), ev.cpu().clone(), evp.cpu().clone()))
    staging = torch.empty(R.roco_decode_host_pipeline_staging_bytes(caches[1]), dtype=torch.uint8, device=DEV)
    h_in = [tuple(x.cpu().pin_memory() for x in t) for t in toks]
    h_out = [(torch.zeros(w.S, w.G, w.d, dtype=w.torch_dtype).pin_memory(),
              torch.zeros(w.S, w.G, dtype=torch.int32).pin_memory(),
              torch.zeros(w.S, w.G, dtype=torch.int32).pin_memory()) for _ in range(n)]
    with pytest.raises(R.RocoError) as e:
        R.roco_decode_step_host_end()                                   # nothing in flight
    assert e.value.code == 5
    for i in range(n):
        R.roco_decode_step_host_begin(caches[1], *h_in[i], w.r, *h_out[i], staging, scale=w.scale)
        if i == 1:
            with pytest.raises(R.RocoError) as e:                       # a third step without an end
                R.roco_decode_step_host_begin(caches[1], *h_in[2], w.r, *h_out[2], staging, scale=w.scale)
            assert e.value.code == 5
        if i >= 1:
            R.roco_decode_step_host_end()                               # step i - 1 is complete
            for a, b in zip(want[i - 1], h_out[i - 1]):
                assert torch.equal(a, b)
    R.roco_decode_step_host_end()
    for a, b in zip(want[n - 1], h_out[n - 1]):
        assert torch.equal(a, b)
    torch.cuda.synchronize()
    for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
        assert torch.equal(getattr(caches[0], name), getattr(caches[1], name)), name
    assert R.roco_device_status(caches[1]) == 0


def test_llama7b_decode_shape_sampled_units():
    """The benchmark's launch configuration (8192 units, B=1024, d=128, bf16, r=64): the cache is built by the
    library's prefill from 2048-token prompts, layer-chunk by layer-chunk; 64 sampled units are followed by the
    oracle through the prefill and 6 decode steps."""
    w = W.LLAMA7B_DECODE
    tally = Tally()
    rng = np.random.default_rng(0)
    units = sorted(rng.choice(w.U, 64, replace=False).tolist())
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    L = w.prompt_lo
    chunk = 256                                  # units per prefill call (keeps Q,K,V at 3 x 128 MiB)
    states = {}
    for b in range(w.S):
        for g0 in range(0, w.G, chunk):
            Q, K, V = (t[None] for t in W.prompt_chunk(w, b, g0, g0 + chunk, L, DEV))
            sub = R.Cache(1, chunk, w.B, w.d, w.torch_dtype, DEV)
            local = [u - (b * w.G + g0) for u in units if b * w.G + g0 <= u < b * w.G + g0 + chunk]
            if local:
                st = prefill_parity(sub, Q, K, V, [L], w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, local, tally, scale=w.scale)
                for i, lu in enumerate(local):
                    states[b * w.G + g0 + lu] = (st, i)
            else:
                R.roco_prefill(Q, K, V, [L], w.B, w.r, sub, scale=w.scale)
            for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
                getattr(cache, name)[b, g0:g0 + chunk].copy_(getattr(sub, name)[0])
            assert R.roco_device_status(sub) == 0
    st = oracle.empty_state(len(units), w.B, w.d)
    for j, u in enumerate(units):
        src, i = states[u]
        for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
            getattr(st, name)[j] = getattr(src, name)[i]
    par = DecodeParity(cache, st, units, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_EVICT_FIRST, tally, scale=w.scale)
    t_pos = [L] * w.S
    for i in range(6):
        par.step(*W.decode_tokens(w, i, t_pos, DEV), check_state=(i == 5))
        t_pos = [t + 1 for t in t_pos]
    assert R.roco_device_status(cache) == 0
    assert tally.decisions == 6 * 64
    # properties that hold for every unit at any size
    assert int(cache.live.min()) == w.B and int(cache.live.max()) == w.B
    assert int(cache.t_next.min()) == L + 6
    np.testing.assert_array_equal((cache.n == (L + 6 - cache.pos)).all().item(), True)   # Count = age
    srt = cache.pos.sort(dim=-1).values
    assert bool((srt[..., 1:] > srt[..., :-1]).all())                                   # live positions distinct
