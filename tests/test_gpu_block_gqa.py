"""GPU parity of the multi-query steps: block-wise evict-and-encode (b tokens per step) and grouped-query decode
(several query heads per key-value head), against the oracle on every unit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2402_06262_b200 as R
import workloads as W
from harness import (BlockParity, DecodeParity, GqaBlockParity, GqaParity, Tally, prefill_parity, state_from_cache, unit_view,
                     widen)

pytestmark = pytest.mark.gpu
DEV = "cuda"


def prompt_tensors(w, L):
    qs, ks, vs = zip(*[W.prompt_chunk(w, b, 0, w.G, L, DEV) for b in range(w.S)])
    return torch.stack(qs), torch.stack(ks), torch.stack(vs)


def block_tokens(w, step0, b, t_pos):
    toks = [W.decode_tokens(w, step0 + i, [t + i for t in t_pos], DEV) for i in range(b)]
    return tuple(torch.stack([t[k] for t in toks], dim=2).contiguous() for k in range(3))   # [S][G][b][d]


def prefilled(w, L, tally, units):
    Q, K, V = prompt_tensors(w, L)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    st = prefill_parity(cache, Q, K, V, [L] * w.S, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, units, tally, scale=w.scale)
    return cache, st


@pytest.mark.parametrize("b", [1, 2, 4, 8, 12, 16])
@pytest.mark.parametrize("dtype,d,B", [("bf16", 128, 300), ("bf16", 128, 302), ("f32", 64, 128)])
def test_block_steps_fill_then_evict(b, dtype, d, B):
    """Short prompt: the first block steps only fill free slots (some mix freed and free slots), later ones evict
    b tokens each.  B = 300 takes the tensor-core kernel with the statistics staged by bulk copy, B = 302 (unit
    offsets not 16-byte aligned) the same kernel with plain loads, fp32 / d = 64 the CUDA-core kernel."""
    w = W.scaled(W.LLAMA7B_DECODE, S=2, layers=1, heads=3, d=d, dtype=dtype, prompt_lo=B - 21, prompt_hi=B - 21,
                 B=B, r=9)
    tally = Tally()
    cache, st = prefilled(w, B - 21, tally, range(w.U))
    par = BlockParity(cache, st, range(w.U), b, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, tally, scale=w.scale)
    t = B - 21
    for i in range(max(4, 40 // b)):
        par.step(*block_tokens(w, i * b, b, [t] * w.S), check_state=True)
        t += b
    assert R.roco_device_status(cache) == 0
    assert tally.decisions > 0


@pytest.mark.parametrize("b", [2, 5, 16])
@pytest.mark.parametrize("r", [1, 9, 150, 290])
@pytest.mark.parametrize("dtype,d,B", [("bf16", 128, 300), ("f32", 64, 128)])
def test_block_steps_lowest_r_scope_refills(b, r, dtype, d, B):
    """The other reading of the scope (the r lowest-variance tokens): within one block step the scope refills
    after every eviction.  r = 1 (each victim is the lowest-variance token left), a small scope, one that is half
    the cache, and one larger than what is left after a few evictions (the scope is then everything)."""
    r = min(r, B - b)
    w = W.scaled(W.LLAMA7B_DECODE, S=2, layers=1, heads=3, d=d, dtype=dtype, prompt_lo=B - 21, prompt_hi=B - 21,
                 B=B, r=r)
    tally = Tally()
    cache, st = prefilled(w, B - 21, tally, range(w.U))
    par = BlockParity(cache, st, range(w.U), b, r, R.ROCO_SCOPE_LOWEST_R, tally, scale=w.scale)
    t = B - 21
    for i in range(max(4, 48 // b)):
        par.step(*block_tokens(w, i * b, b, [t] * w.S), check_state=True)
        t += b
    assert R.roco_device_status(cache) == 0
    assert tally.decisions > 0 and tally.near_ties <= max(4, tally.decisions // 4), tally


@pytest.mark.parametrize("scale", [0.0, -0.05])
def test_block_steps_with_a_scale_that_is_not_positive(scale):
    """Eq. 1 with scale 0 (uniform attention over what a query may see) and with a negative scale (the largest raw
    score is then the smallest scaled one, which the tensor-memory kernel's row maxima do not cover: the step must
    take another kernel and still match)."""
    B, b = 300, 8
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=3, prompt_lo=B - 10, prompt_hi=B - 10, B=B, r=9)
    tally = Tally()
    Q, K, V = prompt_tensors(w, B - 10)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    st = prefill_parity(cache, Q, K, V, [B - 10], w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, range(w.U), tally, scale=w.scale)
    par = BlockParity(cache, st, range(w.U), b, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, tally, scale=scale)
    t = B - 10
    for i in range(4):
        par.step(*block_tokens(w, i * b, b, [t]), check_state=True)
        t += b
    assert R.roco_device_status(cache) == 0


@pytest.mark.parametrize("b,group", [(16, 1), (4, 4), (1, 8), (2, 1)])
@pytest.mark.parametrize("B", [300, 1000])
def test_free_slots_may_hold_anything(b, group, B):
    """Slots past `live` are not part of the cache (the caller's buffers need not be cleared): with NaN in their K
    and V rows and in their statistics, steps that fill them must give what they give on a clean buffer."""
    L = B - 150
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=2, prompt_lo=L, prompt_hi=L, B=B, r=9)
    tally = Tally()
    cache, st = prefilled(w, L, tally, range(w.U))
    cache.K[:, :, L:] = float("nan"); cache.V[:, :, L:] = float("nan")
    cache.s[:, :, L:] = float("nan"); cache.q[:, :, L:] = float("nan"); cache.n[:, :, L:] = -7; cache.pos[:, :, L:] = 123456
    par = (GqaBlockParity(cache, st, range(w.U), b, group, w.r, tally, scale=w.scale) if group > 1 else
           BlockParity(cache, st, range(w.U), b, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, tally, scale=w.scale))
    t = L
    for i in range(3):
        toks = grouped_block_tokens(w, i * b, b, group, [t]) if group > 1 else block_tokens(w, i * b, b, [t])
        par.step(*toks, check_state=False)
        t += b
    assert R.roco_device_status(cache) == 0
    assert bool(torch.isfinite(par.out.float()).all())
    live = int(cache.live[0, 0])
    assert live == L + 3 * b
    for name in ("s", "q"):
        assert bool(torch.isfinite(getattr(cache, name)[:, :, :live]).all())
    assert bool(torch.isfinite(cache.K[:, :, :live].float()).all()) and bool(torch.isfinite(cache.V[:, :, :live].float()).all())


@pytest.mark.parametrize("b", [2, 4, 16])   # warp-level-MMA kernel; tcgen05 kernel with 8 and with 16 query columns
def test_evicted_tokens_held_the_row_maxima(b):
    """The tokens that leave in this step have, by construction, by far the largest scores of every row (keys 30
    times the first new query) and the lowest means: a row maximum taken before the selection is known would sit
    hundreds of binary orders above every score that remains, and the exponentials of the row would all vanish."""
    B, L = 300, 330
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=2, prompt_lo=L, prompt_hi=L, B=B, r=9)
    tally = Tally()
    cache, _ = prefilled(w, L, tally, range(w.U))
    toks = block_tokens(w, 0, b, [L])
    slots = [5, 77, 150, 290, 11, 23, 35, 47, 59, 61, 83, 95, 107, 119, 131, 143][:b]
    slots.sort()
    for u in range(w.U):
        for sl in slots:
            n = float(cache.n[0, u, sl])
            cache.s[0, u, sl] = 1e-6
            cache.q[0, u, sl] = 1e-12 / n          # variance 0, mean the lowest: in scope and first to go
            cache.K[0, u, sl] = (30.0 * toks[0][0, u, 0].float()).to(cache.K.dtype)
    par = BlockParity(cache, state_from_cache(cache, range(w.U)), range(w.U), b, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, tally,
                      scale=w.scale)
    par.step(*toks, check_state=True)
    assert sorted(par.ev_slot[0, 0].tolist()) == slots and sorted(par.ev_slot[0, 1].tolist()) == slots
    assert bool(torch.isfinite(par.out.float()).all()) and R.roco_device_status(cache) == 0


def test_block_step_after_eviction_prefill_llama_shape():
    """Evict-and-encode with b = 16 on a cache built by prefill eviction (B = 1024, d = 128, bf16, sinks)."""
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=8, prompt_lo=1500, prompt_hi=1500)
    tally = Tally()
    cache, st = prefilled(w, 1500, tally, range(w.U))
    par = BlockParity(cache, st, range(w.U), 16, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, tally, scale=w.scale)
    for i in range(3):
        par.step(*block_tokens(w, 16 * i, 16, [1500 + 16 * i]), check_state=(i == 2))
    assert tally.decisions == 3 * 16 * w.U


@pytest.mark.parametrize("B,b", [(2048, 16), (3000, 8), (3968, 16), (4000, 12), (4096, 16)])
def test_block_step_large_budget(B, b):
    """Budgets that leave room for one CTA per SM only (more ring stages, up to 32 tiles of 128 keys; with 32 the output accumulator shares tensor-memory columns with the first tile)."""
    L = B + 300
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=4, prompt_lo=L, prompt_hi=L, B=B, r=64)
    tally = Tally()
    cache, st = prefilled(w, L, tally, range(w.U))
    par = BlockParity(cache, st, range(w.U), b, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, tally, scale=w.scale)
    for i in range(3):
        par.step(*block_tokens(w, b * i, b, [L + b * i]), check_state=(i == 2))
    assert R.roco_device_status(cache) == 0
    assert tally.decisions == 3 * b * w.U


def test_block_of_one_equals_decode_step_bitwise():
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=4, prompt_lo=200, prompt_hi=200, B=128, r=8)
    Q, K, V = prompt_tensors(w, 200)
    caches = [R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV) for _ in range(2)]
    for c in caches:
        R.roco_prefill(Q, K, V, [200], w.B, w.r, c, scale=w.scale)
    out = torch.zeros(w.S, w.G, w.d, dtype=w.torch_dtype, device=DEV)
    outb = torch.zeros(w.S, w.G, 1, w.d, dtype=w.torch_dtype, device=DEV)
    ev = torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV)
    evb = torch.zeros(w.S, w.G, 1, dtype=torch.int32, device=DEV)
    for i in range(6):
        q, k, v = W.decode_tokens(w, i, [200 + i], DEV)
        R.roco_decode_step(caches[0], q, k, v, w.r, out, ev, scale=w.scale)
        R.roco_block_step(caches[1], q[:, :, None].contiguous(), k[:, :, None].contiguous(), v[:, :, None].contiguous(),
                          w.r, outb, evb, scale=w.scale)
        torch.cuda.synchronize()
        assert torch.equal(ev, evb[..., 0])
        assert (out.float() - outb[:, :, 0].float()).abs().max() <= 2e-2
    assert torch.equal(caches[0].pos, caches[1].pos) and torch.equal(caches[0].n, caches[1].n)
    np.testing.assert_allclose(caches[1].s.cpu().numpy(), caches[0].s.cpu().numpy(), rtol=1e-5)


def test_block_step_argument_checks():
    w = W.scaled(W.TOY, B=32, r=4)
    cache = R.Cache(w.S, w.G, w.B, w.d, torch.float32, DEV)
    mk = lambda b: torch.zeros(w.S, w.G, b, w.d, device=DEV)
    out = lambda b: (torch.zeros(w.S, w.G, b, w.d, device=DEV), torch.zeros(w.S, w.G, b, dtype=torch.int32, device=DEV))
    with pytest.raises(R.RocoError) as e:
        R.roco_block_step(cache, mk(17), mk(17), mk(17), 4, *out(17))
    assert e.value.code == 2
    with pytest.raises(R.RocoError) as e:
        R.roco_block_step(cache, mk(8), mk(8), mk(8), 25, *out(8))        # r + b > B
    assert e.value.code == 1


@pytest.mark.parametrize("group", [1, 2, 4, 8, 16])
@pytest.mark.parametrize("mode", [R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_SCOPE_LOWEST_R])
def test_gqa_decode_steps(group, mode):
    """Zephyr-like grouping: `group` query heads per key-value head, statistics from the group mean."""
    w = W.scaled(W.LLAMA7B_DECODE, S=2, layers=1, heads=4, prompt_lo=260, prompt_hi=260, B=200, r=12)
    tally = Tally()
    cache, st = prefilled(w, 260, tally, range(w.U))
    par = GqaParity(cache, st, range(w.U), group, w.r, mode, tally, scale=w.scale)
    for i in range(10):
        qs = [W.decode_tokens(w, 1000 * g + i, [260 + i] * w.S, DEV)[0] for g in range(group)]
        _, k, v = W.decode_tokens(w, i, [260 + i] * w.S, DEV)
        par.step(torch.stack(qs, dim=2).contiguous(), k, v, check_state=(i % 3 == 2))
    assert R.roco_device_status(cache) == 0 and tally.decisions == 10 * w.U


@pytest.mark.parametrize("b", [1, 4, 16])
@pytest.mark.parametrize("lens", [[150, 97], [150, 150, 150]])
def test_blockwise_prompt_encoding(b, lens):
    """The paper's prefill scheme: the whole prompt goes through the budgeted cache b tokens at a time (ragged
    prompt lengths, last block shorter; equal lengths, which the library batches into one launch per block).
    Every sequence is compared: the same entry point is also driven one block per call on a second cache, next to
    the oracle, which continues from the GPU's freed slots at decisions inside the margin; the one-call cache must
    then equal the block-by-block one bit for bit."""
    w = W.scaled(W.LLAMA7B_DECODE, S=len(lens), layers=1, heads=3, prompt_lo=150, prompt_hi=150, B=64, r=6)
    Q, K, V = prompt_tensors(w, 150)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    out = torch.zeros_like(Q)
    ev = torch.zeros(w.S, w.G, b, dtype=torch.int32, device=DEV)
    R.roco_prefill_blockwise(Q, K, V, lens, b, w.r, cache, out, ev, scale=w.scale)
    torch.cuda.synchronize()
    assert R.roco_device_status(cache) == 0
    from harness import compare_state, out_tol
    tally = Tally()
    for s, L in enumerate(lens):
        sub = R.Cache(1, w.G, w.B, w.d, w.torch_dtype, DEV)
        st = oracle.empty_state(w.G, w.B, w.d)
        Qs, Ks, Vs = (widen(x[s]) for x in (Q, K, V))
        for t0 in range(0, L, b):
            m = min(b, L - t0)
            blk = [x[s:s + 1, :, t0:t0 + m].contiguous() for x in (Q, K, V)]
            o1 = torch.zeros_like(blk[0])
            e1 = torch.full((1, w.G, m), -7, dtype=torch.int32, device=DEV)
            R.roco_prefill_blockwise(*blk, [m], m, w.r, sub, o1, e1, scale=w.scale)
            torch.cuda.synchronize()
            g_slot = e1[0].cpu().numpy()
            res = oracle.block_step(st, Qs[:, t0:t0 + m], Ks[:, t0:t0 + m], Vs[:, t0:t0 + m], w.r,
                                    R.ROCO_SCOPE_EXCLUDE_TOP_R, w.scale, delta=1e-5, force_slots=g_slot)
            firm = res.near_tie == 0
            np.testing.assert_array_equal(g_slot[firm], res.choice[firm], err_msg="freed slots differ outside the margin")
            np.testing.assert_array_equal(g_slot, res.evicted_slot)
            tally.near_ties += int((~firm).sum())
            tally.decisions += int((res.choice >= 0).sum())
            assert np.abs(widen(o1[0]) - res.out).max() <= out_tol(w.torch_dtype)
            assert torch.equal(o1[0], out[s, :, t0:t0 + m]), "one-call and block-by-block outputs differ"
        compare_state(sub, st, range(w.G), f"sequence {s}")
        for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
            assert torch.equal(getattr(sub, name)[0], getattr(cache, name)[s]), name
        assert int(cache.live[s].min()) == min(L, w.B) and int(cache.t_next[s].max()) == L
        assert R.roco_device_status(sub) == 0
    assert tally.decisions >= sum(max(0, L - w.B) for L in lens) * w.G
    assert tally.near_ties <= tally.decisions // 10, tally


def grouped_block_tokens(w, step0, b, group, t_pos):
    """Q [S][G][b][group][d] (head g of token i drawn as an independent query), K_new, V_new [S][G][b][d]."""
    toks = [W.decode_tokens(w, step0 + i, [t + i for t in t_pos], DEV) for i in range(b)]
    K = torch.stack([t[1] for t in toks], dim=2).contiguous()
    V = torch.stack([t[2] for t in toks], dim=2).contiguous()
    Q = torch.stack([torch.stack([W.decode_tokens(w, 1000 * (g + 1) + step0 + i, [t + i for t in t_pos], DEV)[0]
                                  for g in range(group)], dim=2) for i in range(b)], dim=2).contiguous()
    return Q, K, V


@pytest.mark.parametrize("b,group", [(2, 2), (4, 4), (2, 8), (8, 2), (3, 5), (4, 1), (1, 4)])
@pytest.mark.parametrize("dtype,d,B", [("bf16", 128, 300), ("bf16", 128, 302), ("f32", 64, 128)])
def test_grouped_block_steps_fill_then_evict(b, group, dtype, d, B):
    """Block-wise evict-and-encode on key-value heads shared by `group` query heads (the paper's block-wise
    experiment on a grouped-query model): fill phase, mixed phase, eviction of b tokens per step; tensor-core
    kernel with staged and with plainly loaded statistics, and the CUDA-core kernel."""
    w = W.scaled(W.LLAMA7B_DECODE, S=2, layers=1, heads=3, d=d, dtype=dtype, prompt_lo=B - 21, prompt_hi=B - 21,
                 B=B, r=9)
    tally = Tally()
    cache, st = prefilled(w, B - 21, tally, range(w.U))
    par = GqaBlockParity(cache, st, range(w.U), b, group, w.r, tally, scale=w.scale)
    t = B - 21
    for i in range(max(4, 40 // b)):
        par.step(*grouped_block_tokens(w, i * b, b, group, [t] * w.S), check_state=True)
        t += b
    assert R.roco_device_status(cache) == 0 and tally.decisions > 0


def test_grouped_block_step_llama_shape():
    """B = 1024, d = 128, bf16 after prefill eviction: 4 tokens x 4 heads per step (16 query rows)."""
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=8, prompt_lo=1500, prompt_hi=1500)
    tally = Tally()
    cache, st = prefilled(w, 1500, tally, range(w.U))
    par = GqaBlockParity(cache, st, range(w.U), 4, 4, w.r, tally, scale=w.scale)
    for i in range(3):
        par.step(*grouped_block_tokens(w, 4 * i, 4, 4, [1500 + 4 * i]), check_state=(i == 2))
    assert tally.decisions == 3 * 4 * w.U


def test_block_steps_at_the_benchmark_size():
    """The launch configuration the bench times: all 8192 units of the Llama-7B decode shape (B = 1024, d = 128,
    bf16) in one call, b = 16 and then 4 tokens x 4 heads; sampled units (first, last, some between) follow the
    oracle from the cache the prefill left, every unit obeys the invariants."""
    w = W.LLAMA7B_DECODE
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    L = 1500
    for s in range(w.S):
        for g0 in range(0, w.G, 256):
            Q, K, V = (t[None] for t in W.prompt_chunk(w, s, g0, g0 + 256, L, DEV))
            sub = R.Cache(1, 256, w.B, w.d, w.torch_dtype, DEV)
            R.roco_prefill(Q, K, V, [L], w.B, w.r, sub, scale=w.scale)
            for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
                getattr(cache, name)[s, g0:g0 + 256].copy_(getattr(sub, name)[0])
    units = [0, 1, 777, 4095, 4096, 8190, 8191]
    tally = Tally()
    par = BlockParity(cache, state_from_cache(cache, units), units, 16, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, tally,
                      scale=w.scale)
    t = L
    for i in range(2):
        par.step(*block_tokens(w, 16 * i, 16, [t] * w.S), check_state=(i == 1))
        t += 16
    assert tally.decisions == 2 * 16 * len(units)
    gpar = GqaBlockParity(cache, state_from_cache(cache, units), units, 4, 4, w.r, tally, scale=w.scale)
    for i in range(2):
        gpar.step(*grouped_block_tokens(w, 100 + 4 * i, 4, 4, [t] * w.S), check_state=(i == 1))
        t += 4
    assert R.roco_device_status(cache) == 0
    assert int(cache.live.min()) == w.B == int(cache.live.max())
    assert int(cache.t_next.min()) == t == int(cache.t_next.max())
    assert bool((cache.n == (t - cache.pos)).all())           # Count = age for every slot of every unit
    srt = cache.pos.sort(-1).values
    assert bool((srt[..., 1:] > srt[..., :-1]).all())          # live positions distinct


def test_grouped_blockwise_prompt_encoding_equals_grouped_block_steps():
    """roco_prefill_blockwise_gqa (strided prompt tensors, ragged lengths) against the same blocks fed one by one
    through roco_gqa_block_step, which the tests above hold against the oracle: bit-equal caches and outputs."""
    b, group = 4, 2
    w = W.scaled(W.LLAMA7B_DECODE, S=2, layers=1, heads=3, prompt_lo=90, prompt_hi=90, B=48, r=5)
    lens = [90, 61]
    _, K, V = prompt_tensors(w, 90)
    g = torch.Generator(device=DEV); g.manual_seed(3)
    Q = torch.randn(w.S, w.G, 90, group, w.d, device=DEV, generator=g).to(w.torch_dtype)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    out = torch.zeros_like(Q)
    ev = torch.zeros(w.S, w.G, b, dtype=torch.int32, device=DEV)
    R.roco_prefill_blockwise_gqa(Q, K, V, lens, b, w.r, cache, out, ev, scale=w.scale)
    for s, L in enumerate(lens):
        sub = R.Cache(1, w.G, w.B, w.d, w.torch_dtype, DEV)
        for t0 in range(0, L, b):
            m = min(b, L - t0)
            o1 = torch.zeros(1, w.G, m, group, w.d, dtype=w.torch_dtype, device=DEV)
            e1 = torch.zeros(1, w.G, m, dtype=torch.int32, device=DEV)
            R.roco_gqa_block_step(sub, Q[s:s + 1, :, t0:t0 + m].contiguous(), K[s:s + 1, :, t0:t0 + m].contiguous(),
                                  V[s:s + 1, :, t0:t0 + m].contiguous(), w.r, o1, e1, scale=w.scale)
            assert torch.equal(o1[0], out[s, :, t0:t0 + m])
        for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
            assert torch.equal(getattr(sub, name)[0], getattr(cache, name)[s]), name
    assert R.roco_device_status(cache) == 0
