"""GPU parity at the sizes of the other workloads (prefill-stage eviction at L = 8192, ragged serving batch,
long context): sampled units / rows / columns that the oracle can compute one by one, plus properties that
hold for every unit at any size."""
import numpy as np
import pytest
import torch

import oracle
import paper_2402_06262_b200 as R
import workloads as W
from harness import DecodeParity, Tally, assert_stats_close, prefill_parity, state_from_cache, unit_view, widen

pytestmark = pytest.mark.gpu
DEV = "cuda"


def check_prefill_properties(sf, qf, lens, G):
    """Every query's probabilities sum to 1 => the column sums of a unit add up to its prompt length;
    0 <= q <= s."""
    for b, L in enumerate(lens):
        tot = sf[b, :, :L].double().sum(-1)
        assert float((tot - L).abs().max()) <= 2e-4 * L
        assert bool((qf[b, :, :L] <= sf[b, :, :L] * (1 + 1e-6) + 1e-30).all()) and bool((qf[b, :, :L] >= 0).all())


def test_llama7b_prefill_shape_sampled_units():
    """Prefill-stage eviction, L = 8192 -> B = 2048, r = 256, low-rank structured Q/K: 8 layers (256 units) on the
    tensor-core path; 3 sampled units go through the oracle in full."""
    w = W.scaled(W.LLAMA7B_PREFILL, layers=8)
    L = w.prompt_lo
    tally = Tally()
    Q, K, V = (t[None] for t in W.prompt_chunk(w, 0, 0, w.G, L, DEV))
    cache = R.Cache(1, w.G, w.B, w.d, w.torch_dtype, DEV)
    assert R.roco_prefill_uses_tensor_cores(cache)
    units = [3, 100, 255]
    prefill_parity(cache, Q, K, V, [L], w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, units, tally, scale=w.scale)
    sf = torch.zeros(1, w.G, L, device=DEV); qf = torch.zeros_like(sf)
    R.roco_prefill(Q, K, V, [L], w.B, w.r, cache, scale=w.scale, s_full=sf, q_full=qf)
    check_prefill_properties(sf, qf, [L], w.G)
    assert int(cache.live.min()) == w.B == int(cache.live.max())
    assert bool((cache.pos[..., 1:] > cache.pos[..., :-1]).all())
    assert bool((cache.n == L - cache.pos).all())
    assert tally.prefill_swapped <= 6, tally


def test_serving_batch_ragged_prompts():
    """13B-shape serving batch with ragged prompts (1024..4096), B = 512, r = 32: 4 sequences x 1600 units;
    prefill per sequence, then decode steps over the whole batch; sampled units followed by the oracle."""
    w = W.scaled(W.LLAMA13B_SERVING, S=4)
    lens = W.prompt_lens(w)
    assert len(set(lens)) > 1 and min(lens) >= 1024 and max(lens) <= 4096
    tally = Tally()
    rng = np.random.default_rng(4)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    states, units = [], []
    for b in range(w.S):
        Q, K, V = (t[None] for t in W.prompt_chunk(w, b, 0, w.G, lens[b], DEV))
        sub = R.Cache(1, w.G, w.B, w.d, w.torch_dtype, DEV)
        local = sorted(rng.choice(w.G, 3, replace=False).tolist())
        st = prefill_parity(sub, Q, K, V, [lens[b]], w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, local, tally, scale=w.scale)
        for i, lu in enumerate(local):
            units.append(b * w.G + lu)
            states.append((st, i))
        for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
            getattr(cache, name)[b].copy_(getattr(sub, name)[0])
        assert R.roco_device_status(sub) == 0
    st = oracle.empty_state(len(units), w.B, w.d)
    for j, (src, i) in enumerate(states):
        for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
            getattr(st, name)[j] = getattr(src, name)[i]
    par = DecodeParity(cache, st, units, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_EVICT_FIRST, tally, scale=w.scale)
    t_pos = list(lens)
    for i in range(5):
        par.step(*W.decode_tokens(w, i, t_pos, DEV), check_state=(i == 4))
        t_pos = [t + 1 for t in t_pos]
    assert R.roco_device_status(cache) == 0
    for b in range(w.S):
        assert int(cache.t_next[b].min()) == lens[b] + 5 == int(cache.t_next[b].max())
        assert bool((cache.n[b] == (lens[b] + 5 - cache.pos[b])).all())


@pytest.mark.parametrize("r", [16, 64, 256])
def test_long_context_prefill_and_decode(r):
    """Long context: L = 32768 -> B = 4096 with recurring key bursts; 2 layers (64 units).  The oracle checks the
    row LSE of sampled rows and the column statistics of sampled late columns (each needs only the rows after
    it), the invariants cover every unit, and decode steps continue from the GPU's cache on sampled units."""
    w = W.scaled(W.LONG_CONTEXT, S=1, layers=2, r=r)
    L = w.prompt_lo
    Q, K, V = (t[None] for t in W.prompt_chunk(w, 0, 0, w.G, L, DEV))
    cache = R.Cache(1, w.G, w.B, w.d, w.torch_dtype, DEV)
    lse = torch.zeros(1, w.G, L, device=DEV); sf = torch.zeros_like(lse); qf = torch.zeros_like(lse)
    R.roco_prefill(Q, K, V, [L], w.B, w.r, cache, scale=w.scale, lse_out=lse, s_full=sf, q_full=qf)
    torch.cuda.synchronize()
    assert R.roco_device_status(cache) == 0
    check_prefill_properties(sf, qf, [L], w.G)
    assert int(cache.live.min()) == w.B and bool((cache.pos[..., 1:] > cache.pos[..., :-1]).all())
    assert bool((cache.n == L - cache.pos).all())
    u = 17
    Ku, Qu = widen(K[0, u]), widen(Q[0, u])
    for i in (0, 1, 127, 128, 1031, 20000, L - 1):          # rows: lse_i = log-sum-exp over keys 0..i
        _, want = oracle.attention_row(Qu[i], Ku[: i + 1], w.scale)
        assert abs(float(lse[0, u, i]) - want) <= 1e-4
    first = L - 96                                           # columns first..L-1 need rows first..L-1 only
    P = np.zeros((L - first, L))
    for i in range(first, L):
        P[i - first, : i + 1], _ = oracle.attention_row(Qu[i], Ku[: i + 1], w.scale)
    for j in (first, first + 31, L - 2, L - 1):
        col = P[j - first:, j]
        assert_stats_close([float(sf[0, u, j])], [col.sum()], f"s column {j}")
        assert_stats_close([float(qf[0, u, j])], [(col ** 2).sum()], f"q column {j}")
    units = [0, 17, 63]
    st = state_from_cache(cache, units)
    tally = Tally()
    par = DecodeParity(cache, st, units, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, R.ROCO_EVICT_FIRST, tally, scale=w.scale)
    for i in range(4):
        par.step(*W.decode_tokens(w, i, [L + i], DEV), check_state=(i == 3))
    assert tally.decisions == 12 and R.roco_device_status(cache) == 0
