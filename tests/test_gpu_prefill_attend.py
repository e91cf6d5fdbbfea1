"""GPU parity of the prompt pass's attention output (roco_prefill_attend, roco_prefill_with_output; tensor cores and
the CUDA-core path) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2402_06262_b200 as R
import workloads as W
from harness import Tally, prefill_parity, unit_view, widen

pytestmark = pytest.mark.gpu
DEV = "cuda"
OUT_TOL = 2e-2   # bf16 output: absolute + relative


def prompt_tensors(w, L):
    qs, ks, vs = zip(*[W.prompt_chunk(w, b, 0, w.G, L, DEV) for b in range(w.S)])
    return torch.stack(qs), torch.stack(ks), torch.stack(vs)


def run_attend(w, lens, Lmax, poison_padding=False):
    Q, K, V = prompt_tensors(w, Lmax)
    if poison_padding:   # rows past a prompt's length may hold anything
        for b, L in enumerate(lens):
            for X in (Q, K, V):
                X[b, :, L:] = float("nan")
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    lse = torch.zeros(w.S, w.G, Lmax, dtype=torch.float32, device=DEV)
    R.roco_prefill(Q, K, V, lens, w.B, w.r, cache, scale=w.scale, lse_out=lse)
    out = torch.full((w.S, w.G, Lmax, w.d), 7.0, dtype=w.torch_dtype, device=DEV)
    R.roco_prefill_attend(cache, Q, K, V, lens, lse, out, scale=w.scale)
    torch.cuda.synchronize()
    assert R.roco_device_status(cache) == 0
    return Q, K, V, lse, out


def check_rows(w, Q, K, V, lse, out, lens, units, rows_of):
    for u in units:
        L = lens[u // w.G]
        q, k, v = (widen(unit_view(X, [u]))[0, :L] for X in (Q, K, V))
        rows = rows_of(L)
        want, want_lse = oracle.prompt_attention_rows(q, k, v, rows, w.scale)
        got = widen(unit_view(out, [u]))[0]
        np.testing.assert_allclose(widen(unit_view(lse, [u]))[0, rows], want_lse, rtol=0, atol=1e-4)
        np.testing.assert_allclose(got[rows], want, rtol=OUT_TOL, atol=OUT_TOL, err_msg=f"unit {u}")
        assert np.all(got[L:] == 7.0), "rows past the prompt must be left untouched"


@pytest.mark.parametrize("kind", ["iid", "sink", "lowrank"])
def test_attend_every_row_ragged(kind):
    """Every row of every unit; lengths of one tile, a ragged multi-tile prompt and a short one (odd and even
    tile counts, so both the paired and the unpaired query tile are exercised)."""
    w = W.scaled(W.LLAMA7B_PREFILL, S=4, layers=1, heads=3, prompt_lo=520, prompt_hi=520, B=64, r=8, kind=kind)
    lens = [520, 333, 128, 7]
    Q, K, V, lse, out = run_attend(w, lens, 520)
    check_rows(w, Q, K, V, lse, out, lens, range(w.U), lambda L: list(range(L)))


def test_attend_ignores_rows_past_the_prompt():
    """NaN in every padding row of Q, K and V changes nothing."""
    w = W.scaled(W.LLAMA7B_PREFILL, S=3, layers=1, heads=2, prompt_lo=400, prompt_hi=400, B=64, r=8, kind="sink")
    lens = [400, 257, 100]
    Q, K, V, lse, out = run_attend(w, lens, 400, poison_padding=True)
    check_rows(w, Q, K, V, lse, out, lens, range(w.U), lambda L: list(range(0, L, 3)) + [L - 1])


def test_attend_long_prompt_sampled_rows():
    """L = 4096 (32 key tiles): sampled rows of sampled units, including both ends of every tile pairing."""
    w = W.scaled(W.LLAMA7B_PREFILL, S=1, layers=1, heads=8, prompt_lo=4096, prompt_hi=4096, B=1024, r=64)
    lens = [4096]
    Q, K, V, lse, out = run_attend(w, lens, 4096)
    rows = [0, 1, 127, 128, 129, 2047, 2048, 3000, 3967, 3968, 4095]
    check_rows(w, Q, K, V, lse, out, lens, [0, 3, 7], lambda L: rows)


@pytest.mark.parametrize("dtype,d", [("f32", 64), ("bf16", 64), ("f32", 128)])
@pytest.mark.parametrize("fused", [False, True])
def test_attend_on_cuda_cores(dtype, d, fused):
    """Dtypes and head dimensions the tensor-core path does not take (the toy configuration is fp32, d = 64): the
    output comes from a CUDA-core pass over the row log-sum-exp, through roco_prefill_attend and through
    roco_prefill_with_output alike.  Every row of every unit, ragged lengths, NaN in the padding rows."""
    w = W.scaled(W.TOY, S=3, heads=2, d=d, dtype=dtype, prompt_lo=200, prompt_hi=200, B=64, r=8)
    lens = [200, 129, 5]
    Q, K, V = prompt_tensors(w, 200)
    for b, L in enumerate(lens):
        for X in (Q, K, V):
            X[b, :, L:] = float("nan")
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    assert not R.roco_prefill_uses_tensor_cores(cache)
    lse = torch.zeros(w.S, w.G, 200, dtype=torch.float32, device=DEV)
    out = torch.full((w.S, w.G, 200, w.d), 7.0, dtype=w.torch_dtype, device=DEV)
    if fused:
        R.roco_prefill(Q, K, V, lens, w.B, w.r, cache, scale=w.scale, lse_out=lse, attn_out=out)
    else:
        R.roco_prefill(Q, K, V, lens, w.B, w.r, cache, scale=w.scale, lse_out=lse)
        R.roco_prefill_attend(cache, Q, K, V, lens, lse, out, scale=w.scale)
    torch.cuda.synchronize()
    assert R.roco_device_status(cache) == 0
    tol = 2e-2 if dtype == "bf16" else 1e-5
    for u in range(w.U):
        L = lens[u // w.G]
        q, k, v = (widen(unit_view(X, [u]))[0, :L] for X in (Q, K, V))
        want, want_lse = oracle.prompt_attention_rows(q, k, v, list(range(L)), w.scale)
        got = widen(unit_view(out, [u]))[0]
        np.testing.assert_allclose(widen(unit_view(lse, [u]))[0, :L], want_lse, rtol=0, atol=1e-4)
        np.testing.assert_allclose(got[:L], want, rtol=tol, atol=tol, err_msg=f"unit {u}")
        assert np.all(got[L:] == 7.0), "rows past the prompt must be left untouched"


# ------------------------------------------------ one sweep: output and row log-sum-exp together (running maximum)

def run_fused(w, lens, Lmax, edit=None, poison_padding=False):
    Q, K, V = prompt_tensors(w, Lmax)
    if edit is not None:
        edit(Q, K, V)
    if poison_padding:
        for b, L in enumerate(lens):
            for X in (Q, K, V):
                X[b, :, L:] = float("nan")
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    lse = torch.zeros(w.S, w.G, Lmax, dtype=torch.float32, device=DEV)
    sf = torch.zeros_like(lse); qf = torch.zeros_like(lse)
    out = torch.full((w.S, w.G, Lmax, w.d), 7.0, dtype=w.torch_dtype, device=DEV)
    R.roco_prefill(Q, K, V, lens, w.B, w.r, cache, scale=w.scale, lse_out=lse, s_full=sf, q_full=qf, attn_out=out)
    torch.cuda.synchronize()
    assert R.roco_device_status(cache) == 0
    return Q, K, V, lse, out, cache, sf, qf


def plain_prefill(w, Q, K, V, lens, Lmax):
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    lse = torch.zeros(w.S, w.G, Lmax, dtype=torch.float32, device=DEV)
    sf = torch.zeros_like(lse); qf = torch.zeros_like(lse)
    R.roco_prefill(Q, K, V, lens, w.B, w.r, cache, scale=w.scale, lse_out=lse, s_full=sf, q_full=qf)
    torch.cuda.synchronize()
    return cache, lse, sf, qf


@pytest.mark.parametrize("kind", ["iid", "sink", "lowrank"])
def test_fused_prompt_pass_every_row_ragged(kind):
    """roco_prefill with attn_out: output and log-sum-exp of every row against the oracle, and the statistics and
    the budgeted cache against the call without the output (which the other tests hold against the oracle)."""
    w = W.scaled(W.LLAMA7B_PREFILL, S=4, layers=1, heads=3, prompt_lo=520, prompt_hi=520, B=64, r=8, kind=kind)
    lens = [520, 333, 128, 7]
    Q, K, V, lse, out, cache, sf, qf = run_fused(w, lens, 520, poison_padding=True)
    check_rows(w, Q, K, V, lse, out, lens, range(w.U), lambda L: list(range(L)))
    ref, lse0, sf0, qf0 = plain_prefill(w, Q, K, V, lens, 520)
    for b, L in enumerate(lens):
        np.testing.assert_allclose(lse[b, :, :L].cpu().numpy(), lse0[b, :, :L].cpu().numpy(), rtol=0, atol=2e-5)
        np.testing.assert_allclose(sf[b, :, :L].cpu().numpy(), sf0[b, :, :L].cpu().numpy(), rtol=1e-4)
        np.testing.assert_allclose(qf[b, :, :L].cpu().numpy(), qf0[b, :, :L].cpu().numpy(), rtol=1e-4)
    assert torch.equal(cache.live, ref.live) and torch.equal(cache.n, ref.n)
    assert (cache.pos != ref.pos).float().mean().item() <= 0.01      # survivors equal up to decisions inside the margin


def test_fused_prompt_pass_moves_the_row_maximum():
    """Keys planted late in the prompt that beat every earlier score by far: the reference maximum of all later
    rows has to move (several times, in different 32-column chunks of a tile), which rescales the output
    accumulator, the running sum and the part of the current P tile already written."""
    w = W.scaled(W.LLAMA7B_PREFILL, S=1, layers=1, heads=4, prompt_lo=900, prompt_hi=900, B=128, r=8, kind="iid")
    # position -> strength: logits of about 3 x strength, each ~48 nats (69 powers of two) above the one before,
    # past the 2^60 at which a row moves its reference; chunks 3, 1, 0, 2 of their key tiles
    planted = {230: 16.0, 417: 32.0, 640: 48.0, 705: 64.0}

    def edit(Q, K, V):
        g = torch.Generator(device=DEV); g.manual_seed(7)
        u = torch.randn(w.S, w.G, 1, w.d, device=DEV, generator=g)
        u = u / u.norm(dim=-1, keepdim=True)
        Q += (3.0 * u).to(Q.dtype)                               # every query has a component along u
        for pos, strength in planted.items():
            K[:, :, pos] = (strength * w.d ** 0.5 * u[:, :, 0]).to(K.dtype)
            V[:, :, pos] = float(pos) / 100.0

    Q, K, V, lse, out, cache, _, _ = run_fused(w, [900], 900, edit=edit)
    check_rows(w, Q, K, V, lse, out, [900], range(w.U), lambda L: list(range(L)))
    # the planted keys dominate: rows after the last one return (nearly) its value, so the rescaling was exercised
    assert abs(float(out[0, 0, 899, 0]) - 7.05) < 0.1


def test_fused_prompt_pass_long_prompt_sampled_rows():
    w = W.scaled(W.LLAMA7B_PREFILL, S=1, layers=1, heads=8, prompt_lo=4096, prompt_hi=4096, B=1024, r=64)
    Q, K, V, lse, out, cache, _, _ = run_fused(w, [4096], 4096)
    rows = [0, 1, 127, 128, 129, 2047, 2048, 3000, 3967, 3968, 4095]
    check_rows(w, Q, K, V, lse, out, [4096], [0, 3, 7], lambda L: rows)


@pytest.mark.parametrize("scale", [0.0, -0.06])
def test_prompt_pass_with_a_scale_that_is_not_positive(scale):
    """The tensor-core sweeps need a positive scale; zero and negative ones take the CUDA-core path and must still
    give Eq. 1: log-sum-exp and output of every row, statistics and survivors against the oracle."""
    w = W.scaled(W.LLAMA7B_PREFILL, S=1, layers=1, heads=2, prompt_lo=300, prompt_hi=300, B=128, r=16)
    Q, K, V = prompt_tensors(w, 300)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    lse = torch.zeros(w.S, w.G, 300, dtype=torch.float32, device=DEV)
    out = torch.full((w.S, w.G, 300, w.d), 7.0, dtype=w.torch_dtype, device=DEV)
    R.roco_prefill(Q, K, V, [300], w.B, w.r, cache, scale=scale, lse_out=lse, attn_out=out)
    torch.cuda.synchronize()
    assert R.roco_device_status(cache) == 0
    for u in range(w.U):
        q, k, v = (widen(unit_view(X, [u]))[0] for X in (Q, K, V))
        want, want_lse = oracle.prompt_attention_rows(q, k, v, list(range(300)), scale)
        np.testing.assert_allclose(widen(unit_view(lse, [u]))[0], want_lse, rtol=0, atol=1e-4)
        np.testing.assert_allclose(widen(unit_view(out, [u]))[0], want, rtol=OUT_TOL, atol=OUT_TOL)
    tally = Tally()
    prefill_parity(R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV), Q, K, V, [300], w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R,
                   range(w.U), tally, scale=scale)
    # the second, separate call for the output takes the same path
    out2 = torch.full_like(out, 7.0)
    R.roco_prefill_attend(cache, Q, K, V, [300], lse, out2, scale=scale)
    torch.cuda.synchronize()
    assert torch.equal(out, out2)


def test_fused_prompt_pass_argument_checks():
    w = W.scaled(W.LLAMA7B_PREFILL, S=1, layers=1, heads=1, prompt_lo=128, prompt_hi=128, B=64, r=8)
    Q, K, V = prompt_tensors(w, 128)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    misaligned = torch.zeros(Q.numel() + 8, dtype=Q.dtype, device=DEV)[1:1 + Q.numel()].view_as(Q)
    with pytest.raises(R.RocoError) as e:                        # the output must be 16-byte aligned
        R.roco_prefill(Q, K, V, [128], w.B, w.r, cache, attn_out=misaligned)
    assert e.value.code == 1
