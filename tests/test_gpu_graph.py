"""The step entry points only enqueue work on the caller's stream, so a decode loop can be captured in a CUDA graph
and replayed: the replay must leave exactly what the same calls leave when issued one by one."""
import pytest
import torch

import paper_2402_06262_b200 as R
import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"
FIELDS = ("K", "V", "s", "q", "n", "pos", "live", "t_next")


def prefilled_copies(w, L, copies):
    Q, K, V = (torch.stack(x) for x in zip(*[W.prompt_chunk(w, b, 0, w.G, L, DEV) for b in range(w.S)]))
    first = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    R.roco_prefill(Q, K, V, [L] * w.S, w.B, w.r, first, scale=w.scale)
    out = [first]
    for _ in range(copies - 1):
        c = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
        for f in FIELDS:
            getattr(c, f).copy_(getattr(first, f))
        out.append(c)
    return out


def same_cache(a, b):
    return all(torch.equal(getattr(a, f), getattr(b, f)) for f in FIELDS)


@pytest.mark.parametrize("heads,B", [(8, 256), (2, 2048)])   # one CTA per unit; a cluster of CTAs per unit
def test_decode_loop_in_a_graph(heads, B):
    w = W.scaled(W.LLAMA7B_DECODE, S=2, layers=1, heads=heads, prompt_lo=B + 60, prompt_hi=B + 60, B=B, r=16)
    L, steps = B + 60, 6
    eager, graphed, warm = prefilled_copies(w, L, 3)
    toks = [W.decode_tokens(w, i, [L + i] * w.S, DEV) for i in range(steps)]
    outs = torch.zeros(2, steps, w.S, w.G, w.d, dtype=w.torch_dtype, device=DEV)
    evs = torch.zeros(2, steps, w.S, w.G, dtype=torch.int32, device=DEV)
    for i, (q, k, v) in enumerate(toks):
        R.roco_decode_step(eager, q, k, v, w.r, outs[0, i], evs[0, i], scale=w.scale)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):   # first use of the kernels outside the capture
        R.roco_decode_step(warm, *toks[0], w.r, torch.zeros_like(outs[0, 0]), torch.zeros_like(evs[0, 0]), scale=w.scale)
    torch.cuda.current_stream().wait_stream(side)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i, (q, k, v) in enumerate(toks):
            R.roco_decode_step(graphed, q, k, v, w.r, outs[1, i], evs[1, i], scale=w.scale)
    assert not same_cache(eager, graphed)      # capturing has not run anything
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(evs[0], evs[1]) and torch.equal(outs[0], outs[1]) and same_cache(eager, graphed)
    assert R.roco_device_status(eager) == 0 and R.roco_device_status(graphed) == 0
    assert int(evs[0].min()) >= 0                # every step evicted


def test_block_steps_in_a_graph():
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=6, prompt_lo=1100, prompt_hi=1100)
    L, b, steps = 1100, 16, 3
    eager, graphed, warm = prefilled_copies(w, L, 3)
    gen = torch.Generator(device=DEV); gen.manual_seed(5)
    toks = [tuple(torch.randn(w.S, w.G, b, w.d, device=DEV, generator=gen).to(w.torch_dtype) for _ in range(3))
            for _ in range(steps)]
    outs = torch.zeros(2, steps, w.S, w.G, b, w.d, dtype=w.torch_dtype, device=DEV)
    evs = torch.zeros(2, steps, w.S, w.G, b, dtype=torch.int32, device=DEV)
    for i, (q, k, v) in enumerate(toks):
        R.roco_block_step(eager, q, k, v, w.r, outs[0, i], evs[0, i], scale=w.scale)
    R.roco_block_step(warm, *toks[0], w.r, torch.zeros_like(outs[0, 0]), torch.zeros_like(evs[0, 0]), scale=w.scale)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i, (q, k, v) in enumerate(toks):
            R.roco_block_step(graphed, q, k, v, w.r, outs[1, i], evs[1, i], scale=w.scale)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(evs[0], evs[1]) and torch.equal(outs[0], outs[1]) and same_cache(eager, graphed)
    assert R.roco_device_status(graphed) == 0
