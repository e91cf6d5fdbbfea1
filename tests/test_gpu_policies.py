"""GPU parity of the other Table 1 policies (same decode kernel, different score / scope in the policy warps)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2402_06262_b200 as R
import workloads as W
from harness import DecodeParity, PolicyParity, Tally

pytestmark = pytest.mark.gpu
DEV = "cuda"
POLICIES = [R.ROCO_POLICY_ROCO, R.ROCO_POLICY_RANDOM, R.ROCO_POLICY_RECENCY, R.ROCO_POLICY_STREAMLLM,
            R.ROCO_POLICY_SCISSORHANDS, R.ROCO_POLICY_H2O, R.ROCO_POLICY_TOVA, R.ROCO_POLICY_MAS_WINDOW]


@pytest.mark.parametrize("policy", POLICIES)
@pytest.mark.parametrize("dtype,d,B", [("bf16", 128, 200), ("f32", 64, 96)])
@pytest.mark.parametrize("order", [None, R.ROCO_EVICT_FIRST, R.ROCO_ATTEND_FIRST])
def test_policy_decode_from_empty_cache(policy, dtype, d, B, order):
    """From an empty cache: B fill steps, then 60 steps that each evict under the policy (sink-structured inputs),
    through the entry point with the order of Fig. 1 and through the ordered one in both orders."""
    w = W.scaled(W.LLAMA7B_DECODE, S=2, layers=1, heads=3, d=d, dtype=dtype, B=B, r=B // 4)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    st = oracle.empty_state(w.U, B, d)
    tally = Tally()
    par = PolicyParity(cache, st, range(w.U), policy, w.r, tally, scale=w.scale, order=order)
    g = torch.Generator(device=DEV); g.manual_seed(policy)
    for i in range(B + 60):
        rnd = torch.randint(0, 2 ** 31 - 1, (w.S, w.G), generator=g, device=DEV, dtype=torch.int32)
        par.step(*W.decode_tokens(w, i, [i] * w.S, DEV), rnd=rnd, check_state=(i % 20 == 19) or i == B + 59)
    assert R.roco_device_status(cache) == 0 and tally.decisions == 60 * w.U
    if policy == R.ROCO_POLICY_RECENCY:
        assert int(cache.pos.min()) == 60                      # exactly the last B tokens remain
    if policy == R.ROCO_POLICY_STREAMLLM:
        assert sorted(cache.pos[0, 0].tolist())[:5] == [0, 1, 2, 3, 64]


def test_policy_roco_is_the_plain_decode_step_bitwise():
    w = W.scaled(W.LLAMA7B_DECODE, S=1, layers=1, heads=4, B=64, r=8)
    caches = [R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV) for _ in range(2)]
    out = [torch.zeros(w.S, w.G, w.d, dtype=w.torch_dtype, device=DEV) for _ in range(2)]
    ev = [torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV) for _ in range(2)]
    for i in range(100):
        q, k, v = W.decode_tokens(w, i, [i], DEV)
        R.roco_decode_step(caches[0], q, k, v, w.r, out[0], ev[0], scale=w.scale)
        R.roco_decode_step_policy(caches[1], q, k, v, R.ROCO_POLICY_ROCO, w.r, out[1], ev[1], scale=w.scale)
    torch.cuda.synchronize()
    for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
        assert torch.equal(getattr(caches[0], name), getattr(caches[1], name))
    assert torch.equal(out[0], out[1]) and torch.equal(ev[0], ev[1])


def test_policy_argument_checks():
    w = W.scaled(W.TOY, B=4, r=1)
    cache = R.Cache(w.S, w.G, w.B, w.d, torch.float32, DEV)
    x = torch.zeros(w.S, w.G, w.d, device=DEV)
    ev = torch.zeros(w.S, w.G, dtype=torch.int32, device=DEV)
    for policy, r, code in ((9, 1, 1), (R.ROCO_POLICY_RANDOM, 1, 1), (R.ROCO_POLICY_STREAMLLM, 1, 1),
                            (R.ROCO_POLICY_H2O, 4, 1)):
        with pytest.raises(R.RocoError) as e:
            R.roco_decode_step_policy(cache, x, x, x, policy, r, x.clone(), ev)
        assert e.value.code == code
