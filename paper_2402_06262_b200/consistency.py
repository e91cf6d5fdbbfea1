"""Consistency of an importance score under a budget with its full-cache version (the preliminary experiment of
Sec. 4.3, on synthetic inputs): Jaccard similarity between the tokens a budgeted cache retains (window size r = 0,
so the policy keeps the top-B tokens by its own score) and the top-B tokens by the same score computed with a full
cache, averaged over decode steps and units.

Everything on the path runs in the library's kernels (roco_prefill, roco_decode_step_policy); torch only ranks the
full-cache scores and intersects the position sets, which is analysis, not part of the method.
"""
from __future__ import annotations

from typing import Dict

import torch

import workloads as W

from . import binding as R

SCORED = {"MAS": R.ROCO_POLICY_MAS_WINDOW, "AAS": R.ROCO_POLICY_H2O, "AQAS": R.ROCO_POLICY_SCISSORHANDS,
          "LTAS": R.ROCO_POLICY_TOVA}


def _score(cache: R.Cache, policy: int) -> torch.Tensor:
    live = torch.arange(cache.B, device=cache.s.device)[None, None, :] < cache.live[..., None]
    if policy == R.ROCO_POLICY_H2O:
        sc = cache.s
    elif policy in (R.ROCO_POLICY_SCISSORHANDS, R.ROCO_POLICY_TOVA):
        sc = cache.q
    else:
        sc = cache.s / cache.n.clamp(min=1)
    return torch.where(live, sc, torch.full_like(sc, -1.0))


def jaccard_consistency(w: W.Workload, score: str, budget: int, steps: int, device="cuda") -> float:
    """Mean Jaccard similarity for importance score `score` in {"MAS", "AAS", "AQAS", "LTAS"}: the sequence of
    w.prompt_lo prompt tokens and `steps` decode tokens is fed one token at a time through a budgeted cache
    (budget tokens, r = 0) and through a cache large enough never to evict."""
    policy = SCORED[score]
    total = w.prompt_lo + steps
    full = R.Cache(w.S, w.G, total, w.d, w.torch_dtype, device)
    small = R.Cache(w.S, w.G, budget, w.d, w.torch_dtype, device)
    out = torch.zeros(w.S, w.G, w.d, dtype=w.torch_dtype, device=device)
    ev = torch.zeros(w.S, w.G, dtype=torch.int32, device=device)
    prompt = [W.prompt_chunk(w, b, 0, w.G, w.prompt_lo, device) for b in range(w.S)]
    Qp, Kp, Vp = (torch.stack([p[i] for p in prompt]) for i in range(3))          # [S][G][L][d]
    acc, cnt = 0.0, 0
    for t in range(total):
        if t < w.prompt_lo:
            q, k, v = (x[:, :, t].contiguous() for x in (Qp, Kp, Vp))
        else:
            q, k, v = W.decode_tokens(w, t - w.prompt_lo, [t] * w.S, device)
        for c in (full, small):
            R.roco_decode_step_policy(c, q, k, v, policy, 0, out, ev, scale=w.scale)
        if t >= budget:                                        # the budgeted cache has started to evict
            top = _score(full, policy).topk(budget, dim=-1).indices              # slots of the full cache
            top_pos = torch.gather(full.pos, 2, top.to(torch.int64))             # their positions
            kept = small.pos                                                     # [S][G][budget]
            inter = (kept[..., :, None] == top_pos[..., None, :]).any(-1).sum(-1).float()
            acc += float((inter / (2 * budget - inter)).mean())
            cnt += 1
    if R.roco_device_status(full) or R.roco_device_status(small):
        raise RuntimeError("device status word set")
    return acc / max(cnt, 1)


def consistency_table(w: W.Workload, rates=(0.3, 0.4, 0.5, 0.6), steps: int = 64, device="cuda") -> Dict[str, Dict[float, float]]:
    """Jaccard consistency of every attention-based score at several budget rates (budget = rate x sequence)."""
    total = w.prompt_lo + steps
    return {name: {rate: jaccard_consistency(w, name, max(8, int(rate * total)), steps, device) for rate in rates}
            for name in SCORED}
