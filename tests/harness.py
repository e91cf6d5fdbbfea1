"""Parity harness: runs the CUDA library and the fp64 oracle on the same bytes and compares them.

Tolerances (fixed by the parity contract): eviction/slot indices bit-exact wherever the oracle's decision
margin exceeds 1e-5 relative (steps inside the margin are counted and the oracle continues from the GPU's
choice, so that one excluded step cannot poison the rest of a run); s and q within 1e-4 relative; n, pos,
live, t_next exact; attention output within 2e-2 max-abs for bf16 and 1e-5 for fp32; lse within 1e-4.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence

import numpy as np
import torch

import oracle
import paper_2402_06262_b200 as R
from workloads import unit_view, widen

DELTA = 1e-5
STAT_RTOL = 1e-4
LSE_ATOL = 1e-4


def out_tol(dtype) -> float:
    return 2e-2 if dtype == torch.bfloat16 else 1e-5


def assert_stats_close(got, want, what):
    got = np.asarray(got, np.float64)
    np.testing.assert_allclose(got, want, rtol=STAT_RTOL, atol=1e-30, err_msg=what)


@dataclasses.dataclass
class Tally:
    steps: int = 0
    decisions: int = 0
    near_ties: int = 0
    near_tie_disagreements: int = 0
    prefill_uncertain: int = 0
    prefill_swapped: int = 0
    prefill_units_evicting: int = 0     # units whose prompt exceeded the budget
    prefill_units_firm: int = 0         # ... of which the survivor set equalled the oracle's own, token for token


def state_from_cache(cache: R.Cache, units: Sequence[int]) -> oracle.State:
    """An oracle state that continues from the device cache of the given units (exact widening)."""
    return oracle.State(widen(unit_view(cache.K, units)), widen(unit_view(cache.V, units)),
                        widen(unit_view(cache.s, units)), widen(unit_view(cache.q, units)),
                        unit_view(cache.n, units).cpu().numpy().copy(), unit_view(cache.pos, units).cpu().numpy().copy(),
                        unit_view(cache.live, units).cpu().numpy().copy(),
                        unit_view(cache.t_next, units).cpu().numpy().copy())


def compare_state(cache: R.Cache, st: oracle.State, units: Sequence[int], what: str, check_kv=True):
    live = unit_view(cache.live, units).cpu().numpy()
    np.testing.assert_array_equal(live, st.live, err_msg=f"{what}: live")
    np.testing.assert_array_equal(unit_view(cache.t_next, units).cpu().numpy(), st.t_next, err_msg=f"{what}: t_next")
    pos = unit_view(cache.pos, units).cpu().numpy()
    n = unit_view(cache.n, units).cpu().numpy()
    s = widen(unit_view(cache.s, units))
    q = widen(unit_view(cache.q, units))
    K = widen(unit_view(cache.K, units)) if check_kv else None
    V = widen(unit_view(cache.V, units)) if check_kv else None
    for i in range(len(units)):
        lv = int(live[i])
        np.testing.assert_array_equal(pos[i, :lv], st.pos[i, :lv], err_msg=f"{what}: pos unit {units[i]}")
        np.testing.assert_array_equal(n[i, :lv], st.n[i, :lv], err_msg=f"{what}: n unit {units[i]}")
        assert_stats_close(s[i, :lv], st.s[i, :lv], f"{what}: s unit {units[i]}")
        assert_stats_close(q[i, :lv], st.q[i, :lv], f"{what}: q unit {units[i]}")
        if check_kv:
            np.testing.assert_array_equal(K[i, :lv], st.K[i, :lv], err_msg=f"{what}: K unit {units[i]}")
            np.testing.assert_array_equal(V[i, :lv], st.V[i, :lv], err_msg=f"{what}: V unit {units[i]}")


def prefill_parity(cache: R.Cache, Q, K, V, lens: Sequence[int], r: int, scope_mode: int, units: Sequence[int],
                   tally: Tally, scale: Optional[float] = None, static: bool = False) -> oracle.State:
    """Runs roco_prefill on the device tensors Q,K,V [S][G][Lmax][d], the oracle on the sampled units, compares,
    and returns the oracle state (continued from the GPU's survivor set where that differs inside the margin)."""
    S, G, Lmax, d = Q.shape
    B = cache.B
    scale = d ** -0.5 if scale is None else scale
    dev = Q.device
    lse = torch.zeros(S, G, Lmax, dtype=torch.float32, device=dev)
    sf = torch.zeros_like(lse)
    qf = torch.zeros_like(lse)
    (R.roco_prefill_static if static else R.roco_prefill)(Q, K, V, lens, B, r, cache, scope_mode=scope_mode, scale=scale,
                                                          lse_out=lse, s_full=sf, q_full=qf)
    torch.cuda.synchronize()
    assert R.roco_device_status(cache) == 0
    ulens = [int(lens[u // G]) for u in units]
    res = oracle.prefill(widen(unit_view(Q, units)), widen(unit_view(K, units)), widen(unit_view(V, units)), ulens,
                         B, r, scope_mode, scale, delta=DELTA)
    g_lse, g_s, g_q = widen(unit_view(lse, units)), widen(unit_view(sf, units)), widen(unit_view(qf, units))
    g_pos = unit_view(cache.pos, units).cpu().numpy()
    g_live = unit_view(cache.live, units).cpu().numpy()
    force = None
    for i, L in enumerate(ulens):
        np.testing.assert_allclose(g_lse[i, :L], res.lse[i, :L], rtol=0, atol=LSE_ATOL, err_msg=f"lse unit {units[i]}")
        assert_stats_close(g_s[i, :L], res.s_full[i, :L], f"s_full unit {units[i]}")
        assert_stats_close(g_q[i, :L], res.q_full[i, :L], f"q_full unit {units[i]}")
        assert g_live[i] == min(L, B)
        kept = g_pos[i, : g_live[i]]
        assert np.all(np.diff(kept) > 0), "survivors must sit in increasing position order"
        gkeep = np.zeros(Lmax, bool)
        gkeep[kept] = True
        diff = gkeep[:L] != res.keep[i, :L]
        tally.prefill_units_evicting += int(L > B)
        tally.prefill_units_firm += int(L > B and not diff.any())
        if diff.any() and scope_mode == R.ROCO_SCOPE_LOWEST_R:
            # iterated form: replay the evictions next to the GPU's set; it may be followed only at iterations
            # inside the margin, and only to a token that could be the victim there
            followed, keep = oracle.select_to_budget_guided(res.s_full[i, :L], res.q_full[i, :L], res.n_full[i, :L],
                                                            B, r, scope_mode, gkeep[:L], delta=DELTA)
            assert followed >= 0, (f"unit {units[i]}: eviction {-followed - 1} of the replay differs outside the "
                                   f"{DELTA} margin")
            assert np.array_equal(keep, gkeep[:L])
            tally.prefill_swapped += followed
        elif diff.any():
            tally.prefill_uncertain += int(res.uncertain[i].sum())
            assert np.all(res.uncertain[i, :L][diff]), \
                f"unit {units[i]}: survivor sets differ outside the {DELTA} margin at {np.nonzero(diff)[0]}"
            tally.prefill_swapped += int(diff.sum())
        if diff.any():
            if force is None:
                force = res.keep.copy()
            force[i] = gkeep
    if force is not None:   # continue from the GPU's (in-margin) survivor set
        res = oracle.prefill(widen(unit_view(Q, units)), widen(unit_view(K, units)), widen(unit_view(V, units)),
                             ulens, B, r, scope_mode, scale, delta=DELTA, force_keep=force)
    compare_state(cache, res.state, units, "after prefill")
    return res.state


class DecodeParity:
    """Steps the GPU cache and the oracle state of the sampled units together."""

    def __init__(self, cache: R.Cache, st: oracle.State, units: Sequence[int], r: int, scope_mode: int, order: int,
                 tally: Tally, scale: Optional[float] = None, strict: bool = False, splits: int = 0,
                 ranks: int = 0):
        self.splits = splits
        self.ranks = ranks      # 0: roco_decode_step picks the launch shape; 1: one CTA per unit; > 1: that cluster
        self.ws = (torch.empty(R.roco_decode_split_workspace_bytes(cache, splits), dtype=torch.uint8,
                               device=cache.K.device) if splits else None)
        self.cache, self.st, self.units = cache, st, list(units)
        self.r, self.mode, self.order, self.tally, self.strict = r, scope_mode, order, tally, strict
        self.scale = cache.d ** -0.5 if scale is None else scale
        dev = cache.K.device
        self.out = torch.zeros(cache.S, cache.G, cache.d, dtype=cache.dtype, device=dev)
        self.lse = torch.zeros(cache.S, cache.G, dtype=torch.float32, device=dev)
        self.ev_slot = torch.zeros(cache.S, cache.G, dtype=torch.int32, device=dev)
        self.ev_pos = torch.zeros(cache.S, cache.G, dtype=torch.int32, device=dev)

    def step(self, q, k_new, v_new, check_state: bool = False):
        c = self.cache
        if self.ranks >= 1:
            R.roco_decode_step_cluster(c, q, k_new, v_new, self.r, self.out, self.ev_slot, self.ev_pos, self.lse,
                                       scope_mode=self.mode, step_order=self.order, ranks=self.ranks, scale=self.scale)
        elif self.splits:
            R.roco_decode_step_split(c, q, k_new, v_new, self.r, self.splits, self.out, self.ev_slot, self.ws,
                                     self.ev_pos, self.lse, scope_mode=self.mode, scale=self.scale,
                                     step_order=(None if self.order == R.ROCO_EVICT_FIRST else self.order))
        else:
            R.roco_decode_step(c, q, k_new, v_new, self.r, self.out, self.ev_slot, self.ev_pos, self.lse,
                               scope_mode=self.mode, step_order=self.order, scale=self.scale)
        torch.cuda.synchronize()
        g_slot = unit_view(self.ev_slot, self.units).cpu().numpy()
        g_pos = unit_view(self.ev_pos, self.units).cpu().numpy()
        res = oracle.decode_step(self.st, widen(unit_view(q, self.units)), widen(unit_view(k_new, self.units)),
                                 widen(unit_view(v_new, self.units)), self.r, self.mode, self.order, self.scale,
                                 delta=DELTA, force_victim=g_slot, force_only_near=not self.strict)
        if self.strict:   # exact ties resolved by position are under test: no exclusions at all
            np.testing.assert_array_equal(g_slot, res.choice)
        else:
            firm = ~res.near_tie
            np.testing.assert_array_equal(g_slot[firm], res.choice[firm],
                                          err_msg="victim differs outside the decision margin")
            self.tally.near_ties += int(res.near_tie.sum())
            self.tally.near_tie_disagreements += int((g_slot != res.choice)[res.near_tie].sum())
        np.testing.assert_array_equal(g_slot, res.evicted_slot)
        np.testing.assert_array_equal(g_pos, res.evicted_pos)
        self.tally.steps += 1
        self.tally.decisions += int((res.choice >= 0).sum())
        g_out = widen(unit_view(self.out, self.units))
        assert np.abs(g_out - res.out).max() <= out_tol(c.dtype), f"attention output off by {np.abs(g_out - res.out).max()}"
        g_lse = widen(unit_view(self.lse, self.units))
        fin = np.isfinite(res.lse)
        np.testing.assert_allclose(g_lse[fin], res.lse[fin], rtol=0, atol=LSE_ATOL)
        assert np.all(np.isneginf(g_lse[~fin]))
        if check_state:
            compare_state(c, self.st, self.units, f"after step {self.tally.steps}", check_kv=True)
        return res


class BlockParity:
    """Steps the GPU cache and the oracle state of the sampled units together, b tokens per step."""

    def __init__(self, cache: R.Cache, st: oracle.State, units: Sequence[int], b: int, r: int, scope_mode: int,
                 tally: Tally, scale: Optional[float] = None):
        self.cache, self.st, self.units, self.b = cache, st, list(units), b
        self.r, self.mode, self.tally = r, scope_mode, tally
        self.scale = cache.d ** -0.5 if scale is None else scale
        dev = cache.K.device
        self.out = torch.zeros(cache.S, cache.G, b, cache.d, dtype=cache.dtype, device=dev)
        self.lse = torch.zeros(cache.S, cache.G, b, dtype=torch.float32, device=dev)
        self.ev_slot = torch.zeros(cache.S, cache.G, b, dtype=torch.int32, device=dev)
        self.ev_pos = torch.zeros(cache.S, cache.G, b, dtype=torch.int32, device=dev)

    def step(self, Q, K_new, V_new, check_state=False):
        c = self.cache
        R.roco_block_step(c, Q, K_new, V_new, self.r, self.out, self.ev_slot, self.ev_pos, self.lse,
                          scope_mode=self.mode, scale=self.scale)
        torch.cuda.synchronize()
        g_slot = unit_view(self.ev_slot, self.units).cpu().numpy()
        g_pos = unit_view(self.ev_pos, self.units).cpu().numpy()
        res = oracle.block_step(self.st, widen(unit_view(Q, self.units)), widen(unit_view(K_new, self.units)),
                                widen(unit_view(V_new, self.units)), self.r, self.mode, self.scale, delta=DELTA,
                                force_slots=g_slot)
        firm = res.near_tie == 0
        np.testing.assert_array_equal(g_slot[firm], res.choice[firm], err_msg="freed slots differ outside the margin")
        self.tally.near_ties += int((~firm).sum())
        self.tally.near_tie_disagreements += int((g_slot != res.choice).any(axis=1)[~firm].sum())
        np.testing.assert_array_equal(g_slot, res.evicted_slot)
        np.testing.assert_array_equal(g_pos, res.evicted_pos)
        self.tally.steps += 1
        self.tally.decisions += int((res.choice >= 0).sum())
        g_out = widen(unit_view(self.out, self.units))
        assert np.abs(g_out - res.out).max() <= out_tol(c.dtype), f"attention output off by {np.abs(g_out - res.out).max()}"
        np.testing.assert_allclose(widen(unit_view(self.lse, self.units)), res.lse, rtol=0, atol=LSE_ATOL)
        if check_state:
            compare_state(c, self.st, self.units, f"after block step {self.tally.steps}")
        return res


class GqaBlockParity:
    """Steps key-value-head caches shared by `group` query heads, b tokens per step, on the GPU and in the oracle."""

    def __init__(self, cache: R.Cache, st: oracle.State, units: Sequence[int], b: int, group: int, r: int, tally: Tally,
                 scale: Optional[float] = None):
        self.cache, self.st, self.units, self.b, self.group, self.r, self.tally = cache, st, list(units), b, group, r, tally
        self.scale = cache.d ** -0.5 if scale is None else scale
        dev = cache.K.device
        self.out = torch.zeros(cache.S, cache.G, b, group, cache.d, dtype=cache.dtype, device=dev)
        self.lse = torch.zeros(cache.S, cache.G, b, group, dtype=torch.float32, device=dev)
        self.ev_slot = torch.zeros(cache.S, cache.G, b, dtype=torch.int32, device=dev)
        self.ev_pos = torch.zeros(cache.S, cache.G, b, dtype=torch.int32, device=dev)

    def step(self, Q, K_new, V_new, check_state=False):
        c = self.cache
        R.roco_gqa_block_step(c, Q, K_new, V_new, self.r, self.out, self.ev_slot, self.ev_pos, self.lse, scale=self.scale)
        torch.cuda.synchronize()
        g_slot = unit_view(self.ev_slot, self.units).cpu().numpy()
        g_pos = unit_view(self.ev_pos, self.units).cpu().numpy()
        res = oracle.gqa_block_step(self.st, widen(unit_view(Q, self.units)), widen(unit_view(K_new, self.units)),
                                    widen(unit_view(V_new, self.units)), self.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, self.scale,
                                    delta=DELTA, force_slots=g_slot)
        firm = res.near_tie == 0
        np.testing.assert_array_equal(g_slot[firm], res.choice[firm], err_msg="freed slots differ outside the margin")
        self.tally.near_ties += int((~firm).sum())
        np.testing.assert_array_equal(g_slot, res.evicted_slot)
        np.testing.assert_array_equal(g_pos, res.evicted_pos)
        self.tally.steps += 1
        self.tally.decisions += int((res.choice >= 0).sum())
        g_out = widen(unit_view(self.out, self.units))
        assert np.abs(g_out - res.out).max() <= out_tol(c.dtype), f"attention output off by {np.abs(g_out - res.out).max()}"
        np.testing.assert_allclose(widen(unit_view(self.lse, self.units)), res.lse, rtol=0, atol=LSE_ATOL)
        if check_state:
            compare_state(c, self.st, self.units, f"after grouped block step {self.tally.steps}")
        return res


class GqaParity:
    """Steps key-value-head caches shared by `group` query heads on the GPU and in the oracle."""

    def __init__(self, cache: R.Cache, st: oracle.State, units: Sequence[int], group: int, r: int, scope_mode: int,
                 tally: Tally, scale: Optional[float] = None):
        self.cache, self.st, self.units, self.group = cache, st, list(units), group
        self.r, self.mode, self.tally = r, scope_mode, tally
        self.scale = cache.d ** -0.5 if scale is None else scale
        dev = cache.K.device
        self.out = torch.zeros(cache.S, cache.G, group, cache.d, dtype=cache.dtype, device=dev)
        self.lse = torch.zeros(cache.S, cache.G, group, dtype=torch.float32, device=dev)
        self.ev_slot = torch.zeros(cache.S, cache.G, dtype=torch.int32, device=dev)
        self.ev_pos = torch.zeros(cache.S, cache.G, dtype=torch.int32, device=dev)

    def step(self, Q, k_new, v_new, check_state=False):
        c = self.cache
        R.roco_gqa_decode_step(c, Q, k_new, v_new, self.r, self.out, self.ev_slot, self.ev_pos, self.lse,
                               scope_mode=self.mode, scale=self.scale)
        torch.cuda.synchronize()
        g_slot = unit_view(self.ev_slot, self.units).cpu().numpy()
        g_pos = unit_view(self.ev_pos, self.units).cpu().numpy()
        res = oracle.gqa_step(self.st, widen(unit_view(Q, self.units)), widen(unit_view(k_new, self.units)),
                              widen(unit_view(v_new, self.units)), self.r, self.mode, self.scale, delta=DELTA,
                              force_victim=g_slot)
        firm = ~res.near_tie
        np.testing.assert_array_equal(g_slot[firm], res.choice[firm], err_msg="victim differs outside the margin")
        self.tally.near_ties += int(res.near_tie.sum())
        np.testing.assert_array_equal(g_slot, res.evicted_slot)
        np.testing.assert_array_equal(g_pos, res.evicted_pos)
        self.tally.steps += 1
        self.tally.decisions += int((res.choice >= 0).sum())
        g_out = widen(unit_view(self.out, self.units))
        assert np.abs(g_out - res.out).max() <= out_tol(c.dtype), f"attention output off by {np.abs(g_out - res.out).max()}"
        np.testing.assert_allclose(widen(unit_view(self.lse, self.units)), res.lse, rtol=0, atol=LSE_ATOL)
        if check_state:
            compare_state(c, self.st, self.units, f"after gqa step {self.tally.steps}")
        return res


class PolicyParity:
    """Steps the GPU cache and the oracle state together under one of the Table 1 policies."""

    def __init__(self, cache: R.Cache, st: oracle.State, units: Sequence[int], policy: int, r: int, tally: Tally,
                 scale: Optional[float] = None, order: Optional[int] = None):
        self.cache, self.st, self.units, self.policy, self.r, self.tally = cache, st, list(units), policy, r, tally
        self.order = order      # None: roco_decode_step_policy (evict, insert, attend); else the ordered entry point
        self.scale = cache.d ** -0.5 if scale is None else scale
        dev = cache.K.device
        self.out = torch.zeros(cache.S, cache.G, cache.d, dtype=cache.dtype, device=dev)
        self.lse = torch.zeros(cache.S, cache.G, dtype=torch.float32, device=dev)
        self.ev_slot = torch.zeros(cache.S, cache.G, dtype=torch.int32, device=dev)
        self.ev_pos = torch.zeros(cache.S, cache.G, dtype=torch.int32, device=dev)
        self.quant_fixups = 0

    def step(self, q, k_new, v_new, rnd=None, check_state=False):
        c = self.cache
        R.roco_decode_step_policy(c, q, k_new, v_new, self.policy, self.r, self.out, self.ev_slot, self.ev_pos,
                                  self.lse, rnd=rnd, scale=self.scale, step_order=self.order)
        torch.cuda.synchronize()
        g_slot = unit_view(self.ev_slot, self.units).cpu().numpy()
        g_pos = unit_view(self.ev_pos, self.units).cpu().numpy()
        rn = None if rnd is None else unit_view(rnd, self.units).cpu().numpy().astype(np.uint32)
        res, qn = oracle.policy_step(self.st, widen(unit_view(q, self.units)), widen(unit_view(k_new, self.units)),
                                     widen(unit_view(v_new, self.units)), self.policy, self.r, self.scale, rnd=rn,
                                     delta=DELTA, force_victim=g_slot,
                                     order=R.ROCO_EVICT_FIRST if self.order is None else self.order)
        firm = ~res.near_tie
        np.testing.assert_array_equal(g_slot[firm], res.choice[firm], err_msg="victim differs outside the margin")
        self.tally.near_ties += int(res.near_tie.sum())
        np.testing.assert_array_equal(g_slot, res.evicted_slot)
        np.testing.assert_array_equal(g_pos, res.evicted_pos)
        self.tally.steps += 1
        self.tally.decisions += int((res.choice >= 0).sum())
        if qn.any():   # a quantisation on the edge of "above average": continue from the GPU's count there
            gq = widen(unit_view(c.q, self.units))
            self.st.q[qn] = gq[qn]
            self.quant_fixups += int(qn.sum())
        g_out = widen(unit_view(self.out, self.units))
        assert np.abs(g_out - res.out).max() <= out_tol(c.dtype)
        g_lse = widen(unit_view(self.lse, self.units))
        fin = np.isfinite(res.lse)      # ATTEND_FIRST on an empty cache attends over nothing
        np.testing.assert_allclose(g_lse[fin], res.lse[fin], rtol=0, atol=LSE_ATOL)
        assert np.all(np.isneginf(g_lse[~fin]))
        if check_state:
            compare_state(c, self.st, self.units, f"after policy step {self.tally.steps}")
        return res
