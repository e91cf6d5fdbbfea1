#!/usr/bin/env python
"""Benchmark of the RoCo decode hot path on B200 (one JSON line on stdout).

A *step* is one decode step of every (sequence, layer, head) unit of the Llama-2-7B-shape workload:
attention over the budgeted cache, statistics update, scope/victim selection and in-place overwrite, all
in one kernel launch per step.  The cache is first built by the library's own prefill (2048-token prompts
evicted to B = 1024).  `value` is decode tokens/s of the attention path (one step yields S tokens and needs
all layers*heads units of each sequence).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--scope-mode exclude_top_r|lowest_r] [--step-order evict_first|attend_first]
                    [--all-workloads] [--readings] [--no-extras]

On one GPU the line also carries the calls with few units (`few_units`), the block-wise and grouped-query steps
(`multi_query`), the four readings (`readings`), the two other decode workloads (`workloads`) and the prompt pass
(`prefill`); `--no-extras` trims it to the decode step, the calls with few units and the prompt pass.  `--readings` adds the three other combinations of scope reading and step order on the same workload, and
`--all-workloads` the serving-batch and long-context decode workloads, as extra keys of the same line.

N > 1 (under torch.distributed.run): every rank runs the same-sized workload on its own GPU with its own
seed (units are independent; no data-path collective) and the aggregate is reported: weak scaling.
`--impl reference` times the fp64 CPU oracle instead (rank 0 only), on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import workloads as W

# dram__bytes_read.sum + dram__bytes_write.sum of decode_step_kernel, per unit, from a profiler capture
NCU_TRAFFIC = {"kernel_hash": "0d5a2a112d144a25", "shape": (1024, 128, "bf16"), "dram_bytes_per_unit": 571663}

METRIC = "decode_tokens_per_s"
UNIT = "tokens/s"
SCOPE_MODES = {"exclude_top_r": 0, "lowest_r": 1}
STEP_ORDERS = {"evict_first": 0, "attend_first": 1}
MODE_NAMES = {0: "EXCLUDE_TOP_R", 1: "LOWEST_R"}
ORDER_NAMES = {0: "EVICT_FIRST", 1: "ATTEND_FIRST"}
MIN_WARMUP = 10


# ----------------------------------------------------------------------------------------- helpers

def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), float(p["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


def algorithmic_bytes_per_unit_step(B: int, d: int, elem: int) -> int:
    """K and V read once (2*B*d elements) plus s, q, n read and written (24*B bytes)."""
    return 2 * B * d * elem + 24 * B


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [x.strip() for x in line.split(",")]))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        rows = [r for t, r in self.rows if t0 <= t <= t1 + 0.1] or [r for _, r in self.rows[-3:]]
        sm, reasons, mx = [], set(), None
        for r in rows:
            try:
                sm.append(float(r[1])); mx = float(r[2])
            except (ValueError, IndexError):
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def aggregate(tokens_per_rank: float, seconds_this_rank: float, world: int, backend_device=None) -> tuple:
    """Whole-job throughput: tokens of all ranks / max over ranks of the elapsed time."""
    if world == 1:
        return tokens_per_rank / seconds_this_rank, seconds_this_rank
    import torch.distributed as dist
    t = torch.tensor([seconds_this_rank], dtype=torch.float64, device=backend_device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    tmax = float(t.item())
    return world * tokens_per_rank / tmax, tmax


# ----------------------------------------------------------------------------------------- workload

def build_cache(w, device, R, seed_offset=0, scope_mode=0):
    """Prefill every unit with the library (prompt -> budget B), layer-chunk by layer-chunk."""
    w = W.scaled(w, seed=w.seed + 1000 * seed_offset)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, device)
    lens = W.prompt_lens(w)
    chunk = min(w.G, 256)
    ws = None
    for b in range(w.S):
        for g0 in range(0, w.G, chunk):
            g1 = min(g0 + chunk, w.G)
            Q, K, V = (t[None] for t in W.prompt_chunk(w, b, g0, g1, lens[b], device))
            sub = R.Cache(1, g1 - g0, w.B, w.d, w.torch_dtype, device)
            need = (R.roco_prefill_workspace_bytes_lowest_r if scope_mode else R.roco_prefill_workspace_bytes)(sub, lens[b])
            if ws is None or ws.numel() < need:
                ws = torch.empty(need, dtype=torch.uint8, device=device)
            R.roco_prefill(Q, K, V, [lens[b]], w.B, w.r, sub, scope_mode=scope_mode, scale=w.scale, workspace=ws)
            for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
                getattr(cache, name)[b, g0:g1].copy_(getattr(sub, name)[0])
            if R.roco_device_status(sub) != 0:
                raise RuntimeError("device status set during prefill")
    return w, cache, lens


def oracle_sample(w, cache, sample_units, n_steps, first_step, t_pos, scope_mode=0, step_order=0):
    """Times the fp64 oracle (as it stands) on `sample_units` of the cache for n_steps decode steps."""
    import oracle
    from workloads import unit_view, widen
    st = oracle.State(widen(unit_view(cache.K, sample_units)), widen(unit_view(cache.V, sample_units)),
                      widen(unit_view(cache.s, sample_units)), widen(unit_view(cache.q, sample_units)),
                      unit_view(cache.n, sample_units).cpu().numpy().copy(),
                      unit_view(cache.pos, sample_units).cpu().numpy().copy(),
                      unit_view(cache.live, sample_units).cpu().numpy().copy(),
                      unit_view(cache.t_next, sample_units).cpu().numpy().copy())
    toks = []
    tp = list(t_pos)
    for i in range(n_steps):
        q, k, v = W.decode_tokens(w, first_step + i, tp, cache.K.device)
        toks.append(tuple(widen(unit_view(x, sample_units)) for x in (q, k, v)))
        tp = [t + 1 for t in tp]
    per_step = []
    for q, k, v in toks:
        t0 = time.perf_counter()
        oracle.decode_step(st, q, k, v, w.r, scope_mode, step_order, w.scale)
        per_step.append(time.perf_counter() - t0)
    return per_step, oracle.threads()


def prefill_oracle_baseline(w, L, n_units=16):
    """The fp64 oracle's prefill (statistics + select-to-budget) on `n_units` units of the prompt workload, timed
    on the host cores; returns the cpu_baseline block (prompt tokens/s of the whole workload, scaled by U/sample)."""
    import oracle
    Q, K, V = (x.to(torch.float64).numpy() for x in W.prompt_chunk(w, 0, 0, n_units, L, "cpu"))
    t0 = time.perf_counter()
    oracle.prefill(Q, K, V, [L] * n_units, w.B, w.r, oracle.EXCLUDE_TOP_R, w.scale)
    sec = time.perf_counter() - t0
    return {"value": W.ALL[w.name].S * L / (sec * W.ALL[w.name].U / n_units), "unit": "prompt tokens/s",
            "cores": oracle.threads(), "kind": "oracle", "seconds": sec,
            "sample": f"{n_units} of {W.ALL[w.name].U} units, whole prompt of {L} tokens each; scaled by U/sample"}


def prefill_bench(R, device, small=False, reps=5, workload="llama7b_prefill", with_oracle=False):
    """Prefill-stage statistics + eviction to budget on the Llama-2-7B-shape prompt workload (8192-token causal
    prompt, 32 x 32 heads, evicted to B = 2048 with r = 256): best of `reps` calls of roco_prefill.  Workloads whose
    prompts do not fit at once (long_context: 32768 tokens x 4096 units) are measured on one sequence's first 8
    layers (256 units) and scaled by the unit count (units are independent; the figure is labelled)."""
    w = W.ALL[workload]
    scale_units = 1.0
    if small:
        w = W.scaled(w, layers=1)
    if w.S * w.G * w.prompt_hi > (1 << 24) * 2:        # more than 32 Mi prompt tokens of units: measure a slice
        full_units = w.U
        w = W.scaled(w, S=1, layers=8)
        scale_units = full_units / w.U
    L = w.prompt_lo
    _, bf16_peak, which = peaks()
    chunk = min(w.G, 256)
    Q, K, V = (torch.cat(x)[None] for x in zip(*[W.prompt_chunk(w, 0, g0, g0 + chunk, L, device)
                                                  for g0 in range(0, w.G, chunk)]))
    cache = R.Cache(1, w.G, w.B, w.d, w.torch_dtype, device)
    ws = R.roco_prefill(Q, K, V, [L], w.B, w.r, cache, scale=w.scale)
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        R.roco_prefill(Q, K, V, [L], w.B, w.r, cache, scale=w.scale, workspace=ws)
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) / 1e3)
    # attention output of the same prompt pass (optional second call; not part of the statistics figure)
    attend = None
    if R.roco_prefill_uses_tensor_cores(cache):
        lse = torch.zeros(1, w.G, L, dtype=torch.float32, device=device)
        R.roco_prefill(Q, K, V, [L], w.B, w.r, cache, scale=w.scale, workspace=ws, lse_out=lse)
        out = torch.empty_like(Q)
        aws = R.roco_prefill_attend(cache, Q, K, V, [L], lse, out, scale=w.scale)
        torch.cuda.synchronize()
        best_a = float("inf")
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            R.roco_prefill_attend(cache, Q, K, V, [L], lse, out, scale=w.scale, workspace=aws)
            e1.record()
            torch.cuda.synchronize()
            best_a = min(best_a, e0.elapsed_time(e1) / 1e3)
        Tt = (L + 127) // 128
        ex_a = w.U * (Tt * (Tt + 1) // 2) * 2 * 2 * 128 ** 3      # Q K^T and P V per tile
        attend = {"ms": best_a * 1e3, "ms_whole_workload": best_a * 1e3 * scale_units,
                  "tflops_executed": ex_a / best_a / 1e12, "frac_executed": ex_a / best_a / 1e12 / bf16_peak}
        # the same outputs from one call: the sweep that yields the row log-sum-exp also accumulates P.V
        best_f = float("inf")
        R.roco_prefill(Q, K, V, [L], w.B, w.r, cache, scale=w.scale, workspace=ws, attn_out=out)
        torch.cuda.synchronize()
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            R.roco_prefill(Q, K, V, [L], w.B, w.r, cache, scale=w.scale, workspace=ws, attn_out=out)
            e1.record()
            torch.cuda.synchronize()
            best_f = min(best_f, e0.elapsed_time(e1) / 1e3)
        ex_f = w.U * (Tt * (Tt + 1) // 2) * 3 * 2 * 128 ** 3      # scores + P V in the sweep, scores again for the statistics
        attend["fused_call"] = {"ms": best_f * 1e3, "ms_whole_workload": best_f * 1e3 * scale_units,
                                "what": "roco_prefill_with_output: statistics + eviction to budget + attention output, "
                                        "three L x L contractions",
                                "ms_separate_calls": (best + best_a) * 1e3,
                                "tflops_executed": ex_f / best_f / 1e12,
                                "frac_executed": ex_f / best_f / 1e12 / bf16_peak}
        del out, lse
    if R.roco_device_status(cache) != 0:
        raise RuntimeError("device status word set during prefill")
    T = (L + 127) // 128
    executed = 2 * w.U * (T * (T + 1) // 2) * 2 * 128 ** 3          # two passes of 128^3 tile products
    algorithmic = w.U * L * (L + 1) * w.d                            # one causal Q K^T
    tc = R.roco_prefill_uses_tensor_cores(cache)
    return {"workload": f"{w.name}: {w.layers} layers x {w.heads} heads, d={w.d}, {w.dtype}, causal prompt {L} -> "
                        f"B={w.B}, r={w.r}, EXCLUDE_TOP_R" +
                        (f" (measured on {w.U} units; whole-workload time = x{scale_units:g})" if scale_units != 1 else ""),
            "ms": best * 1e3, "ms_whole_workload": best * 1e3 * scale_units,
            "tokens_per_s": W.ALL[workload].S * L / (best * scale_units) if not small else w.S * L / best,
            "tensor_cores": tc, "tflops_executed": executed / best / 1e12,
            "tflops_algorithmic": algorithmic / best / 1e12, "peak_tflops": bf16_peak, "peak_source": f"of {which}",
            "frac_executed": executed / best / 1e12 / bf16_peak,
            "frac_algorithmic": algorithmic / best / 1e12 / bf16_peak,
            "launches_per_call": 4, "timing": f"best of {reps} whole roco_prefill calls (both passes, select, gather)",
            "exp_unit_bound": exp_unit_bound(w.U, T, best), "attention_output": attend,
            "cpu_baseline": prefill_oracle_baseline(w, L, 64 if L <= 8192 else 8) if with_oracle else None}


def exp_unit_bound(U, T, seconds):
    """What the exponentials alone cost: both passes evaluate one exponential per score, 128 x 128 per tile
    product; the SM's exponential unit retires 16 per cycle, and the kernels move two of every eight onto the
    FMA pipe.  At the maximum SM clock, all SMs busy."""
    p = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(
        os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
    mhz, sms = float(p.get("sm_max_mhz", 1965.0)), 148
    tiles = 2 * U * (T * (T + 1) // 2)
    ms = tiles * (128 * 128 / 16) * 0.75 / (sms * mhz * 1e3)
    return {"ms": ms, "frac_of_measured_time": ms / (seconds * 1e3),
            "note": "16384 exponentials per tile product / 16 per cycle per SM x 0.75 (a quarter runs as a "
                    "polynomial on the FMA pipe), 148 SMs at the maximum SM clock; the MMA work of the same tile "
                    "is 512 cycles"}


def multi_bench(R, cache, w, device, reps=6):
    """Block-wise evict-and-encode (b tokens per pass over the cache) and grouped-query decode on the cache of the
    decode workload: ms per step, tokens encoded per second, and the speed-up over token-wise eviction (b = 1)."""
    hbm_peak, _, which = peaks()
    elem = 2 if w.dtype == "bf16" else 4
    alg = algorithmic_bytes_per_unit_step(w.B, w.d, elem) * w.U
    res = {"block": [], "gqa": [], "peak_source": f"of {which}"}
    dt = w.torch_dtype
    gen = torch.Generator(device=device); gen.manual_seed(99)
    def timed(fn):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record(); torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return statistics.median(ts)
    base = None
    for b in (1, 2, 4, 8, 16):
        Q, K, V = (torch.randn(w.S, w.G, b, w.d, device=device, generator=gen).to(dt) for _ in range(3))
        out = torch.zeros(w.S, w.G, b, w.d, dtype=dt, device=device)
        ev = torch.zeros(w.S, w.G, b, dtype=torch.int32, device=device)
        ms = timed(lambda: R.roco_block_step(cache, Q, K, V, w.r, out, ev, scale=w.scale))
        base = base or ms
        res["block"].append({"b": b, "ms_per_step": ms, "tokens_per_s": w.S * b / ms * 1e3,
                             "speedup_vs_b1_per_token": base * b / ms, "hbm_frac": alg / ms / 1e6 / hbm_peak})
    res["few_units"] = few_units_bench(R, cache, w, device, reps)
    # the paper's prefill scheme: the whole prompt through the budgeted cache, b tokens per evict-and-encode step
    # (its Table "block-wise eviction" reports the speed-up over b = 1)
    Lp = w.prompt_lo
    Qp, Kp, Vp = (torch.randn(w.S, w.G, Lp, w.d, device=device, generator=gen, dtype=torch.float32).to(dt)
                  for _ in range(3))
    outp = torch.empty_like(Qp)
    pc = R.Cache(w.S, w.G, w.B, w.d, dt, device)
    res["blockwise_prefill"] = []
    t_b1 = None
    for b in (1, 4, 16):
        evp = torch.zeros(w.S, w.G, b, dtype=torch.int32, device=device)
        pc.live.zero_(); pc.t_next.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        R.roco_prefill_blockwise(Qp, Kp, Vp, [Lp] * w.S, b, w.r, pc, outp, evp, scale=w.scale)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        t_b1 = t_b1 or ms
        res["blockwise_prefill"].append({"b": b, "prompt": Lp, "ms": ms, "prompt_tokens_per_s": w.S * Lp / ms * 1e3,
                                         "speedup_vs_b1": t_b1 / ms})
    del Qp, Kp, Vp, outp, pc
    # block-wise evict-and-encode on key-value heads shared by `group` query heads (b x group <= 16 query rows)
    res["gqa_block"] = []
    for b, g in ((4, 4), (8, 2), (2, 8)):
        Q = torch.randn(w.S, w.G, b, g, w.d, device=device, generator=gen).to(dt)
        K, V = (torch.randn(w.S, w.G, b, w.d, device=device, generator=gen).to(dt) for _ in range(2))
        out = torch.zeros(w.S, w.G, b, g, w.d, dtype=dt, device=device)
        ev = torch.zeros(w.S, w.G, b, dtype=torch.int32, device=device)
        ms = timed(lambda: R.roco_gqa_block_step(cache, Q, K, V, w.r, out, ev, scale=w.scale))
        res["gqa_block"].append({"b": b, "group": g, "ms_per_step": ms, "tokens_per_s": w.S * b / ms * 1e3,
                                 "hbm_frac": alg / ms / 1e6 / hbm_peak})
    for g in (4, 8):
        Q = torch.randn(w.S, w.G, g, w.d, device=device, generator=gen).to(dt)
        k, v = (torch.randn(w.S, w.G, w.d, device=device, generator=gen).to(dt) for _ in range(2))
        out = torch.zeros(w.S, w.G, g, w.d, dtype=dt, device=device)
        ev = torch.zeros(w.S, w.G, dtype=torch.int32, device=device)
        ms = timed(lambda: R.roco_gqa_decode_step(cache, Q, k, v, w.r, out, ev, scale=w.scale))
        res["gqa"].append({"group": g, "ms_per_step": ms, "hbm_frac": alg / ms / 1e6 / hbm_peak})
    return res


def few_units_bench(R, cache, w, device, reps=6):
    """Decode calls with few units (one layer at a time, what a transformer's decode loop issues): one layer of the
    decode workload, and one layer of a single long sequence (32 units, B = 8192).  Paths: one CTA per unit, the
    three-launch split, the one-launch cluster kernel, and a bare read of the same number of bytes.  Two timings
    each: a single launch between two events with L2 flushed before it (includes the launch and event overhead of a
    lone call), and a sweep over 8 distinct caches back to back (every call still reads cold rows); the sweep is also
    timed as one replay of a CUDA graph that holds its 8 calls."""
    hbm_peak, _, which = peaks()
    elem = 2 if w.dtype == "bf16" else 4
    dt = w.torch_dtype
    gen = torch.Generator(device=device); gen.manual_seed(98)
    # calls with few units (one layer at a time, what a transformer's decode loop does): the same step with each
    # unit's slots divided among several CTAs.  Two cases: one layer of the decode workload, and one layer of a
    # single long-context sequence (32 units, B = 8192).  L2 is flushed between launches (the caches are small).
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    def timed_cold(fn):
        ts = []
        for _ in range(reps + 2):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record(); torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return statistics.median(ts[2:])
    sub = R.Cache(w.S, w.heads, w.B, w.d, dt, device)
    for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
        getattr(sub, name).copy_(getattr(cache, name)[:, :w.heads])
    wl = W.scaled(W.LONG_CONTEXT, S=1, layers=1, prompt_lo=8192, prompt_hi=8192, B=8192)
    _, long_cache, _ = build_cache(wl, device, R)
    out_rows = []
    n_layers = 8   # distinct caches swept back to back: together far larger than L2, so every call reads cold rows

    def clone_cache(src):
        c = R.Cache(src.S, src.G, src.B, src.d, dt, device)
        for name in ("K", "V", "s", "q", "n", "pos", "live", "t_next"):
            getattr(c, name).copy_(getattr(src, name))
        return c

    def timed_sweep(fns):
        """One call per cache of the sweep, back to back on the stream (what a decode loop over layers issues);
        median over repetitions of the time per call."""
        ts = []
        for _ in range(reps + 2):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for fn in fns:
                fn()
            e1.record(); torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) / len(fns))
        return statistics.median(ts[2:])

    def timed_graph(fns):
        """The same sweep captured once in a CUDA graph and replayed: what a decode loop pays per call when it does
        not launch from the host every time."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for fn in fns:
                fn()
        ts = []
        for _ in range(reps + 2):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); g.replay(); e1.record(); torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) / len(fns))
        del g
        return statistics.median(ts[2:])

    for label, cch, rr in ((f"{sub.U} units, B={sub.B}", sub, w.r), (f"{long_cache.U} units, B={long_cache.B}", long_cache, wl.r)):
        algb = algorithmic_bytes_per_unit_step(cch.B, cch.d, elem) * cch.U
        q1, k1, v1 = (torch.randn(cch.S, cch.G, cch.d, device=device, generator=gen).to(dt) for _ in range(3))
        out1 = torch.zeros(cch.S, cch.G, cch.d, dtype=dt, device=device)
        ev1 = torch.zeros(cch.S, cch.G, dtype=torch.int32, device=device)
        layers = [clone_cache(cch) for _ in range(n_layers)]
        sc = cch.d ** -0.5

        def row(name, make):
            """make(cache) -> callable of one step on that cache."""
            iso = timed_cold(make(cch))
            sweep = timed_sweep([make(c) for c in layers])
            graph = timed_graph([make(c) for c in layers])
            return {"path": name, "us_per_step": iso * 1e3, "hbm_frac": algb / iso / 1e6 / hbm_peak,
                    "us_per_step_layer_sweep": sweep * 1e3, "hbm_frac_layer_sweep": algb / sweep / 1e6 / hbm_peak,
                    "us_per_step_graph": graph * 1e3, "hbm_frac_graph": algb / graph / 1e6 / hbm_peak}

        rows = [row("one CTA per unit", lambda c: (lambda: R.roco_decode_step_cluster(c, q1, k1, v1, rr, out1, ev1, ranks=1,
                                                                                      scale=sc)))]
        rows[-1]["splits"] = 0
        for sp in (2, 4, 8):
            ws = torch.empty(R.roco_decode_split_workspace_bytes(cch, sp), dtype=torch.uint8, device=device)
            rows.append(row(f"three launches, {sp} splits",
                            lambda c, sp=sp, ws=ws: (lambda: R.roco_decode_step_split(c, q1, k1, v1, rr, sp, out1, ev1, ws, scale=sc))))
            rows[-1]["splits"] = sp
        kr = R.roco_decode_cluster_ranks(cch)
        for order, oname in ((0, "EVICT_FIRST"), (1, "ATTEND_FIRST")):
            if kr > 1:
                rows.append(row(f"one launch, cluster of {kr} CTAs per unit (what roco_decode_step picks), {oname}",
                                lambda c, order=order: (lambda: R.roco_decode_step_cluster(c, q1, k1, v1, rr, out1, ev1,
                                                                                           step_order=order, ranks=kr, scale=sc))))
                rows[-1]["ranks"] = kr
        # what a bare read of the same number of bytes takes, launched the same two ways (own streaming kernel)
        n_bytes = (algb // 16) * 16
        bufs = [torch.empty(n_bytes, dtype=torch.uint8, device=device) for _ in range(n_layers)]
        sink = torch.zeros(1, dtype=torch.int64, device=device)
        buf_of = {id(c): b for c, b in zip(layers, bufs)}
        buf_of[id(cch)] = bufs[0]
        rows.append(row("bare read of the same bytes",
                        lambda c: (lambda b=buf_of[id(c)]: R.roco_selftest_read_stream(b, sink))))
        out_rows.append({"case": label, "algorithmic_bytes": algb, "layers_in_sweep": n_layers, "rows": rows})
        del layers, bufs
    del flush, long_cache
    return out_rows


def describe(w, world, scope_mode=0, step_order=0):
    elem = 2 if w.dtype == "bf16" else 4
    return {"workload": f"{w.name}: S={w.S} x {w.layers} layers x {w.heads} heads, d={w.d}, {w.dtype}, "
                        f"prompt {w.prompt_lo}" + (f"-{w.prompt_hi}" if w.prompt_hi != w.prompt_lo else "") +
                        f" -> B={w.B}, r={w.r}, {MODE_NAMES[scope_mode]}, {ORDER_NAMES[step_order]}",
            "units": w.U, "budget": w.B, "scope_r": w.r,
            "l2": "inputs larger than L2 (K+V cache per step %.2f GB)" % (w.U * 2 * w.B * w.d * elem / 1e9),
            "parallelism": f"units sharded over {world} GPU(s), no collective" if world > 1 else "1 GPU"}


def reference_arm(args, steps, warmup):
    """The fp64 oracle as it stands, on the host cores only (no GPU): a sample of units of the same workload is
    prefilled and stepped by the oracle; its time is scaled by U / sample (units are independent)."""
    import oracle
    w = W.ALL[args.workload]
    n_units = min(w.G, 32)
    lens = W.prompt_lens(w)
    Q, K, V = (x[None].to(torch.float64).numpy() for x in W.prompt_chunk(w, 0, 0, n_units, lens[0], "cpu"))
    mode, order = SCOPE_MODES[args.scope_mode], STEP_ORDERS[args.step_order]
    res = oracle.prefill(Q[0], K[0], V[0], [lens[0]] * n_units, w.B, w.r, mode, w.scale)
    st = res.state
    per_step = []
    tp = list(lens)
    for i in range(warmup + steps):
        q, k, v = (x[0, :n_units].to(torch.float64).numpy() for x in W.decode_tokens(w, i, tp, "cpu"))
        t0 = time.perf_counter()
        oracle.decode_step(st, q, k, v, w.r, mode, order, w.scale)
        per_step.append(time.perf_counter() - t0)
        tp = [t + 1 for t in tp]
    timed = per_step[warmup:]
    sec = sum(timed)
    value = (n_units * len(timed) / sec) * w.S / w.U
    cores = oracle.threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warmup, "ms_per_step": 1e3 * sec / len(timed) * w.U / n_units, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": describe(w, 1, mode, order),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{n_units} of {w.U} units, every step; time scaled by U/sample"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0




# ----------------------------------------------------------------------------------------- decode measurement

def kernel_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for fn in ("decode.cu", "select.cuh", "common.cuh"):
        h.update(open(os.path.join(ROOT, "paper_2402_06262_b200", "csrc", fn), "rb").read())
    return h.hexdigest()[:16]


def read_stream_gbs(R, device, gib=4, reps=5):
    """Read-only streaming rate of this GPU: the library's own sum-over-a-buffer kernel over `gib` GiB, best of reps."""
    buf = torch.empty(gib << 30, dtype=torch.uint8, device=device)
    buf.fill_(1)
    sink = torch.zeros(1, dtype=torch.int64, device=device)
    R.roco_selftest_read_stream(buf, sink)
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); R.roco_selftest_read_stream(buf, sink); e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) / 1e3)
    n = buf.numel()
    del buf
    torch.cuda.empty_cache()
    return n / best / 1e9


def decode_bench(R, w0, device, rank, world, local_rank, steps, warmup, scope_mode, step_order, e2e_steps=32,
                 clocks=True, read_gbs=None):
    """Builds the workload's cache with the library's prefill, then times `steps` decode steps (one launch each)
    after `warmup` untimed ones, device-timed per launch; then the end-to-end rate through the host-buffer entry
    points.  Returns (result dict, workload, cache, lens, steps consumed)."""
    w, cache, lens = build_cache(w0, device, R, seed_offset=rank, scope_mode=scope_mode)
    elem = 2 if w.dtype == "bf16" else 4
    total = warmup + steps
    t_pos = list(lens)
    toks, tp = [], list(t_pos)
    for i in range(total):                      # inputs of every step resident on the device before the timed region
        toks.append(W.decode_tokens(w, i, tp, device))
        tp = [t + 1 for t in tp]
    out = torch.zeros(w.S, w.G, w.d, dtype=w.torch_dtype, device=device)
    ev_slot = torch.zeros(w.S, w.G, dtype=torch.int32, device=device)
    ev_pos = torch.zeros_like(ev_slot)

    def step(i):
        q, k, v = toks[i]
        R.roco_decode_step(cache, q, k, v, w.r, out, ev_slot, ev_pos, scope_mode=scope_mode, step_order=step_order,
                           scale=w.scale)

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
    sampler = None
    if clocks:
        visible = [x for x in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if x]
        sampler = ClockSampler(visible[local_rank] if local_rank < len(visible) else local_rank)
        sampler.start()
        time.sleep(0.3)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    torch.cuda.synchronize()
    t_wall0 = time.perf_counter()
    evs[0].record()
    for i in range(steps):
        step(warmup + i)
        evs[i + 1].record()
    torch.cuda.synchronize()
    t_wall1 = time.perf_counter()
    if world > 1:
        torch.distributed.barrier()
    clk = sampler.stop(t_wall0, t_wall1) if sampler else None
    launch_ms = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]
    sec = evs[0].elapsed_time(evs[steps]) / 1e3
    if R.roco_device_status(cache) != 0:
        raise RuntimeError("device status word set during the timed region")
    value, tmax = aggregate(w.S * steps, sec, world, device)
    del toks

    # ---- end to end: pinned host tensors in, results out, every step, through the public host-buffer entry points
    # (two steps in flight: the copies of one step run under the kernel of the other), and through the
    # synchronising single call beside it
    h_toks = [tuple(x.cpu().pin_memory() for x in W.decode_tokens(w, total + i, [t + total + i for t in t_pos], device))
              for i in range(2 * e2e_steps)]
    h_res = [(torch.zeros(w.S, w.G, w.d, dtype=w.torch_dtype).pin_memory(),
              torch.zeros(w.S, w.G, dtype=torch.int32).pin_memory(),
              torch.zeros(w.S, w.G, dtype=torch.int32).pin_memory()) for _ in range(2)]
    staging = torch.empty(R.roco_decode_host_pipeline_staging_bytes(cache), dtype=torch.uint8, device=device)
    kw = dict(scope_mode=scope_mode, step_order=step_order, scale=w.scale)
    R.roco_decode_step_host(cache, *h_toks[0], w.r, *h_res[0], staging, **kw)           # creates the copy streams
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(1, e2e_steps):
        R.roco_decode_step_host_begin(cache, *h_toks[i], w.r, *h_res[i & 1], staging, **kw)
        if i > 1:
            R.roco_decode_step_host_end()
    R.roco_decode_step_host_end()
    e1.record()
    torch.cuda.synchronize()
    pipe_sec = e0.elapsed_time(e1) / 1e3
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(e2e_steps, 2 * e2e_steps - 1):
        R.roco_decode_step_host(cache, *h_toks[i], w.r, *h_res[0], staging, **kw)
    e1.record()
    torch.cuda.synchronize()
    sync_sec = e0.elapsed_time(e1) / 1e3
    n_e2e = e2e_steps - 1
    e2e_value, _ = aggregate(w.S * n_e2e, pipe_sec, world, device)
    e2e_sync, _ = aggregate(w.S * n_e2e, sync_sec, world, device)
    vec = w.U * w.d * elem
    e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 3 * vec, "d2h_bytes_per_step": vec + 8 * w.U,
           "steps": n_e2e, "api": "roco_decode_step_host_begin / _end, two steps in flight",
           "frac_of_device_timed": e2e_value / value,
           "synchronising_single_call": {"value": e2e_sync, "api": "roco_decode_step_host"}}
    if R.roco_device_status(cache) != 0:
        raise RuntimeError("device status word set during the end-to-end steps")
    del h_toks, staging

    # ---- roofline of the decode kernel (the only kernel in a step)
    hbm_peak, _, which = peaks()
    alg = algorithmic_bytes_per_unit_step(w.B, w.d, elem) * w.U
    avg_launch = sum(launch_ms) / len(launch_ms) / 1e3
    med_launch = statistics.median(launch_ms) / 1e3
    roofline = {"bound": "hbm", "achieved": alg / avg_launch / 1e9, "peak": hbm_peak, "unit": "GB/s",
                "frac": alg / avg_launch / 1e9 / hbm_peak, "traffic": None, "peak_source": f"of {which}",
                "kernel": "decode_step_kernel", "algorithmic_bytes_per_launch": alg,
                "avg_launch_ms": avg_launch * 1e3, "median_launch_ms": med_launch * 1e3,
                "frac_of_nominal_8TBs": alg / avg_launch / 8e12}
    if read_gbs:
        roofline["read_stream_gbs"] = read_gbs
        roofline["frac_of_read_stream"] = alg / avg_launch / 1e9 / read_gbs
    # DRAM bytes per unit from a profiler capture of a 512-unit launch of the same shape (traffic grows in
    # proportion to the units); dropped as soon as the kernel sources differ from the captured ones
    if kernel_hash() == NCU_TRAFFIC["kernel_hash"] and (w.B, w.d, w.dtype) == NCU_TRAFFIC["shape"] and \
            (scope_mode, step_order) == (0, 0):
        roofline["traffic"] = NCU_TRAFFIC["dram_bytes_per_unit"] * w.U
    res = {"value": value, "ms_per_step": statistics.median(launch_ms) if world == 1 else 1e3 * tmax / steps,
           "ms_per_step_mean": 1e3 * tmax / steps, "clocks": clk, "e2e": e2e, "roofline": roofline,
           "config": describe(w, world, scope_mode, step_order)}
    return res, w, cache, lens, total + 2 * e2e_steps


# ----------------------------------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=MIN_WARMUP)
    ap.add_argument("--impl", default="roco", choices=["roco", "reference"])
    ap.add_argument("--workload", default="llama7b_decode")
    ap.add_argument("--small", action="store_true", help="1/16 of the units (for profiler captures)")
    ap.add_argument("--prefill-only", action="store_true", help="run only the prefill measurement")
    ap.add_argument("--no-prefill", action="store_true", help="skip the prefill measurement")
    ap.add_argument("--extras", action="store_true",
                    help="time the block-wise and grouped-query steps too (the default on one GPU; with several, only "
                         "when asked)")
    ap.add_argument("--no-extras", action="store_true", help="skip the block-wise and grouped-query steps")
    ap.add_argument("--no-few-units", action="store_true", help="skip the calls with few units (one layer at a time)")
    ap.add_argument("--prefill-workload", default="llama7b_prefill", help="workload of the prefill measurement")
    ap.add_argument("--scope-r", type=int, default=None, help="override the workload's scope parameter r")
    ap.add_argument("--scope-mode", default="exclude_top_r", choices=sorted(SCOPE_MODES),
                    help="reading of the eviction scope (Sec. 4.3: all but the r highest-variance tokens; Sec. 1: "
                         "the r lowest-variance tokens)")
    ap.add_argument("--step-order", default="evict_first", choices=sorted(STEP_ORDERS),
                    help="order inside a decode step (Fig. 1: evict, insert, attend; or attend, then evict and insert)")
    ap.add_argument("--readings", action="store_true",
                    help="also time the other three combinations of scope reading and step order (extra key)")
    ap.add_argument("--all-workloads", action="store_true",
                    help="also time the serving-batch and long-context decode workloads (extra key)")
    args = ap.parse_args()
    rank, local_rank, world = dist_env()
    if args.impl == "reference" and rank != 0:
        return 0
    steps, warmup = args.steps, max(args.warmup, MIN_WARMUP)

    if args.impl == "reference":
        return reference_arm(args, steps, warmup)

    import paper_2402_06262_b200 as R
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(device))

    if args.prefill_only:
        print(json.dumps({"prefill": prefill_bench(R, device, small=args.small, workload=args.prefill_workload,
                                                   with_oracle=(rank == 0 and not args.small))}))
        return 0
    w0 = W.ALL[args.workload]
    if args.scope_r is not None:
        w0 = W.scaled(w0, r=args.scope_r)
    if args.small:
        w0 = W.scaled(w0, layers=max(1, w0.layers // 16))
    mode, order = SCOPE_MODES[args.scope_mode], STEP_ORDERS[args.step_order]
    read_gbs = read_stream_gbs(R, device)
    res, w, cache, lens, used = decode_bench(R, w0, device, rank, world, local_rank, steps, warmup, mode, order,
                                             read_gbs=read_gbs)

    line = {"metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": res["ms_per_step"], "ms_per_step_mean": res["ms_per_step_mean"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 K/V, fp32 softmax and statistics" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": res["config"], "clocks": res["clocks"], "e2e": res["e2e"], "gpu_launches": steps,
            "roofline": res["roofline"]}

    torch.cuda.empty_cache()
    extras = (args.extras or world == 1) and not args.no_extras and w.dtype == "bf16"
    if extras and args.no_few_units and not args.extras:
        extras = False   # a run trimmed to the decode step alone
    if extras:
        try:
            line["multi_query"] = multi_bench(R, cache, w, device)
            line["few_units"] = line["multi_query"].pop("few_units")
        except Exception as e:   # the headline must not depend on the extra rows
            line["multi_query"] = {"error": f"{type(e).__name__}: {e}"}
        if R.roco_device_status(cache) != 0:
            raise RuntimeError("device status word set during the multi-query steps")
    elif not args.no_few_units and w.dtype == "bf16":
        line["few_units"] = few_units_bench(R, cache, w, device)
        if R.roco_device_status(cache) != 0:
            raise RuntimeError("device status word set during the multi-query steps")

    if rank == 0:   # the oracle beside the GPU figure, same run, same cache, on a bounded sample of units
        n_units, n_steps = min(w.U, 512), 512
        sample = sorted(np.random.default_rng(0).choice(w.U, n_units, replace=False).tolist())
        per_step, cores = oracle_sample(w, cache, sample, n_steps, used, [t + used for t in lens], mode, order)
        osec = sum(per_step)
        line["cpu_baseline"] = {"value": (n_units * n_steps / osec) * w.S / w.U, "unit": UNIT, "cores": cores,
                                "kind": "oracle", "seconds": osec,
                                "sample": f"{n_units} of {w.U} units x {n_steps} decode steps; scaled by U/sample"}
    del cache
    torch.cuda.empty_cache()

    def brief(r):
        return {"config": r["config"]["workload"], "units": r["config"]["units"], "tokens_per_s": r["value"],
                "ms_per_step": r["ms_per_step"], "ms_per_step_mean": r["ms_per_step_mean"],
                "gbs": r["roofline"]["achieved"], "frac": r["roofline"]["frac"],
                "frac_of_nominal_8TBs": r["roofline"]["frac_of_nominal_8TBs"],
                "frac_of_read_stream": r["roofline"].get("frac_of_read_stream"),
                "e2e_tokens_per_s": r["e2e"]["value"], "e2e_frac_of_device_timed": r["e2e"]["frac_of_device_timed"]}

    # on one GPU the plain run carries the extra keys too (they take about 20 s)
    full_line = (world == 1 and not args.no_extras and not args.no_few_units and not args.small and
                 not args.no_prefill and args.workload == "llama7b_decode")
    if args.readings or full_line:      # the same workload under the other readings of scope and order
        line["readings"] = [dict(brief(res), scope_mode=args.scope_mode, step_order=args.step_order)]
        for sm_name, so_name in [(a, b) for a in ("exclude_top_r", "lowest_r") for b in ("evict_first", "attend_first")]:
            if (sm_name, so_name) == (args.scope_mode, args.step_order):
                continue
            r2, _, c2, _, _ = decode_bench(R, w0, device, rank, world, local_rank, min(steps, 64), warmup,
                                           SCOPE_MODES[sm_name], STEP_ORDERS[so_name], e2e_steps=8, clocks=False,
                                           read_gbs=read_gbs)
            line["readings"].append(dict(brief(r2), scope_mode=sm_name, step_order=so_name))
            del c2
            torch.cuda.empty_cache()
    if args.all_workloads or full_line:  # the other decode workloads at their full sizes (extra keys, not the headline)
        line["workloads"] = {}
        for name in ("llama13b_serving", "long_context"):
            if name == args.workload:
                continue
            r2, _, c2, _, _ = decode_bench(R, W.ALL[name], device, rank, world, local_rank, min(steps, 64), warmup,
                                           mode, order, e2e_steps=8, clocks=False, read_gbs=read_gbs)
            line["workloads"][name] = brief(r2)
            del c2
            torch.cuda.empty_cache()

    if not args.no_prefill:
        line["prefill"] = prefill_bench(R, device, small=args.small, workload=args.prefill_workload,
                                        with_oracle=(rank == 0 and not args.small))
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
