"""roco_prefill_static -- the prefill entry point for callers that cannot allocate device memory at call
time (a plug-in inside a serving runtime whose pool owns the GPU, or a loop that must not call cudaMalloc
because it synchronises the device).  Its scratch is an array built into the library, shared by all calls on a
device, and it keeps the previous call's contents.  Checked here: two calls in a row, on different inputs,
each give what roco_prefill gives with a caller-provided workspace; oversized problems are rejected.

This file is collected last on purpose: if the new entry point misbehaves, every other test has already run."""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2402_06262_b200 as R
import workloads as W
from harness import Tally, prefill_parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
NAMES = ("K", "V", "s", "q", "n", "pos", "live", "t_next")


def run_both(w, lens, seed):
    w = W.scaled(w, seed=seed)
    Lmax = max(lens)
    Q, K, V = (torch.stack(x) for x in zip(*[W.prompt_chunk(w, b, 0, w.G, Lmax, DEV) for b in range(w.S)]))
    outs = []
    for static in (False, True):
        cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
        lse, sf, qf = (torch.zeros(w.S, w.G, Lmax, dtype=torch.float32, device=DEV) for _ in range(3))
        if static:
            R.roco_prefill_static(Q, K, V, lens, w.B, w.r, cache, scale=w.scale, lse_out=lse, s_full=sf, q_full=qf)
        else:
            R.roco_prefill(Q, K, V, lens, w.B, w.r, cache, scale=w.scale, lse_out=lse, s_full=sf, q_full=qf)
        torch.cuda.synchronize()
        assert R.roco_device_status(cache) == 0
        outs.append((cache, lse, sf, qf))
    (c0, *f0), (c1, *f1) = outs
    for name in NAMES:
        a, b = getattr(c0, name), getattr(c1, name)
        if a.dtype in (torch.int32,):
            assert torch.equal(a, b), name
        elif name in ("K", "V"):
            live = c0.live.max().item()
            assert torch.equal(a[:, :, :live], b[:, :, :live]), name
        else:
            np.testing.assert_allclose(b.cpu().numpy(), a.cpu().numpy(), rtol=1e-4, atol=1e-30, err_msg=name)
    for a, b, lim in zip(f0, f1, (1e-4, None, None)):
        for bi, L in enumerate(lens):
            x, y = a[bi, :, :L].cpu().numpy(), b[bi, :, :L].cpu().numpy()
            if lim is not None:
                np.testing.assert_allclose(y, x, rtol=0, atol=lim)          # lse
            else:
                np.testing.assert_allclose(y, x, rtol=1e-4, atol=1e-30)     # s_full, q_full


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # bf16, d = 128 (tensor-core path), ragged lengths, eviction to budget; then a different, smaller problem
    # through the same built-in scratch, which still holds the first call's data
    w = W.scaled(W.LLAMA7B_PREFILL, S=2, layers=1, heads=4, prompt_lo=600, prompt_hi=600, B=150, r=20)
    run_both(w, [600, 417], seed=11)
    w2 = W.scaled(W.TOY, prompt_lo=256, prompt_hi=256, B=128, r=16)
    run_both(w2, [256], seed=12)


def test_oversized_problem_is_rejected_with_the_workspace_error():
    w = W.scaled(W.LLAMA7B_PREFILL, S=1, layers=1, heads=2, prompt_lo=64, prompt_hi=64, B=32, r=4)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    Lmax = 400_000                      # 2 units x 400k tokens x 16 bytes of scratch > 8 MiB
    assert R.roco_prefill_workspace_bytes(cache, Lmax) > R.binding.PREFILL_STATIC_SCRATCH_BYTES
    lens = (C.c_int32 * 1)(64)
    dummy = torch.zeros(16, dtype=torch.bfloat16, device=DEV)   # never touched: the size check comes first
    rc = R.lib().roco_prefill_static(dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(), C.cast(lens, C.c_void_p),
                                     Lmax, w.B, w.r, R.ROCO_SCOPE_EXCLUDE_TOP_R, 1, 0.1, C.byref(cache.c), None, None,
                                     None, None)
    assert rc == 3 and "workspace" in R.status_string(rc)


@pytest.mark.parametrize("mode,r", [(R.ROCO_SCOPE_EXCLUDE_TOP_R, 20), (R.ROCO_SCOPE_LOWEST_R, 20)])
def test_static_call_against_the_oracle_and_allocates_nothing(mode, r):
    """The built-in-scratch call compared with the fp64 oracle directly (both scope readings; LOWEST_R also needs
    the sort buffer, which fits here), and a repeat of the call leaves the device's free memory and torch's
    allocator untouched."""
    w = W.scaled(W.LLAMA7B_PREFILL, S=2, layers=1, heads=3, prompt_lo=500, prompt_hi=500, B=160, r=r, seed=21)
    lens = [500, 301]
    Q, K, V = (torch.stack(x) for x in zip(*[W.prompt_chunk(w, b, 0, w.G, 500, DEV) for b in range(w.S)]))
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    tally = Tally()
    prefill_parity(cache, Q, K, V, lens, r, mode, range(w.U), tally, scale=w.scale, static=True)
    assert tally.prefill_units_evicting == w.U
    torch.cuda.synchronize()
    # what may not move: the driver's free memory, and the number of requests torch's allocator has served (the
    # bytes it holds may still drop while the call runs, when Python lets go of earlier temporaries)
    free0 = torch.cuda.mem_get_info()[0]
    served0 = torch.cuda.memory_stats()["allocation.all.allocated"]
    R.roco_prefill_static(Q, K, V, lens, w.B, r, cache, scope_mode=mode, scale=w.scale)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_stats()["allocation.all.allocated"] == served0
    assert R.roco_device_status(cache) == 0


def test_lowest_r_needs_more_scratch_and_is_rejected_earlier():
    """Under ROCO_SCOPE_LOWEST_R a prompt longer than the budget also needs the sort buffer: a problem that fits
    under the other reading is rejected with the workspace status."""
    w = W.scaled(W.LLAMA7B_PREFILL, S=1, layers=1, heads=48, prompt_lo=8192, prompt_hi=8192, B=2048, r=256)
    cache = R.Cache(w.S, w.G, w.B, w.d, w.torch_dtype, DEV)
    assert R.roco_prefill_workspace_bytes(cache, 8192) <= R.binding.PREFILL_STATIC_SCRATCH_BYTES
    assert R.roco_prefill_workspace_bytes_lowest_r(cache, 8192) > R.binding.PREFILL_STATIC_SCRATCH_BYTES
    Q, K, V = (t[None] for t in W.prompt_chunk(w, 0, 0, w.G, 8192, DEV))
    R.roco_prefill_static(Q, K, V, [8192], w.B, w.r, cache, scale=w.scale)            # fits
    with pytest.raises(R.RocoError) as e:
        R.roco_prefill_static(Q, K, V, [8192], w.B, w.r, cache, scope_mode=R.ROCO_SCOPE_LOWEST_R, scale=w.scale)
    assert e.value.code == 3
    torch.cuda.synchronize()
    assert R.roco_device_status(cache) == 0
