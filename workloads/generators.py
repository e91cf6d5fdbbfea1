"""Seeded synthetic inputs for KV-constrained inference with RoCo eviction.

This module only draws random tensors with a prescribed structure (attention
sinks, a shared low-rank component, recurring key bursts).  It contains none of
the method's arithmetic: no softmax, no statistics, no selection.  Both the
CUDA library's tests/benchmarks and the CPU oracle's tests consume the tensors
produced here; a tensor is generated once and the *same bytes* are handed to
both sides (bf16 workloads are rounded to bf16 here, so both sides widen the
identical bf16 values).

Shapes follow the models the paper evaluates (LLaMa-2 7B: 32 layers x 32 heads,
head dim 128; 13B: 40 x 40 x 128; Sec. 5.1).  The value distributions stand in
for the paper's datasets, which are not used here.

Layout of every tensor: unit-major.  A *unit* is one (sequence, layer, head)
triple; ``G`` is layers*heads, so a prompt tensor for one sequence is
``[G][L][d]`` and a decode-token tensor for the whole batch is ``[S][G][d]``.
"""
from __future__ import annotations

import dataclasses
import hashlib
import math
from typing import List, Tuple

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    S: int              # sequences in the batch
    layers: int
    heads: int
    d: int              # head dimension (the paper's d')
    dtype: str          # "f32" or "bf16": storage type of Q/K/V
    prompt_lo: int      # prompt length (lo == hi) or range of ragged lengths
    prompt_hi: int
    B: int              # per-head token budget
    r: int              # eviction-scope parameter
    steps: int          # decode steps after prefill
    kind: str           # "iid" | "sink" | "lowrank" | "burst"
    seed: int = 0

    @property
    def G(self) -> int:
        return self.layers * self.heads

    @property
    def U(self) -> int:
        return self.S * self.G

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


# The five synthetic configurations (one small correctness case, four at the
# paper's model shapes).  "sink": four high-norm keys at positions 0-3 along the
# mean query direction.  "lowrank": a rank-4 component shared by Q and K.
# "burst": every 1024 positions, 8 consecutive tokens share a direction.
TOY = Workload("toy", 1, 1, 4, 64, "f32", 256, 256, 128, 16, 64, "iid", seed=0)
LLAMA7B_DECODE = Workload("llama7b_decode", 8, 32, 32, 128, "bf16", 2048, 2048, 1024, 64, 256, "sink", seed=2)
LLAMA7B_PREFILL = Workload("llama7b_prefill", 1, 32, 32, 128, "bf16", 8192, 8192, 2048, 256, 0, "lowrank", seed=3)
LLAMA13B_SERVING = Workload("llama13b_serving", 64, 40, 40, 128, "bf16", 1024, 4096, 512, 32, 128, "sink", seed=4)
LONG_CONTEXT = Workload("long_context", 4, 32, 32, 128, "bf16", 32768, 32768, 4096, 64, 512, "burst", seed=5)

ALL = {w.name: w for w in (TOY, LLAMA7B_DECODE, LLAMA7B_PREFILL, LLAMA13B_SERVING, LONG_CONTEXT)}


def scaled(w: Workload, **changes) -> Workload:
    """A smaller (or otherwise altered) copy of a workload with the same structure."""
    return dataclasses.replace(w, **changes)


def _seed64(*parts) -> int:
    h = hashlib.blake2b(repr(parts).encode(), digest_size=8).digest()
    return int.from_bytes(h, "little") & ((1 << 63) - 1)


def _gen(device, *parts) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed64(*parts))
    return g


def prompt_lens(w: Workload) -> List[int]:
    """Prompt length of every sequence (ragged when prompt_lo < prompt_hi)."""
    if w.prompt_lo == w.prompt_hi:
        return [w.prompt_lo] * w.S
    g = _gen("cpu", w.seed, "lens")
    return torch.randint(w.prompt_lo, w.prompt_hi + 1, (w.S,), generator=g).tolist()


def unit_directions(w: Workload, b: int, device) -> torch.Tensor:
    """One unit vector per unit of sequence b: [G][d] fp32 (sink / burst direction)."""
    g = _gen(device, w.seed, "dir", b)
    u = torch.randn(w.G, w.d, generator=g, device=device, dtype=torch.float32)
    return u / u.norm(dim=-1, keepdim=True)


def unit_bases(w: Workload, b: int, device) -> torch.Tensor:
    """An orthonormal d x 4 basis per unit of sequence b: [G][d][4] fp32."""
    g = _gen(device, w.seed, "basis", b)
    a = torch.randn(w.G, w.d, 4, generator=g, device=device, dtype=torch.float32)
    qmat, _ = torch.linalg.qr(a.cpu())          # QR on the host: tiny, and identical everywhere
    return qmat.to(device)


def _structure(w: Workload, b: int, g0: int, g1: int, positions: torch.Tensor,
               Q: torch.Tensor, K: torch.Tensor, gen: torch.Generator, device) -> None:
    """Add the workload's structure in place.  Q, K: [g1-g0][T][d] fp32; positions: [T]."""
    d = w.d
    if w.kind == "iid":
        return
    if w.kind == "sink":
        u = unit_directions(w, b, device)[g0:g1]                    # [g][d]
        Q += 2.0 * u[:, None, :]
        sink = positions < 4
        if bool(sink.any()):
            idx = sink.nonzero().flatten()
            noise = torch.randn(g1 - g0, idx.numel(), d, generator=gen, device=device)
            K[:, idx, :] = 3.0 * math.sqrt(d) * u[:, None, :] + 0.1 * noise
        return
    if w.kind == "lowrank":
        basis = unit_bases(w, b, device)[g0:g1]                     # [g][d][4]
        amp = 2.0 * d ** 0.25
        for X in (Q, K):
            a = torch.randn(g1 - g0, X.shape[1], 4, generator=gen, device=device)
            a = a / a.norm(dim=-1, keepdim=True)
            X += amp * torch.einsum("gdk,gtk->gtd", basis, a)
        return
    if w.kind == "burst":
        u = unit_directions(w, b, device)[g0:g1]
        amp = 2.5 * d ** 0.25
        hit = ((positions % 1024) < 8).to(torch.float32)            # [T]
        bump = amp * hit[None, :, None] * u[:, None, :]
        Q += bump
        K += bump
        return
    raise ValueError(f"unknown workload kind {w.kind!r}")


def prompt_chunk(w: Workload, b: int, g0: int, g1: int, L: int, device
                 ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """Q, K, V of the first L prompt tokens of units g0..g1-1 of sequence b: [g1-g0][L][d]."""
    gen = _gen(device, w.seed, "prompt", b, g0, g1, L)
    shape = (g1 - g0, L, w.d)
    Q = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    K = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    V = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    pos = torch.arange(L, device=device)
    _structure(w, b, g0, g1, pos, Q, K, gen, device)
    dt = w.torch_dtype
    return Q.to(dt), K.to(dt), V.to(dt)


def decode_tokens(w: Workload, step: int, t_pos: List[int], device
                  ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """q, k_new, v_new of decode step `step` for the whole batch: [S][G][d].

    t_pos[b] is the absolute position the new token of sequence b gets."""
    qs, ks, vs = [], [], []
    for b in range(w.S):
        gen = _gen(device, w.seed, "decode", b, step)
        shape = (w.G, 1, w.d)
        Q = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        K = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        V = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        pos = torch.tensor([t_pos[b]], device=device)
        _structure(w, b, 0, w.G, pos, Q, K, gen, device)
        qs.append(Q[:, 0]); ks.append(K[:, 0]); vs.append(V[:, 0])
    dt = w.torch_dtype
    return (torch.stack(qs).to(dt), torch.stack(ks).to(dt), torch.stack(vs).to(dt))
