"""Views and exact widenings of the unit-major tensors (no arithmetic of the method)."""
from __future__ import annotations

from typing import Sequence

import numpy as np
import torch


def unit_view(t: torch.Tensor, units: Sequence[int]) -> torch.Tensor:
    """Rows of a [S][G][...] tensor for flat unit indices."""
    flat = t.reshape((-1,) + tuple(t.shape[2:]))
    return flat[torch.as_tensor(list(units), device=t.device)]


def widen(t: torch.Tensor) -> np.ndarray:
    """Exact widening of device fp32/bf16 values to float64 on the host."""
    return t.detach().to("cpu").to(torch.float64).numpy()
