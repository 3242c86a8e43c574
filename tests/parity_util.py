"""Helpers of the GPU parity tests: tensor <-> numpy bridges, guard-banded buffers, tolerances."""
from __future__ import annotations

import numpy as np
import torch

# Tolerances of the contract: float32 gradients rtol 1e-6 / atol 1e-7; bfloat16 gradient inputs
# rtol 1e-2 (the kernel and the oracle widen bfloat16 exactly, so far tighter bounds hold, and the
# tests also report bit equality).
TOL = {"f32": dict(rtol=1e-6, atol=1e-7), "bf16": dict(rtol=1e-2, atol=1e-7)}
SQNORM_RTOL = 1e-5
GUARD = 64  # elements of guard band on each side of every test buffer


def to_np(t: torch.Tensor) -> np.ndarray:
    """Device tensor -> host numpy array with the same bits (bfloat16 as uint16)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    return t.numpy().copy()


class Guarded:
    """A device buffer with poisoned guard bands in front and behind; ``t`` is the usable part
    (16-byte aligned because GUARD elements are a multiple of 16 bytes)."""

    def __init__(self, n: int, dtype, device, fill=None):
        self.dtype = dtype
        self.raw = torch.empty(n + 2 * GUARD, dtype=dtype, device=device)
        self.poison = 12345.0 if dtype != torch.bfloat16 else 123.0
        self.raw.fill_(self.poison)
        self.t = self.raw[GUARD:GUARD + n]
        if fill is not None:
            self.t.copy_(fill)
        assert self.t.data_ptr() % 16 == 0

    def intact(self) -> bool:
        a = self.raw[:GUARD].float().cpu()
        b = self.raw[GUARD + self.t.numel():].float().cpu()
        return bool((a == self.poison).all() and (b == self.poison).all())


def assert_close(got: np.ndarray, want: np.ndarray, kind: str, what: str = "") -> float:
    """Element-wise comparison at the contract tolerance; returns the fraction of bit-equal elements."""
    np.testing.assert_allclose(got, want, err_msg=what, **TOL[kind])
    return float((got.view(np.uint32) == want.view(np.uint32)).mean()) if got.size else 1.0
