"""Helpers shared by the GPU parity tests: tolerance rule, guard-banded outputs, host copies."""
from __future__ import annotations

import numpy as np
import torch

# Tolerances of the comparison against the float64 oracle, by data dtype of the call:
# pass iff |got - ref| <= tol * max(1, |ref|) for every element (absolute below 1, relative above).
# fp16 data (a widening step beyond the benchmark dtypes): the final RNE store alone is 2^-11 = 4.9e-4 relative
# and the hardware tanh / ex2 approximations add up to about as much, so 2e-3 leaves a factor of two to four.
TOL = {torch.float32: 1e-5, torch.bfloat16: 2e-2, torch.float16: 2e-3}
SENTINEL = 0x5A


def tol_of(dtype) -> float:
    return TOL[dtype]


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def assert_close(got: torch.Tensor, ref: np.ndarray, tol: float, what: str):
    g = to_f64(got)
    assert g.shape == ref.shape, f"{what}: shape {g.shape} vs {ref.shape}"
    both_nan = np.isnan(g) & np.isnan(ref)
    err = np.abs(g - ref)
    bound = tol * np.maximum(1.0, np.abs(ref))
    bad = ~((err <= bound) | both_nan)
    if bad.any():
        i = np.unravel_index(np.argmax(np.where(bad, err, 0)), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside tol={tol:g}; worst at {i}: "
                             f"got {g[i]!r} ref {ref[i]!r} err {err[i]:.3e}")
    return float(np.nanmax(err)) if err.size and not np.isnan(err).all() else 0.0


def assert_bf16_tight(got: torch.Tensor, ref: np.ndarray, what: str, rel=2.0 ** -7, floor=4e-3):
    """A much tighter sanity bound for bf16 outputs than the 2e-2 gate: the result must sit
    within about two bf16 steps of the float64 value (plus a small absolute floor for the
    hardware-approximation error near zero)."""
    g = to_f64(got)
    err = np.abs(g - ref)
    bound = rel * np.abs(ref) + floor
    ok = (err <= bound) | (np.isnan(g) & np.isnan(ref))
    assert ok.all(), f"{what}: {(~ok).sum()} elements beyond the tight bf16 bound, max err {np.nanmax(err):.3e}"


class Guarded:
    """An output tensor carved out of a larger byte buffer whose pads are filled with a sentinel;
    `check()` verifies that the kernel wrote nothing outside the tensor."""

    PAD = 512

    def __init__(self, shape, dtype, device="cuda"):
        n = int(np.prod(shape)) if len(shape) else 1
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        self.buf = torch.full((nbytes + 2 * self.PAD,), SENTINEL, dtype=torch.uint8, device=device)
        self.nbytes = nbytes
        self.t = self.buf[self.PAD:self.PAD + nbytes].view(dtype).view(shape)

    def check(self, what=""):
        lo = self.buf[:self.PAD]
        hi = self.buf[self.PAD + self.nbytes:]
        assert bool((lo == SENTINEL).all()) and bool((hi == SENTINEL).all()), f"{what}: wrote outside the output"
