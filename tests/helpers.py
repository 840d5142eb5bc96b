"""Shared test helpers: tolerance checks and tensor <-> numpy conversion."""

import numpy as np
import torch

# float32 outputs: |gpu - oracle| <= ATOL + RTOL * |oracle| per element.
RTOL = 2e-6
ATOL = 1e-7


def to_np(t: torch.Tensor) -> np.ndarray:
    """CPU numpy view; bfloat16 comes back as uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def assert_close_f32(got: np.ndarray, want: np.ndarray, what: str):
    got = got.astype(np.float64)
    want = want.astype(np.float64)
    err = np.abs(got - want)
    lim = ATOL + RTOL * np.abs(want)
    bad = ~(err <= lim)
    bad &= ~(np.isnan(got) & np.isnan(want))
    if bad.any():
        i = np.argwhere(bad)[0]
        raise AssertionError(
            f"{what}: {bad.sum()} of {bad.size} elements out of tolerance; first at {tuple(i)}: "
            f"got {got[tuple(i)]!r} want {want[tuple(i)]!r}; max err {np.nanmax(err):.3e}")


def bf16_ordered(bits: np.ndarray) -> np.ndarray:
    """Map bfloat16 bit patterns to integers whose order is the numeric order."""
    b = bits.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def assert_bf16_within_1ulp(got_bits: np.ndarray, want_bits: np.ndarray, what: str):
    """bfloat16 theta: at most 1 ulp apart.  Next to zero a bfloat16 ulp is far smaller than
    the float32 absolute tolerance on phi' (of which theta is the rounding), so there the
    float32 bound ATOL + RTOL*|x| applies instead."""
    d = np.abs(bf16_ordered(got_bits) - bf16_ordered(want_bits))
    if (d > 1).any():
        g, w = bf16_to_f64(got_bits), bf16_to_f64(want_bits)
        d = np.where(np.abs(g - w) <= 1.01 * ATOL + RTOL * np.abs(w), 0, d)
    if (d > 1).any():
        i = np.argwhere(d > 1)[0]
        raise AssertionError(f"{what}: {int((d > 1).sum())} elements differ by more than 1 bf16 ulp; "
                             f"first at {tuple(i)}: {got_bits[tuple(i)]:#06x} vs {want_bits[tuple(i)]:#06x}")
    return int((d == 1).sum())
