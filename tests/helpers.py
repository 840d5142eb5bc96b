"""Shared test helpers: tolerance checks and tensor <-> numpy conversion."""

import numpy as np
import torch

# float32 outputs: |gpu - oracle| <= ATOL + RTOL * |oracle| per element.
RTOL = 2e-6
ATOL = 1e-7
# One float32 unit in the last place, relative.  phi' = phi + delta' is formed from the stored
# float32 delta', so wherever phi and delta' cancel, phi' (and theta', its copy) inherits the
# rounding of delta': up to half an ulp of delta' from its own rounding plus as much from the
# fused multiply-adds before it.  The comparisons of phi' and theta' therefore allow
# ULP32 * |delta'| on top of the bound above (pass the oracle's delta' as `carried`).  For weights
# of ordinary size |delta'| << |phi'| and the allowance vanishes (1e-10 at |delta'| = 1e-3); it is
# the same for every kernel.
ULP32 = 2.0 ** -23


def to_np(t: torch.Tensor) -> np.ndarray:
    """CPU numpy view; bfloat16 comes back as uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def f32_limit(want: np.ndarray, carried=None) -> np.ndarray:
    lim = ATOL + RTOL * np.abs(want.astype(np.float64))
    if carried is not None:
        lim = lim + ULP32 * np.abs(np.asarray(carried, dtype=np.float64))
    return lim


def assert_close_f32(got: np.ndarray, want: np.ndarray, what: str, carried=None):
    got = got.astype(np.float64)
    want = want.astype(np.float64)
    err = np.abs(got - want)
    bad = ~(err <= f32_limit(want, carried))
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


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    """Spacing of bfloat16 (8 significand bits) at |x|; the subnormal spacing near zero."""
    _, e = np.frexp(np.abs(x))
    return np.ldexp(1.0, np.maximum(e - 8, -133))


def assert_bf16_within_1ulp(got_bits: np.ndarray, want_bits: np.ndarray, what: str, carried=None):
    """bfloat16 theta' = RNE(phi'): at most 1 bfloat16 ulp from the oracle's.  Where a bfloat16 ulp
    is smaller than the float32 tolerance T of the phi' it is rounded from (next to zero), two
    roundings of values at most T apart can be T plus one ulp apart, so that is the bound there."""
    d = np.abs(bf16_ordered(got_bits) - bf16_ordered(want_bits))
    if (d > 1).any():
        g, w = bf16_to_f64(got_bits), bf16_to_f64(want_bits)
        bound = f32_limit(w, carried) + bf16_ulp(np.maximum(np.abs(g), np.abs(w)))
        d = np.where(np.abs(g - w) <= bound, 0, d)
    if (d > 1).any():
        i = np.argwhere(d > 1)[0]
        raise AssertionError(f"{what}: {int((d > 1).sum())} elements differ by more than 1 bf16 ulp; "
                             f"first at {tuple(i)}: {got_bits[tuple(i)]:#06x} vs {want_bits[tuple(i)]:#06x}")
    return int((d == 1).sum())


def assert_outer_step_parity(got_phi, got_delta, got_theta, want, bf16: bool, what: str = ""):
    """phi', delta', theta' of the CUDA path against the oracle's (phi', delta', theta')."""
    assert_close_f32(got_delta, want[1], f"{what}delta")
    assert_close_f32(got_phi, want[0], f"{what}phi", carried=want[1])
    if bf16:
        assert_bf16_within_1ulp(got_theta, want[2], f"{what}theta(bf16)", carried=want[1])
    else:
        assert_close_f32(got_theta, want[2], f"{what}theta", carried=want[1])
