"""The two independent writings of the oracle -- NumPy (vectorised over parameters, one
subgroup at a time) and plain C (one parameter at a time) -- must agree before either judges
the CUDA library: integers and routed bytes exactly, float64 results to 1e-12 relative.

Outputs that are rounded to float32 can differ where the two float64 results straddle a
rounding boundary of float32 (they differ by a few 1e-16 relative, so this happens to about one
element in 1e8); such an element may be one float32 ulp apart and is counted."""

import numpy as np
import pytest

from oracle import c_oracle as C
from oracle import nolo_oracle as O

RTOL = 1e-12


def state(W, P, seed, bf16, scale=0.02):
    rng = np.random.default_rng(seed)
    phi = (scale * rng.standard_normal((W, P)) + rng.choice([0.0, 1.0, -3.0], size=(1, P))).astype(np.float32)
    theta = (phi + 1e-3 * rng.standard_normal((W, P))).astype(np.float32)
    delta = (1e-4 * rng.standard_normal((W, P))).astype(np.float32)
    if bf16:
        theta = O.f32_to_bf16_bits(theta)
    return phi, theta, delta


def assert_same_f32(a, b, what):
    assert a.dtype == b.dtype == np.float32 and a.shape == b.shape
    a64, b64 = a.astype(np.float64), b.astype(np.float64)
    off = np.abs(a64 - b64) > RTOL * np.abs(b64)
    if off.any():
        one_ulp = np.abs(a64 - b64) <= np.spacing(np.abs(b).astype(np.float32)).astype(np.float64)
        assert (off <= one_ulp).all(), f"{what}: more than a rounding flip apart"
        assert off.sum() <= max(1, a.size // 1_000_000), f"{what}: {off.sum()} rounding flips in {a.size}"


def test_philox_blocks_agree():
    rng = np.random.default_rng(1)
    cases = [((0, 0, 0, 0), (0, 0)), ((2**64 - 1,) * 4, (2**64 - 1,) * 2), ((1, 2, 3, 4), (5, 6))]
    cases += [(tuple(int(x) for x in rng.integers(0, 2**64, 4, dtype=np.uint64)),
               tuple(int(x) for x in rng.integers(0, 2**64, 2, dtype=np.uint64))) for _ in range(200)]
    for ctr, key in cases:
        assert C.philox4x64_10(ctr, key) == O.philox4x64_10(ctr, key)


@pytest.mark.parametrize("N", [1, 2, 3, 8, 16, 127, 128, 1000])
def test_permutations_agree(N):
    for seed, step, domain, b, k in [(0, 0, 1, 0, 0), (7, 3, 2, 1, 2), (2**64 - 1, 2**63, 2, 5, 0), (123456789, 42, 1, 0, 0)]:
        got = C.draw_perm(seed, step, domain, b, k, N)
        assert got.dtype == np.int32
        assert np.array_equal(got, O.draw_perm(seed, step, domain, b, k, N))


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("W,n", [(2, 2), (4, 2), (8, 4), (16, 1), (24, 8), (96, 96), (130, 65)])
def test_outer_step_agrees(W, n, bf16):
    P = 4099
    phi, theta, delta = state(W, P, 100 * W + n, bf16)
    perm = O.draw_groups(W, n, W, n)
    dt = O.THETA_BF16 if bf16 else O.THETA_F32
    for hp in [(0.5, 0.7, 0.5), (0.0, 1.0, 0.0), (0.9, 0.3, 1.0)]:
        want = O.outer_step(phi, theta, delta, perm, n, *hp, dt)
        got = C.outer_step(phi, theta, delta, perm, n, *hp, dt)
        assert_same_f32(got[0], want[0], "phi")
        assert_same_f32(got[1], want[1], "delta")
        if bf16:
            # bfloat16 theta' is a rounding of the float32 phi': equal wherever phi' is
            same_phi = got[0] == want[0]
            assert np.array_equal(got[2][same_phi], want[2][same_phi])
        else:
            assert np.array_equal(got[2], got[0]) and np.array_equal(want[2], want[0])


def test_outer_step_on_a_column_slice_and_hand_case():
    # column slices of larger arrays (rows not contiguous) give the same as copies of them
    phi, theta, delta = state(8, 1000, 5, True)
    perm = O.draw_groups(1, 2, 8, 4)
    a = C.outer_step(phi[:, 100:700], theta[:, 100:700], delta[:, 100:700], perm, 4, 0.5, 0.7, 0.5, O.THETA_BF16)
    b = O.outer_step(phi[:, 100:700], theta[:, 100:700], delta[:, 100:700], perm, 4, 0.5, 0.7, 0.5, O.THETA_BF16)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
    # the hand-computed pair of the paper's Eq. 2-3 (exact rationals; values in tests/golden)
    phi = np.array([[1, 2, -1, 0], [3, 2, 1, 0.5]], dtype=np.float32)
    theta = np.array([[0.5, 2, -1.5, 0.25], [2, 1, 1, 0.5]], dtype=np.float32)
    delta = np.array([[0.2, 0, -0.4, 0], [0, 0.2, 0.4, -0.2]], dtype=np.float32)
    p, d, t = C.outer_step(phi, theta, delta, np.array([0, 1], dtype=np.int32), 2, 0.5, 0.7, 0.5)
    np.testing.assert_allclose(d, [[0.075, -0.35, 0.125, 0.2125], [-1.025, -0.25, -0.475, -0.1375]], rtol=3e-7)
    np.testing.assert_allclose(p, [[1.075, 1.65, -0.875, 0.2125], [1.975, 1.75, 0.525, 0.3625]], rtol=3e-7)
    assert np.array_equal(p, t)


def test_bf16_rounding_agrees_on_every_pattern_class():
    # theta' = RNE(phi') through the C path against the NumPy helper, on ties, denormals, Inf, NaN
    vals = np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, -1e-40, np.inf, -np.inf, np.nan,
                     0.1, -0.1, 65504.0, 2.0 ** -126, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8], dtype=np.float32)
    rng = np.random.default_rng(3)
    bits = rng.integers(0, 2**32, 100_000, dtype=np.uint64).astype(np.uint32)
    vals = np.concatenate([vals, bits.view(np.float32)])
    phi = vals.reshape(1, -1)
    zeros = np.zeros_like(phi)
    # n = 1, alpha = beta = gamma = 0: phi' = phi for finite phi (-0 becomes +0, Inf - Inf gives NaN),
    # and theta' must be the NumPy helper's rounding of whatever float32 phi' came out
    p, d, t = C.outer_step(phi, O.f32_to_bf16_bits(zeros), zeros, np.array([0], dtype=np.int32), 1, 0.0, 0.0, 0.0,
                           O.THETA_BF16)
    finite = np.isfinite(phi)
    assert np.array_equal(p[finite], phi[finite])
    want = O.f32_to_bf16_bits(p)
    nan = np.isnan(p)
    assert nan.sum() >= 3 and (~nan).sum() > 90_000
    assert np.array_equal(t[~nan], want[~nan])
    assert (np.isnan(O.bf16_bits_to_f32(t[nan]))).all()


def test_subgroup_means_divergence_and_routing_agree():
    phi, _, _ = state(12, 3001, 9, False)
    perm = O.draw_groups(3, 4, 12, 3)
    np.testing.assert_allclose(C.subgroup_mean_phi(phi, perm, 3), O.subgroup_mean_phi(phi, perm, 3), rtol=RTOL, atol=0)
    np.testing.assert_allclose(C.divergence(phi), O.divergence(phi), rtol=1e-11)
    rng = np.random.default_rng(4)
    for per_mb in (False, True):
        table = O.draw_route(5, 6, 4, 6, 3, per_mb)
        acts = rng.integers(0, 2**16, (3, 6, 3, 37), dtype=np.uint16)
        fwd = C.route_forward(acts, table)
        assert np.array_equal(fwd, O.route_forward(acts, table))
        assert np.array_equal(C.route_backward(fwd, table), O.route_backward(fwd, table))
        assert np.array_equal(C.route_backward(fwd, table), acts)


def test_thread_count_changes_nothing():
    phi, theta, delta = state(8, 50_001, 11, False)
    perm = O.draw_groups(0, 0, 8, 2)
    before = C.threads()
    try:
        C.set_threads(1)
        a = C.outer_step(phi, theta, delta, perm, 2, 0.5, 0.7, 0.5)
        C.set_threads(4)
        b = C.outer_step(phi, theta, delta, perm, 2, 0.5, 0.7, 0.5)
    finally:
        C.set_threads(before)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
