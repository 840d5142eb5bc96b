"""Are the pins sharp?  Each plausible mistake is planted in the oracle (on the
CPU, by wrapping ``outer_step`` so that it computes what the mistaken code
would) and the pin tests are re-run against it: every mutant must make at
least one pin fail, and the unmutated oracle must pass them all."""

import numpy as np
import pytest

from oracle import nolo_oracle as O
from tests import test_oracle_pins as pins

TRUE = O.outer_step

PINS = [
    pins.test_hand_computed_w2_p4,
    pins.test_diloco_reduction_full_group,
    pins.test_sign_pin_local_sgd_average,
    pins.test_group_mean_identity_and_preservation,
    pins.test_spread_identity,
    pins.test_n1_is_lookahead_momentum,
    pins.test_gossip_corner,
    pins.test_fixed_point_and_theta_reset,
    pins.test_relabelling_workers_relabels_outputs,
    pins.test_bf16_theta_in_and_out,
    pins.test_noise_free_quadratic_follows_appendix_d_recursion,
]


def widen(theta, dt):
    return O.bf16_bits_to_f32(theta) if dt == O.THETA_BF16 else theta


def m_wrong_sign(phi, theta, delta, perm, n, a, b, c, dt=O.THETA_F32):
    """Delta = theta - phi (Eq. 1 as printed) fed into Eq. 2 as printed."""
    t = (2.0 * phi.astype(np.float64) - widen(theta, dt)).astype(np.float32)
    p, d, th = TRUE(phi, t, delta, perm, n, a, b, c)
    return p, d, (O.f32_to_bf16_bits(p) if dt == O.THETA_BF16 else th)


def m_no_pull(phi, theta, delta, perm, n, a, b, c, dt=O.THETA_F32):
    return TRUE(phi, theta, delta, perm, n, a, b, 0.0, dt)


def m_no_momentum(phi, theta, delta, perm, n, a, b, c, dt=O.THETA_F32):
    return TRUE(phi, theta, delta, perm, n, 0.0, b, c, dt)


def m_sum_not_mean(phi, theta, delta, perm, n, a, b, c, dt=O.THETA_F32):
    """beta * sum(Delta) instead of (beta / n) * sum(Delta)."""
    return TRUE(phi, theta, delta, perm, n, a, b * n, c, dt)


def m_mean_of_others(phi, theta, delta, perm, n, a, b, c, dt=O.THETA_F32):
    """phi_i minus the mean of the other members: (n/(n-1)) (phi_i - mean of all)."""
    return TRUE(phi, theta, delta, perm, n, a, b, c * n / (n - 1) if n > 1 else c, dt)


def m_pull_sign(phi, theta, delta, perm, n, a, b, c, dt=O.THETA_F32):
    return TRUE(phi, theta, delta, perm, n, a, b, -c, dt)


def m_stale_momentum(phi, theta, delta, perm, n, a, b, c, dt=O.THETA_F32):
    """Returns the old momentum instead of the new one."""
    p, d, t = TRUE(phi, theta, delta, perm, n, a, b, c, dt)
    return p, delta.copy(), t


def m_no_theta_reset(phi, theta, delta, perm, n, a, b, c, dt=O.THETA_F32):
    p, d, t = TRUE(phi, theta, delta, perm, n, a, b, c, dt)
    return p, d, theta.copy()


def m_shifted_groups(phi, theta, delta, perm, n, a, b, c, dt=O.THETA_F32):
    """Groups cut one position late: perm[1:n+1], ... (wraps around)."""
    return TRUE(phi, theta, delta, np.roll(perm, -1), n, a, b, c, dt)


def m_own_delta_only(phi, theta, delta, perm, n, a, b, c, dt=O.THETA_F32):
    """Uses the worker's own outer gradient instead of the subgroup mean."""
    W = phi.shape[0]
    p1, d1, t1 = TRUE(phi, theta, delta, np.arange(W, dtype=np.int32), 1, a, b, 0.0, dt)
    p0, d0, _ = TRUE(phi, theta, delta, perm, n, a, 0.0, c, dt)          # momentum + pull only
    pz, dz, _ = TRUE(phi, theta, delta, perm, n, a, 0.0, 0.0, dt)        # momentum only
    d = (d1.astype(np.float64) + d0 - dz).astype(np.float32)
    p = (phi.astype(np.float64) + d).astype(np.float32)
    return p, d, (O.f32_to_bf16_bits(p) if dt == O.THETA_BF16 else p.copy())


def m_bf16_truncates(phi, theta, delta, perm, n, a, b, c, dt=O.THETA_F32):
    """bfloat16 theta by truncation instead of round-to-nearest-even."""
    p, d, t = TRUE(phi, theta, delta, perm, n, a, b, c, dt)
    if dt == O.THETA_BF16:
        t = (p.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    return p, d, t


MUTANTS = [m_wrong_sign, m_no_pull, m_no_momentum, m_sum_not_mean, m_mean_of_others, m_pull_sign,
           m_stale_momentum, m_no_theta_reset, m_shifted_groups, m_own_delta_only, m_bf16_truncates]


def failing_pins(monkeypatch, fn):
    monkeypatch.setattr(O, "outer_step", fn)
    failed = []
    for pin in PINS:
        try:
            pin()
        except AssertionError:
            failed.append(pin.__name__)
    monkeypatch.setattr(O, "outer_step", TRUE)
    return failed


def test_unmutated_oracle_passes_every_pin(monkeypatch):
    assert failing_pins(monkeypatch, TRUE) == []


@pytest.mark.parametrize("mutant", MUTANTS, ids=lambda f: f.__name__)
def test_every_planted_mistake_is_caught(monkeypatch, mutant):
    assert failing_pins(monkeypatch, mutant), f"no pin notices {mutant.__name__}"
