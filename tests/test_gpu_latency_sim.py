"""The CUDA latency simulations against the CPU oracle, trial by trial (same
counter-based random stream on both sides, float64; the only differences are
last-digit roundings of log/cos/exp), plus the closed forms at any size."""

import math

import numpy as np
import pytest

from oracle import latency_oracle as L

pytestmark = pytest.mark.gpu
RTOL = 1e-11


@pytest.fixture(scope="module")
def nolo():
    from paper_2506_10911_b200 import binding
    return binding


@pytest.mark.parametrize("W,mu,sigma,trials,seed", [
    (2, 0.5, 0.8, 50, 3), (4, 0.0, 1.0, 40, 2), (64, 1.0, math.sqrt(0.5), 12, 9), (1024, -0.3, 0.25, 3, 1),
    (4096, 0.0, 0.5, 1, 5),
])
def test_tree_allreduce_trials_match_oracle(nolo, W, mu, sigma, trials, seed):
    mean, se, per = nolo.nolo_sim_tree_allreduce(W, mu, sigma, trials, seed, return_trials=True)
    want = L.sim_tree_allreduce(W, mu, sigma, trials, seed)
    np.testing.assert_allclose(per, want, rtol=RTOL)
    assert mean == pytest.approx(want.mean(), rel=RTOL)
    if trials > 1:
        assert se == pytest.approx(want.std(ddof=1) / math.sqrt(trials), rel=1e-9)


def test_tree_allreduce_closed_forms_at_scale(nolo):
    for W in (2, 32, 1024):
        mean, se = nolo.nolo_sim_tree_allreduce(W, 0.3, 0.0, 100, 1)
        assert mean == pytest.approx(2 * math.exp(0.3) * math.log2(W), rel=1e-13) and se < 1e-12
    mu, sigma = 0.5, 0.8
    mean, se = nolo.nolo_sim_tree_allreduce(2, mu, sigma, 400_000, 7)
    closed = nolo.nolo_expected_pair_exchange(mu, sigma)
    assert closed == pytest.approx(L.expected_pair_exchange(mu, sigma), rel=1e-15)
    assert abs(mean - closed) < 4.5 * se                       # the appendix's E[max] formula
    # Fig. 5a: the advantage over pair exchange grows with W and with the variance
    r = {(W, s): nolo.nolo_sim_tree_allreduce(W, 0.0, s, 20_000, 11)[0] / nolo.nolo_expected_pair_exchange(0.0, s)
         for W in (4, 64, 1024) for s in (0.1, 1.0)}
    assert r[(4, 1.0)] < r[(64, 1.0)] < r[(1024, 1.0)]
    assert r[(1024, 1.0)] > r[(1024, 0.1)] > 0.99 * 10


@pytest.mark.parametrize("W,n,H,T,trials,seed", [
    (4, 2, 3, 2, 5, 11), (16, 4, 10, 6, 4, 2), (8, 8, 5, 7, 3, 4), (1, 1, 4, 3, 2, 0), (100, 5, 7, 4, 2, 6),
    (1024, 2, 100, 4, 1, 0), (2048, 2, 3, 2, 1, 8),
])
def test_straggler_trials_match_oracle(nolo, W, n, H, T, trials, seed):
    mu, sigma = 1.0, math.sqrt(0.5)
    *stats, per = nolo.nolo_sim_straggler(W, n, H, T, mu, sigma, trials, seed, return_trials=True)
    want = L.sim_straggler(W, n, H, T, mu, sigma, trials, seed)
    np.testing.assert_allclose(per, want, rtol=RTOL)
    assert stats[0] == pytest.approx(want[:, 0].mean(), rel=RTOL)
    assert stats[1] == pytest.approx(want[:, 1].mean(), rel=RTOL)
    assert (per[:, 1] <= per[:, 0] * (1 + 1e-15)).all()


def test_straggler_reproduces_the_papers_figure_at_full_size(nolo):
    """W = 1024, pairs, 100 inner steps per outer step, 250 outer iterations,
    LogNormal(1, 0.5): the global barrier costs about 20 % (Section 4.3)."""
    b, s, eb, es = nolo.nolo_sim_straggler(1024, 2, 100, 250, 1.0, math.sqrt(0.5), 8, 0)
    assert 1.14 < b / s < 1.26
    # no variance -> nobody waits
    b, s, _, _ = nolo.nolo_sim_straggler(1024, 2, 100, 5, 1.0, 0.0, 2, 0)
    assert b == pytest.approx(500 * math.e, rel=1e-12) and s == pytest.approx(b, rel=1e-15)


def test_simulation_argument_checks(nolo):
    for bad in [(6, 0.0, 1.0, 10), (1, 0.0, 1.0, 10), (8, 0.0, -1.0, 10), (8, 0.0, 1.0, 0), (8, float("nan"), 1.0, 1)]:
        with pytest.raises(nolo.NoloError) as e:
            nolo.nolo_sim_tree_allreduce(bad[0], bad[1], bad[2], bad[3], 0)
        assert e.value.status == nolo.NOLO_EINVAL
    for bad in [(8, 3, 1, 1), (8, 2, 0, 1), (8, 2, 1, 0), (0, 1, 1, 1)]:
        with pytest.raises(nolo.NoloError) as e:
            nolo.nolo_sim_straggler(*bad, 1.0, 0.5, 1, 0)
        assert e.value.status == nolo.NOLO_EINVAL
