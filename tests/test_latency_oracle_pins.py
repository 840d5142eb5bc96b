"""Pins of the latency-simulation oracle: library generators, closed forms
(constant message time, the appendix's E[max] formula), exact special cases and
the paper's ~20 % straggler figure."""

import math

import numpy as np
import pytest
from scipy import stats

from oracle import latency_oracle as L
from oracle import nolo_oracle as O


def test_vectorised_philox_matches_scalar_and_numpy():
    rng = np.random.default_rng(0)
    c = rng.integers(0, 2**64, (4, 50), dtype=np.uint64)
    k0, k1 = 0xDEADBEEFCAFEF00D, 2**64 - 3
    got = L.philox4x64_10_np(c[0], c[1], c[2], c[3], k0, k1)
    for i in range(50):
        want = O.philox4x64_10([int(c[j, i]) for j in range(4)], (k0, k1))
        assert tuple(int(g[i]) for g in got) == want
    # broadcasting of scalar counters
    g2 = L.philox4x64_10_np(np.arange(5, dtype=np.uint64), 7, 8, 9, 1, 2)
    assert int(g2[0][3]) == O.philox4x64_10((3, 7, 8, 9), (1, 2))[0]
    # numpy's generator (bumps the counter once before the first block)
    bg = np.random.Philox(counter=np.array([4, 7, 8, 9], dtype=np.uint64), key=np.array([1, 2], dtype=np.uint64))
    assert [int(x) for x in bg.random_raw(4)] == [int(g[5 - 5 + 0]) for g in
                                                  L.philox4x64_10_np(np.array([5], dtype=np.uint64), 7, 8, 9, 1, 2)]


def test_uniform_and_normal_transforms():
    assert L.uniform_open(np.array([0], dtype=np.uint64))[0] == 2.0 ** -54
    assert L.uniform_open(np.array([2**64 - 1], dtype=np.uint64))[0] == 1.0 - 2.0 ** -54
    w0, w1, _, _ = L.philox4x64_10_np(np.arange(200_000, dtype=np.uint64), 0, 0, 9, 5, 6)
    u = L.uniform_open(w0)
    assert stats.kstest(u, "uniform").pvalue > 1e-3
    w = L.philox4x64_10_np(np.arange(200_000, dtype=np.uint64), 0, 0, 9, 5, 6)
    t = L.lognormal4_from_block(*w, 1.0, math.sqrt(0.5))               # [200000, 4]
    z = (np.log(t) - 1.0) / math.sqrt(0.5)
    for lane in range(4):                                              # cos and sin halves of both word pairs
        assert stats.kstest(z[:, lane], "norm").pvalue > 1e-3
    assert stats.kstest(z.ravel(), "norm").pvalue > 1e-3
    # the four normals of a block are uncorrelated (Box-Muller's two outputs are independent)
    assert np.abs(np.corrcoef(z.T) - np.eye(4)).max() < 0.01
    assert abs(t.mean() - math.exp(1.25)) < 4 * t.std() / math.sqrt(t.size)


def scalar_sample(j, c1, c2, domain, mu, sigma, k0, k1):
    """Sample j of a stream, recomputed with the scalar Philox and the math module: block j // 4,
    word pair (j % 4) // 2, cosine for even j and sine for odd j."""
    words = O.philox4x64_10((j // 4, c1, c2, domain), (k0, k1))
    u = [((x >> 11) + 0.5) * 2.0 ** -53 for x in words]
    a, b = (u[0], u[1]) if (j % 4) < 2 else (u[2], u[3])
    r = math.sqrt(-2.0 * math.log(a))
    z = r * (math.cos(2.0 * math.pi * b) if j % 2 == 0 else math.sin(2.0 * math.pi * b))
    return math.exp(mu + sigma * z)


def test_stream_layout_against_scalar_recomputation():
    mu, sigma = 0.3, 0.9
    got = L.stream_times(11, np.arange(3), 6, L.DOMAIN_STRAGGLER, mu, sigma, 21, 4)       # [3 workers, 11 steps]
    assert got.shape == (3, 11)
    for w in range(3):
        for j in range(11):
            assert got[w, j] == pytest.approx(scalar_sample(j, w, 6, L.DOMAIN_STRAGGLER, mu, sigma, 21, 4), rel=1e-14)
    up = L.message_times(8, 3, 0, mu, sigma, 5)
    assert up.shape == (16,)
    for node in range(2, 16):
        assert up[node] == pytest.approx(scalar_sample(node, 3, 0, L.DOMAIN_TREE, mu, sigma, 5, 0), rel=1e-14)


def test_pair_exchange_closed_form_against_independent_sampling():
    rng = np.random.default_rng(1)
    for mu, sigma in [(0.0, 0.3), (1.0, math.sqrt(0.5)), (-1.0, 1.2)]:
        t = rng.lognormal(mu, sigma, (2_000_000, 2)).max(axis=1)       # numpy's own log-normal
        want = L.expected_pair_exchange(mu, sigma) / 2
        assert abs(t.mean() - want) < 5 * t.std() / math.sqrt(t.shape[0])
    assert L.expected_pair_exchange(0.7, 0.0) == pytest.approx(2 * math.exp(0.7))


def test_tree_with_constant_message_time_is_2_tc_log2_W():
    for W in (2, 4, 32, 256):
        got = L.sim_tree_allreduce(W, 0.3, 0.0, 3, seed=1)
        np.testing.assert_allclose(got, 2 * math.exp(0.3) * math.log2(W), rtol=1e-13)


def test_tree_of_two_is_the_pair_exchange():
    mu, sigma = 0.5, 0.8
    got = L.sim_tree_allreduce(2, mu, sigma, 4_000, seed=3)
    assert abs(got.mean() - L.expected_pair_exchange(mu, sigma)) < 4 * got.std() / math.sqrt(got.size)
    # by hand for one trial: max(t_up(2), t_up(3)) + max(t_down(2), t_down(3))
    up = L.message_times(2, 0, 0, mu, sigma, 3)
    down = L.message_times(2, 0, 1, mu, sigma, 3)
    assert got[0] == max(up[2], up[3]) + max(down[2], down[3])


def test_tree_by_hand_W4():
    mu, sigma = 0.0, 1.0
    up = L.message_times(4, 5, 0, mu, sigma, 2)
    dn = L.message_times(4, 5, 1, mu, sigma, 2)
    r2 = max(up[4], up[5]); r3 = max(up[6], up[7])
    r1 = max(r2 + up[2], r3 + up[3])
    leaves = [r1 + dn[2] + dn[4], r1 + dn[2] + dn[5], r1 + dn[3] + dn[6], r1 + dn[3] + dn[7]]
    assert L.sim_tree_allreduce(4, mu, sigma, 6, seed=2)[5] == pytest.approx(max(leaves), rel=1e-15)


def test_speedup_grows_with_world_size_and_variance():
    def ratio(W, sigma):
        return L.sim_tree_allreduce(W, 0.0, sigma, 1500, seed=7).mean() / L.expected_pair_exchange(0.0, sigma)
    assert ratio(4, 0.5) < ratio(16, 0.5) < ratio(64, 0.5)
    assert ratio(64, 1.0) > ratio(64, 0.1) > 0.99 * math.log2(64)
    with pytest.raises(ValueError):
        L.sim_tree_allreduce(6, 0.0, 1.0, 1, 0)


def test_straggler_exact_cases():
    # one subgroup of everybody is the global barrier
    a = L.sim_straggler(8, 8, 5, 7, 1.0, 0.7, 3, seed=4)
    np.testing.assert_allclose(a[:, 0], a[:, 1], rtol=1e-15)
    # constant step time: nobody ever waits
    b = L.sim_straggler(8, 2, 5, 7, 1.0, 0.0, 2, seed=4)
    np.testing.assert_allclose(b, 7 * 5 * math.e, rtol=1e-13)
    # waiting for fewer peers can only be faster; a lone worker never waits
    c = L.sim_straggler(16, 2, 10, 20, 1.0, 0.7, 4, seed=5)
    assert (c[:, 1] <= c[:, 0]).all() and (c[:, 1] < c[:, 0]).any()
    d = L.sim_straggler(1, 1, 10, 20, 1.0, 0.7, 2, seed=5)
    np.testing.assert_allclose(d[:, 0], d[:, 1], rtol=1e-15)


def test_straggler_by_hand_two_steps():
    W, n, H, T, mu, sg, seed = 4, 2, 6, 2, 1.0, 0.5, 11
    work = []
    for t in range(T):
        per_worker = []
        for w in range(W):
            total = 0.0
            for k in range(H):                                 # inner steps in order, scalar arithmetic
                total += scalar_sample(k, w, t, L.DOMAIN_STRAGGLER, mu, sg, seed, 0)
            per_worker.append(total)
        work.append(np.array(per_worker))
    barrier = work[0].max() + work[1].max()
    clock = np.zeros(W)
    for t in range(T):
        perm = O.draw_perm(seed, t, O.DOMAIN_GROUPS, 0, 0, W)
        done = clock + work[t]
        for g in range(2):
            i, j = perm[2 * g], perm[2 * g + 1]
            clock[i] = clock[j] = max(done[i], done[j])
    got = L.sim_straggler(W, n, H, T, mu, sg, 1, seed)[0]
    assert got[0] == pytest.approx(barrier, rel=1e-13) and got[1] == pytest.approx(clock.max(), rel=1e-13)


def test_straggler_reproduces_the_papers_20_percent_at_1024():
    """Section 4.3: with inner-step latency LogNormal(1, 0.5), 100 inner steps per
    outer step and pairs, the global barrier costs about 20 % at 1024 workers."""
    r = L.sim_straggler(1024, 2, 100, 60, 1.0, math.sqrt(0.5), 1, seed=0)[0]
    assert 1.12 < r[0] / r[1] < 1.30
