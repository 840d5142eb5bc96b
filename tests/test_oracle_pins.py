"""Pins of the CPU oracle against things other than itself: numpy's Philox,
torch's bfloat16 rounding, a hand-computed case, the paper's special cases and
identities of Eq. 1-3, and the convergence recursion of Appendix D."""

import os

import numpy as np
import pytest
import torch

from oracle import nolo_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
F32 = np.float32


def rnd_state(W, P, seed, phi_std=0.02, drift=1e-3, dstd=1e-4):
    rng = np.random.default_rng(seed)
    phi = rng.normal(0, phi_std, (W, P)).astype(F32)
    theta = (phi + rng.normal(0, drift, (W, P))).astype(F32)
    delta = rng.normal(0, dstd, (W, P)).astype(F32)
    return phi, theta, delta


# ---------------------------------------------------------------- generator

def test_philox_matches_numpy_library():
    """numpy.random.Philox is an independent Philox-4x64-10; it bumps the
    256-bit counter once before producing its first block."""
    rng = np.random.default_rng(7)
    cases = [((0, 0, 0, 0), (0, 0)), ((2**64 - 2, 2**64 - 1, 3, 4), (2**64 - 1, 12345))]
    for _ in range(20):
        c = tuple(int(x) for x in rng.integers(0, 2**64, 4, dtype=np.uint64))
        k = tuple(int(x) for x in rng.integers(0, 2**64, 2, dtype=np.uint64))
        cases.append((c, k))
    for ctr, key in cases:
        bg = np.random.Philox(counter=np.array(ctr, dtype=np.uint64),
                              key=np.array(key, dtype=np.uint64))
        raw = [int(x) for x in bg.random_raw(4)]
        big = (sum(v << (64 * i) for i, v in enumerate(ctr)) + 1) % (1 << 256)
        bumped = [(big >> (64 * i)) & O.MASK64 for i in range(4)]
        assert list(O.philox4x64_10(bumped, key)) == raw


def test_draw_perm_is_stable_sort_of_keys():
    for N in (1, 2, 5, 16, 128):
        keys = np.array(O.draw_keys(3, 9, O.DOMAIN_GROUPS, 0, 0, N), dtype=np.uint64)
        perm = O.draw_perm(3, 9, O.DOMAIN_GROUPS, 0, 0, N)
        assert perm.dtype == np.int32
        assert sorted(perm.tolist()) == list(range(N))           # bijection
        assert np.array_equal(perm, np.argsort(keys, kind="stable"))


def test_draw_perm_tie_break_by_index(monkeypatch):
    monkeypatch.setattr(O, "draw_keys", lambda *a: [5, 1, 5, 1, 0])
    assert O.draw_perm(0, 0, 1, 0, 0, 5).tolist() == [4, 1, 3, 0, 2]


def test_draw_is_deterministic_and_separated():
    a = O.draw_perm(1, 2, O.DOMAIN_GROUPS, 0, 0, 64)
    assert np.array_equal(a, O.draw_perm(1, 2, O.DOMAIN_GROUPS, 0, 0, 64))
    others = [O.draw_perm(2, 2, O.DOMAIN_GROUPS, 0, 0, 64),
              O.draw_perm(1, 3, O.DOMAIN_GROUPS, 0, 0, 64),
              O.draw_perm(1, 2, O.DOMAIN_ROUTE, 0, 0, 64),
              O.draw_perm(1, 2, O.DOMAIN_ROUTE, 1, 0, 64),
              O.draw_perm(1, 2, O.DOMAIN_ROUTE, 0, 1, 64)]
    for o in others:
        assert not np.array_equal(a, o)
    for i in range(len(others)):
        for j in range(i + 1, len(others)):
            assert not np.array_equal(others[i], others[j])


def test_groups_are_uniform_partitions():
    """W=4, n=2 has 3 possible pairings; each must come up about 1/3 of the
    time, and each worker must sit in each slot about equally often."""
    counts = {}
    slot = np.zeros((4, 4), dtype=int)
    T = 3000
    for step in range(T):
        perm = O.draw_groups(11, step, 4, 2)
        pairing = frozenset(frozenset(perm[g * 2:g * 2 + 2].tolist()) for g in range(2))
        counts[pairing] = counts.get(pairing, 0) + 1
        for s, w in enumerate(perm):
            slot[s, w] += 1
    assert len(counts) == 3
    chi2 = sum((c - T / 3) ** 2 / (T / 3) for c in counts.values())
    assert chi2 < 13.8            # chi-square, 2 dof, p = 0.001
    chi2s = ((slot - T / 4) ** 2 / (T / 4)).sum()
    assert chi2s < 27.9           # 9 dof, p = 0.001


def test_draw_groups_rejects_bad_sizes():
    for W, n in ((4, 3), (4, 0), (2, 4), (0, 1)):
        with pytest.raises(ValueError):
            O.draw_groups(0, 0, W, n)


# ------------------------------------------------------------------ bfloat16

def test_bf16_helpers_match_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 1, 20000).astype(F32),
                        rng.normal(0, 1e-30, 1000).astype(F32),
                        np.array([0.0, -0.0, np.inf, -np.inf, 1.0, 1.00390625, 1.01171875,
                                  3.3895314e38, 1e-45, 65504.0], dtype=F32)])
    # exact ties: mantissa low half = 0x8000
    ties = (rng.integers(0, 2**15, 5000, dtype=np.uint32) << 16 | 0x8000).astype(np.uint32).view(F32)
    x = np.concatenate([x, ties[np.isfinite(ties)]])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = O.f32_to_bf16_bits(x)
    assert np.array_equal(got, want)
    back = torch.from_numpy(want.view(np.int16)).view(torch.bfloat16).float().numpy()
    assert np.array_equal(O.bf16_bits_to_f32(want).view(np.uint32), back.view(np.uint32))
    assert np.isnan(O.bf16_bits_to_f32(O.f32_to_bf16_bits(np.array([np.nan], dtype=F32)))).all()


# ------------------------------------------------------------- Eq. 1-3 pins

def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            out[k] = np.array([float(t) for t in v])
    return out


def test_hand_computed_w2_p4():
    g = read_golden("outer_step_w2_p4.txt")
    phi = np.stack([g["phi_0"], g["phi_1"]]).astype(F32)
    theta = np.stack([g["theta_0"], g["theta_1"]]).astype(F32)
    delta = np.stack([g["delta_0"], g["delta_1"]]).astype(F32)
    a, b, c = (float(F32(g[k][0])) for k in ("alpha", "beta", "gamma"))
    for perm in ([0, 1], [1, 0]):
        p, d, t = O.outer_step(phi, theta, delta, np.array(perm, dtype=np.int32), 2, a, b, c)
        np.testing.assert_allclose(d, np.stack([g["delta_new_0"], g["delta_new_1"]]), rtol=3e-7, atol=1e-8)
        np.testing.assert_allclose(p, np.stack([g["phi_new_0"], g["phi_new_1"]]), rtol=3e-7, atol=1e-8)
        assert np.array_equal(t, p)


def test_subgroup_mean_phi_pins():
    """The early-exchange part of Eq. 2: the hand-computed case's mean phi, numpy's own mean
    over the member rows, the gossip corner (alpha = beta = 0, gamma = 1 makes every member
    equal to it), and the pull term of Eq. 2 recovered from a full step."""
    g = read_golden("outer_step_w2_p4.txt")
    phi = np.stack([g["phi_0"], g["phi_1"]]).astype(F32)
    m = O.subgroup_mean_phi(phi, np.array([1, 0], dtype=np.int32), 2)
    assert m.dtype == np.float64 and np.array_equal(m, [[2.0, 2.0, 0.0, 0.25]])   # from the golden file's header
    phi, theta, delta = rnd_state(12, 37, 5, phi_std=1.0)
    perm = O.draw_groups(3, 4, 12, 4)
    m = O.subgroup_mean_phi(phi, perm, 4)
    assert m.shape == (3, 37)
    for gi in range(3):
        rows = perm[gi * 4:(gi + 1) * 4]
        np.testing.assert_allclose(m[gi], np.mean(phi[rows], axis=0, dtype=np.float64), rtol=1e-14, atol=0)
        # a row swapped in from another group must change the mean (wrong member list is caught)
        other = perm[((gi + 1) % 3) * 4]
        assert not np.allclose(m[gi], np.mean(phi[[*rows[:3], other]], axis=0, dtype=np.float64))
    p, _, _ = O.outer_step(phi, theta, delta, perm, 4, 0.0, 0.0, 1.0)
    for gi in range(3):
        for w in perm[gi * 4:(gi + 1) * 4]:
            np.testing.assert_allclose(p[w], m[gi], rtol=2e-7, atol=1e-7)
    # Eq. 2 with alpha = beta = 0: delta_i' = -gamma (phi_i - mean)  =>  mean = phi_i + delta_i'/gamma
    _, d, _ = O.outer_step(phi, theta, delta, perm, 4, 0.0, 0.0, 0.5)
    for gi in range(3):
        w = perm[gi * 4]
        np.testing.assert_allclose(phi[w].astype(np.float64) + d[w].astype(np.float64) / 0.5, m[gi], atol=3e-7)


def test_diloco_reduction_full_group():
    """n = W: the third term of Eq. 2 vanishes only with gamma = 0 or equal
    phi; then the step is one global momentum step on the all-worker mean
    outer gradient (Section 3.2, the paragraph after Eq. 3)."""
    W, P = 8, 257
    phi, theta, delta = rnd_state(W, P, 1)
    delta[:] = delta[0]                         # DiLoCo: one shared momentum
    perm = O.draw_groups(5, 0, W, W)
    a, b = 0.3, 0.7
    g_all = (phi.astype(np.float64) - theta.astype(np.float64)).mean(axis=0)
    d_ref = a * delta[0].astype(np.float64) - b * g_all
    p, d, t = O.outer_step(phi, theta, delta, perm, W, a, b, 0.0)
    for i in range(W):
        np.testing.assert_allclose(d[i], d_ref, rtol=2e-7, atol=1e-12)
        np.testing.assert_allclose(p[i], phi[i] + d_ref, rtol=2e-7, atol=1e-12)
    # identical phi: any gamma gives the same result and all replicas stay equal
    phi[:] = phi[0]
    p0, d0, _ = O.outer_step(phi, theta, delta, perm, W, a, b, 0.0)
    p1, d1, _ = O.outer_step(phi, theta, delta, perm, W, a, b, 0.9)
    assert np.array_equal(p0, p1) and np.array_equal(d0, d1)
    assert all(np.array_equal(p0[0], p0[i]) for i in range(W))


def test_sign_pin_local_sgd_average():
    """alpha=0, beta=1, gamma=0, n=W, identical phi: phi' is the plain average
    of the fast weights (local SGD / federated averaging).  With the opposite
    sign of Eq. 1 the result would be 2*phi - mean(theta)."""
    W, P = 4, 33
    phi, theta, delta = rnd_state(W, P, 2, drift=0.5)
    phi[:] = phi[0]
    perm = np.arange(W, dtype=np.int32)
    p, d, t = O.outer_step(phi, theta, delta, perm, W, 0.0, 1.0, 0.0)
    want = theta.astype(np.float64).mean(axis=0)
    for i in range(W):
        np.testing.assert_allclose(p[i], want, rtol=2e-7, atol=1e-9)


def test_group_mean_identity_and_preservation():
    """Summing Eq. 2-3 over a group: the gamma term cancels, so
    mean_G phi' = mean_G phi + alpha mean_G delta - beta mean_G Delta."""
    W, n, P = 12, 4, 101
    phi, theta, delta = rnd_state(W, P, 3)
    perm = O.draw_groups(1, 1, W, n)
    a, b, c = 0.5, 0.7, 0.4
    p, d, _ = O.outer_step(phi, theta, delta, perm, n, a, b, c)
    for g in range(W // n):
        m = perm[g * n:(g + 1) * n]
        lhs = p[m].astype(np.float64).mean(0)
        rhs = (phi[m].astype(np.float64).mean(0) + a * delta[m].astype(np.float64).mean(0)
               - b * (phi[m].astype(np.float64) - theta[m]).mean(0))
        np.testing.assert_allclose(lhs, rhs, rtol=0, atol=3e-9)
    # beta = 0 and zero momentum: the pull toward the mean keeps the group mean
    z = np.zeros_like(delta)
    p, d, _ = O.outer_step(phi, theta, z, perm, n, a, 0.0, c)
    for g in range(W // n):
        m = perm[g * n:(g + 1) * n]
        np.testing.assert_allclose(p[m].astype(np.float64).mean(0),
                                   phi[m].astype(np.float64).mean(0), rtol=0, atol=3e-9)
        assert np.abs(p[m] - phi[m]).max() > 1e-3      # yet individual rows moved


def test_spread_identity():
    """phi_i' - mean' = (1-gamma)(phi_i - mean) + alpha (delta_i - mean delta)."""
    W, n, P = 8, 4, 64
    phi, theta, delta = rnd_state(W, P, 4, dstd=1e-2)
    perm = O.draw_groups(2, 0, W, n)
    a, b, c = 0.5, 0.7, 0.3
    p, _, _ = O.outer_step(phi, theta, delta, perm, n, a, b, c)
    for g in range(W // n):
        m = perm[g * n:(g + 1) * n]
        P64, D64, N64 = (x[m].astype(np.float64) for x in (phi, delta, p))
        lhs = N64 - N64.mean(0)
        rhs = (1 - c) * (P64 - P64.mean(0)) + a * (D64 - D64.mean(0))
        np.testing.assert_allclose(lhs, rhs, rtol=0, atol=5e-9)


def test_n1_is_lookahead_momentum():
    """n = 1: the group mean is the worker itself, so delta' = alpha delta - beta Delta."""
    W, P = 3, 50
    phi, theta, delta = rnd_state(W, P, 5)
    perm = O.draw_groups(0, 0, W, 1)
    p, d, _ = O.outer_step(phi, theta, delta, perm, 1, 0.5, 0.7, 0.8)
    want = 0.5 * delta.astype(np.float64) - 0.7 * (phi.astype(np.float64) - theta)
    np.testing.assert_allclose(d, want, rtol=2e-7, atol=1e-12)


def test_gossip_corner():
    """alpha = beta = 0, gamma = 1: every member lands on the group mean
    (pairwise weight averaging, as in epidemic learning)."""
    W, n, P = 6, 2, 40
    phi, theta, delta = rnd_state(W, P, 6)
    perm = O.draw_groups(9, 4, W, n)
    p, d, t = O.outer_step(phi, theta, delta, perm, n, 0.0, 0.0, 1.0)
    for g in range(W // n):
        m = perm[g * n:(g + 1) * n]
        want = phi[m].astype(np.float64).mean(0)
        for i in m:
            np.testing.assert_allclose(p[i], want, rtol=2e-7, atol=1e-12)


def test_fixed_point_and_theta_reset():
    W, n, P = 4, 2, 16
    phi, _, _ = rnd_state(W, P, 7)
    phi[:] = phi[0]
    z = np.zeros_like(phi)
    p, d, t = O.outer_step(phi, phi.copy(), z, np.arange(W, dtype=np.int32), n, 0.5, 0.7, 0.5)
    assert np.array_equal(p, phi) and not d.any() and np.array_equal(t, p)


def test_relabelling_workers_relabels_outputs():
    W, n, P = 8, 2, 30
    phi, theta, delta = rnd_state(W, P, 8)
    perm = O.draw_groups(3, 3, W, n)
    relabel = np.random.default_rng(0).permutation(W)        # new row r holds old worker relabel[r]
    inv = np.argsort(relabel)
    p, d, _ = O.outer_step(phi, theta, delta, perm, n, 0.5, 0.7, 0.5)
    p2, d2, _ = O.outer_step(phi[relabel], theta[relabel], delta[relabel],
                             inv[perm].astype(np.int32), n, 0.5, 0.7, 0.5)
    assert np.array_equal(p2, p[relabel]) and np.array_equal(d2, d[relabel])


def test_member_order_does_not_matter():
    W, n, P = 8, 4, 30
    phi, theta, delta = rnd_state(W, P, 9)
    perm = O.draw_groups(3, 3, W, n)
    perm2 = perm.copy()
    perm2[0:4] = perm[[3, 1, 0, 2]]
    a = O.outer_step(phi, theta, delta, perm, n, 0.5, 0.7, 0.5)
    b = O.outer_step(phi, theta, delta, perm2, n, 0.5, 0.7, 0.5)
    for x, y in zip(a, b):
        np.testing.assert_allclose(x, y, rtol=2e-7, atol=1e-12)


def test_bf16_theta_in_and_out():
    W, n, P = 4, 2, 1000
    phi, theta, delta = rnd_state(W, P, 10)
    tb = O.f32_to_bf16_bits(theta)
    perm = O.draw_groups(0, 0, W, n)
    p, d, t = O.outer_step(phi, tb, delta, perm, n, 0.5, 0.7, 0.5, O.THETA_BF16)
    p2, d2, _ = O.outer_step(phi, O.bf16_bits_to_f32(tb), delta, perm, n, 0.5, 0.7, 0.5)
    assert np.array_equal(p, p2) and np.array_equal(d, d2)
    assert t.dtype == np.uint16
    want = torch.from_numpy(p).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(t, want)


# ------------------------------------------------- Appendix D (convergence)

def quad_inner(phi, omega_lam, m, noise):
    """m SGD steps on the noisy quadratic: theta <- (1 - w L) theta + w L c."""
    theta = phi.astype(np.float64)
    for k in range(m):
        theta = (1 - omega_lam) * theta + omega_lam * noise[k]
    return theta.astype(F32)


def test_noise_free_quadratic_follows_appendix_d_recursion():
    """All workers equal and no noise: E(phi) obeys
    phi_{t+1} = D phi_t - alpha phi_{t-1}, D = 1 + alpha + beta (B^m - 1),
    whose solution is C1 r1^t + C2 r2^t with r the roots of r^2 - D r + alpha."""
    W, n, P = 4, 2, 3
    alpha, beta, gamma = 0.5, 0.7, 0.5
    wl = np.array([0.02, 0.1, 0.5])
    m = 5
    phi = np.tile(np.array([1.0, -2.0, 0.5], dtype=F32), (W, 1))
    delta = np.zeros_like(phi)
    Bm = (1 - wl) ** m
    D = 1 + alpha + beta * (Bm - 1)
    assert (np.abs(D) < 1 + alpha).all()
    r1 = (D + np.sqrt(D.astype(complex) ** 2 - 4 * alpha)) / 2
    r2 = (D - np.sqrt(D.astype(complex) ** 2 - 4 * alpha)) / 2
    phi0 = phi[0].astype(np.float64)
    phi1 = (1 + beta * (Bm - 1)) * phi0
    C2 = (phi1 - r1 * phi0) / (r2 - r1)
    C1 = phi0 - C2
    zeros = np.zeros((m, W, P))
    for t in range(40):
        theta = quad_inner(phi, wl, m, zeros)
        phi, delta, theta, _ = O.outer_step_seeded(phi, theta, delta, 0, t, n, alpha, beta, gamma)
        closed = (C1 * r1 ** (t + 1) + C2 * r2 ** (t + 1)).real
        for i in range(W):
            np.testing.assert_allclose(phi[i], closed, rtol=2e-5, atol=2e-6)
    assert np.abs(phi).max() < 2e-2 * np.abs(phi0).max()          # converging to the optimum 0


def test_noisy_quadratic_converges_to_neighbourhood():
    """Theorem 1: E(phi) -> 0 and the spread shrinks with the inner learning rate."""
    W, n, P, m, T = 16, 2, 2000, 10, 120
    alpha, beta, gamma = 0.5, 0.7, 0.7
    var = {}
    for omega in (0.2, 0.1):
        rng = np.random.default_rng(1)
        phi = np.full((W, P), 3.0, dtype=F32)
        delta = np.zeros_like(phi)
        acc = []
        for t in range(T):
            theta = quad_inner(phi, omega, m, rng.normal(0, 1, (m, W, P)))
            phi, delta, theta, _ = O.outer_step_seeded(phi, theta, delta, 4, t, n, alpha, beta, gamma)
            if t >= T - 40:
                acc.append(phi.astype(np.float64))
        acc = np.stack(acc)
        assert abs(acc.mean()) < 0.02                       # started at 3.0
        var[omega] = acc.var()
    assert 1.5 < var[0.2] / var[0.1] < 4.5


# ------------------------------------------------------------ divergence

def test_divergence_closed_forms():
    # hand example: values 1,2,3,4 across 4 workers: mean 2.5, population variance 1.25
    a, b = O.divergence(np.array([[1.0], [2.0], [3.0], [4.0]], dtype=F32))
    assert abs(a - 1.25 ** 0.5) < 1e-12 and abs(b - 1.25 ** 0.5) < 1e-12
    # two workers: std = |x0 - x1| / 2 per parameter
    x = np.array([[1.0, -2.0, 0.5], [3.0, -2.0, 0.0]], dtype=F32)
    a, b = O.divergence(x)
    assert abs(a - (1.0 + 0.0 + 0.25) / 3) < 1e-12
    assert abs(b - ((1.0 + 0.0 + 0.0625) / 3) ** 0.5) < 1e-12
    # identical replicas have no spread; one worker has none either
    assert O.divergence(np.tile(x[0], (5, 1))) == (0.0, 0.0)
    assert O.divergence(x[:1]) == (0.0, 0.0)


def test_divergence_against_numpy_and_invariances():
    rng = np.random.default_rng(3)
    x = (0.02 * rng.normal(size=(9, 1001)) + rng.normal(size=(1, 1001))).astype(F32)
    a, b = O.divergence(x)
    sd = np.std(x.astype(np.float64), axis=0)              # library routine, ddof = 0
    assert abs(a - sd.mean()) < 1e-14 and abs(b - np.sqrt((sd ** 2).mean())) < 1e-14
    assert a <= b + 1e-15                                   # Jensen: mean of roots <= root of mean
    sh = O.divergence((x.astype(np.float64) + 7.0))
    assert abs(sh[0] - a) < 1e-12 and abs(sh[1] - b) < 1e-12
    sc = O.divergence(x.astype(np.float64) * -3.0)
    assert abs(sc[0] - 3 * a) < 1e-12 and abs(sc[1] - 3 * b) < 1e-12
    assert O.divergence(x[rng.permutation(9)]) == pytest.approx((a, b), rel=1e-14)
    # brute force with python floats on a tiny case
    t = x[:3, :4].astype(np.float64)
    tot_s = tot_v = 0.0
    for p in range(4):
        m = sum(t[w, p] for w in range(3)) / 3
        v = sum((t[w, p] - m) ** 2 for w in range(3)) / 3
        tot_s += v ** 0.5
        tot_v += v
    got = O.divergence(x[:3, :4])
    assert abs(got[0] - tot_s / 4) < 1e-15 and abs(got[1] - (tot_v / 4) ** 0.5) < 1e-15


def test_gossip_step_removes_divergence_and_pull_shrinks_it():
    """Spread identity: with alpha = 0 a full-group step scales the spread by (1 - gamma)."""
    W, P = 8, 500
    phi, theta, delta = rnd_state(W, P, 12)
    perm = np.arange(W, dtype=np.int32)
    before = O.divergence(phi)
    p1, _, _ = O.outer_step(phi, theta, delta, perm, W, 0.0, 0.7, 0.25)
    after = O.divergence(p1)
    assert after[0] == pytest.approx(0.75 * before[0], rel=1e-5)
    assert after[1] == pytest.approx(0.75 * before[1], rel=1e-5)
    p2, _, _ = O.outer_step(phi, theta, delta, perm, W, 0.0, 0.7, 1.0)
    assert O.divergence(p2)[1] < 1e-8 * before[1] + 1e-9


# ------------------------------------------------------------------ routing

def test_route_tables_are_permutations():
    S, R, K = 4, 8, 4
    t = O.draw_route(1, 2, S, R, K)
    assert t.shape == (S - 1, K, R) and t.dtype == np.int32
    for b in range(S - 1):
        for k in range(K):
            assert sorted(t[b, k].tolist()) == list(range(R))
            assert np.array_equal(t[b, k], t[b, 0])          # slots travel together
    assert not np.array_equal(t[0], t[1])
    assert not np.array_equal(t, O.draw_route(1, 3, S, R, K))   # re-randomised every step
    pm = O.draw_route(1, 2, S, R, K, per_microbatch=True)
    assert np.array_equal(pm[:, 0], t[:, 0])
    assert not np.array_equal(pm[0, 0], pm[0, 1])
    assert O.draw_route(0, 0, 1, R, K).shape == (0, K, R)


def test_route_forward_backward():
    S, R, K, E = 3, 4, 2, 7
    rng = np.random.default_rng(0)
    acts = rng.integers(0, 2**16, (S - 1, R, K, E)).astype(np.uint16)
    for pm in (False, True):
        t = O.draw_route(5, 6, S, R, K, pm)
        out = O.route_forward(acts, t)
        # brute force: block identity by content
        for b in range(S - 1):
            for k in range(K):
                src = {acts[b, r, k].tobytes(): r for r in range(R)}
                assert [src[out[b, r, k].tobytes()] for r in range(R)] == t[b, k].tolist()
        assert np.array_equal(O.route_backward(out, t), acts)     # same path back
        assert np.array_equal(O.route_forward(O.route_backward(acts, t), t), acts)
