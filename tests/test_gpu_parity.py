"""Element-by-element parity of the CUDA path (through the C ABI) with the CPU
oracle on the same seeded inputs: subgroup and routing tables bit-exact,
float32 outputs within 1e-7 + 2e-6*|x|, bfloat16 theta within 1 ulp."""

import numpy as np
import pytest
import torch

from oracle import nolo_oracle as O
from paper_2506_10911_b200 import synth
from tests.helpers import assert_bf16_within_1ulp, assert_close_f32, assert_outer_step_parity, to_np

pytestmark = pytest.mark.gpu

F = float(np.float32(0.5)), float(np.float32(0.7)), float(np.float32(0.5))


@pytest.fixture(scope="module")
def nolo():
    from paper_2506_10911_b200 import binding
    return binding


def run_both(nolo, W, n, P, seed, step, theta_dtype=torch.float32, stride=None, hp=F,
             drift="normal", state_seed=0, pad_value=float("nan")):
    """One outer step on the GPU and in the oracle from the same state.
    Returns nothing; asserts parity, padding untouched and table equality."""
    alpha, beta, gamma = hp
    phi, theta, delta = synth.make_state(W, P, state_seed, theta_dtype, drift, stride, "cpu", pad_value)
    ins = [to_np(x).copy() for x in (phi, theta, delta)]
    d_phi, d_theta, d_delta = (x.cuda() for x in (phi, theta, delta))
    h = nolo.nolo_create(W, n, P, 1, alpha, beta, gamma)
    nolo.nolo_bind_state(h, d_phi, d_theta, d_delta)
    nolo.nolo_outer_step(h, seed, step)
    torch.cuda.synchronize()
    perm_gpu = nolo.nolo_get_groups(h)
    nolo.nolo_destroy(h)

    perm = O.draw_groups(seed, step, W, n)
    assert np.array_equal(perm_gpu, perm), "subgroup table differs from the oracle"
    bf16 = theta_dtype == torch.bfloat16
    want = O.outer_step(ins[0][:, :P], ins[1][:, :P], ins[2][:, :P], perm, n, alpha, beta, gamma,
                        O.THETA_BF16 if bf16 else O.THETA_F32)
    got = [to_np(x) for x in (d_phi, d_delta, d_theta)]
    assert_outer_step_parity(got[0][:, :P], got[1][:, :P], got[2][:, :P], want, bf16)
    if bf16:
        # theta is the GPU's own phi' rounded to nearest even: exact
        assert np.array_equal(got[2][:, :P], O.f32_to_bf16_bits(got[0][:, :P]))
    else:
        assert np.array_equal(got[2][:, :P].view(np.uint32), got[0][:, :P].view(np.uint32))
    # padding columns keep their bits
    for g, i in zip((got[0], got[2], got[1]), ins):
        assert np.array_equal(np.ascontiguousarray(g[:, P:]).view(np.uint8),
                              np.ascontiguousarray(i[:, P:]).view(np.uint8)), "padding was written"


# ------------------------------------------------------------------ tables

@pytest.mark.parametrize("W,n", [(1, 1), (2, 2), (4, 2), (8, 4), (16, 2), (32, 8), (128, 8), (128, 128),
                                 (1000, 5), (4096, 2)])
def test_subgroup_tables_bit_exact(nolo, W, n):
    phi, theta, delta = (x.cuda() for x in synth.make_state(W, 8, 0))
    h = nolo.nolo_create(W, n, 8, 1, *F)
    nolo.nolo_bind_state(h, phi, theta, delta)
    for seed, step in [(0, 0), (1, 0), (0, 1), (2**64 - 1, 2**63 + 5), (123456789, 42)]:
        nolo.nolo_outer_step(h, seed, step)
        got = nolo.nolo_get_groups(h)
        assert np.array_equal(got, O.draw_groups(seed, step, W, n))
    nolo.nolo_destroy(h)


# -------------------------------------------------------------- outer step

def test_config1_full(nolo):
    """W=4, n=2, P=2^20 float32, alpha=.5 beta=.7 gamma=.5, seed 0, step 0."""
    run_both(nolo, 4, 2, 1 << 20, 0, 0)


@pytest.mark.parametrize("n", [1, 2, 3, 4, 8, 12, 24])
@pytest.mark.parametrize("bf16", [False, True])
def test_group_sizes_and_ragged_tiles(nolo, n, bf16):
    """P spans several tiles with a ragged tail (not a multiple of 4)."""
    W = 24
    dt = torch.bfloat16 if bf16 else torch.float32
    run_both(nolo, W, n, 5 * 1024 + 3, 7, 3, dt, stride=5 * 1024 + 16)


@pytest.mark.parametrize("n", [5, 6, 7, 9, 10, 12, 13, 16, 17, 24, 25, 32, 33, 48, 49, 64, 65, 96, 97, 100, 112, 113, 128, 129, 160, 192, 193, 224,
                               225, 256, 300, 512, 520, 640, 641])
@pytest.mark.parametrize("bf16", [False, True])
def test_large_subgroups(nolo, n, bf16):
    """n > 8 runs the two-pass kernel in its eight shapes (up to 12, 24, 64, 96, 128, 224 and 640
    members, and beyond; slots of one to four warps or of half a warp, with member slots masked
    when n does not fill them).  Two subgroups, ragged P."""
    dt = torch.bfloat16 if bf16 else torch.float32
    run_both(nolo, 2 * n, n, 1000 + 3, 11, 4, dt)
    if n in (16, 100, 128):
        run_both(nolo, n, n, 257, 2, 9, dt, hp=(F[0], F[1], 0.0))     # one group of all workers


@pytest.mark.parametrize("P", [1, 2, 3, 4, 5, 7, 8, 9, 1023, 1024, 1025, 2047, 2049, 4100])
@pytest.mark.parametrize("bf16", [False, True])
def test_small_and_odd_P(nolo, P, bf16):
    dt = torch.bfloat16 if bf16 else torch.float32
    run_both(nolo, 4, 2, P, 1, 2, dt)
    run_both(nolo, 6, 3, P, 1, 2, dt)


@pytest.mark.parametrize("hp", [(0.0, 0.0, 1.0), (0.3, 0.7, 0.0), (0.9, 1.0, 1.5), (0.5, 0.7, 0.0)])
def test_hyperparameter_corners(nolo, hp):
    hp = tuple(float(np.float32(x)) for x in hp)
    run_both(nolo, 8, 2, 3000, 5, 5, hp=hp)
    run_both(nolo, 8, 8, 3000, 5, 5, hp=hp)       # n = W: the DiLoCo case


def test_heavy_tailed_drift(nolo):
    run_both(nolo, 8, 4, 1 << 16, 3, 1, drift="student_t3")
    run_both(nolo, 32, 8, 1 << 14, 3, 1, drift="student_t3")


@pytest.mark.parametrize("bf16", [False, True])
def test_nan_and_inf_propagate_within_their_subgroup_only(nolo, bf16):
    """No special-casing: a NaN or Inf in one member's column poisons that column for the members
    of its subgroup and nothing else."""
    W, n, P = 8, 2, 2048 + 5
    dt = torch.bfloat16 if bf16 else torch.float32
    phi, theta, delta = synth.make_state(W, P, 13, dt)
    phi[3, 17] = float("nan")
    theta[5, 100] = float("inf")
    delta[0, 2050] = float("-inf")            # in the ragged tail
    d = [x.cuda() for x in (phi, theta, delta)]
    h = nolo.nolo_create(W, n, P, 1, *F)
    nolo.nolo_bind_state(h, *d)
    nolo.nolo_outer_step(h, 2, 2)
    torch.cuda.synchronize()
    perm = nolo.nolo_get_groups(h)
    nolo.nolo_destroy(h)
    want = O.outer_step(to_np(phi)[:, :P], to_np(theta)[:, :P], to_np(delta)[:, :P], perm, n, *F,
                        O.THETA_BF16 if bf16 else O.THETA_F32)
    got_phi = to_np(d[0])[:, :P]
    assert np.array_equal(np.isfinite(got_phi), np.isfinite(want[0]))
    assert np.array_equal(np.isnan(got_phi), np.isnan(want[0]))
    bad = ~np.isfinite(want[0])
    assert 3 <= bad.sum() <= 5                  # 2 members x 2 columns, plus the one row with -inf momentum
    assert_close_f32(np.where(bad, 0, got_phi), np.where(bad, 0, want[0]), "phi")
    assert np.array_equal(got_phi[bad & ~np.isnan(want[0])], want[0][bad & ~np.isnan(want[0])])   # signed Inf


@pytest.mark.parametrize("W,n", [(8, 2), (32, 16), (256, 128)])
def test_infinite_slow_weight_stays_within_its_subgroup(nolo, W, n):
    """An infinite phi (a replica that has already diverged) makes that parameter non-finite for
    every member of its subgroup, as in the float64 definition, and touches nothing else.  Only
    finiteness is compared there: Inf - Inf arises in both, in different places."""
    P = 777
    phi, theta, delta = synth.make_state(W, P, 31)
    phi[1, 5] = float("inf")
    phi[W - 1, 700] = float("-inf")
    d = [x.cuda() for x in (phi, theta, delta)]
    h = nolo.nolo_create(W, n, P, 1, *F)
    nolo.nolo_bind_state(h, *d)
    nolo.nolo_outer_step(h, 4, 4)
    torch.cuda.synchronize()
    perm = nolo.nolo_get_groups(h)
    nolo.nolo_destroy(h)
    with np.errstate(invalid="ignore"):               # Inf - Inf in the definition itself
        want = O.outer_step(to_np(phi)[:, :P], to_np(theta)[:, :P], to_np(delta)[:, :P], perm, n, *F, O.THETA_F32)
    for got, w in zip((to_np(d[0])[:, :P], to_np(d[2])[:, :P], to_np(d[1])[:, :P]), want):
        assert np.array_equal(np.isfinite(got), np.isfinite(w))
        bad = ~np.isfinite(w)
        assert bad.sum() == 2 * n
        assert_close_f32(np.where(bad, 0, got), np.where(bad, 0, w), "finite part")


@pytest.mark.parametrize("W,n", [(4, 2), (8, 8), (24, 12), (40, 20), (64, 32), (72, 72), (130, 130), (200, 200), (600, 600), (700, 700)])
@pytest.mark.parametrize("bf16", [False, True])
def test_guard_bands_around_every_buffer_stay_intact(nolo, W, n, bf16):
    """Each state tensor sits between two 4 KiB bands of a known pattern inside a larger
    allocation; no kernel path (register-resident, two-pass in its shapes, ragged tail)
    may write outside its rows."""
    P, stride, band = 1000 + 3, 1008, 1024            # band in elements
    dt = torch.bfloat16 if bf16 else torch.float32
    state = synth.make_state(W, P, 8, dt, stride=stride, pad_value=7.0)
    bufs, views = [], []
    for x in state:
        big = torch.full((2 * band + W * stride,), -123.0, dtype=x.dtype, device="cuda")
        v = big[band:band + W * stride].view(W, stride)
        v.copy_(x)
        bufs.append(big)
        views.append(v)
    h = nolo.nolo_create(W, n, P, 1, *F)
    nolo.nolo_bind_state(h, *views)
    nolo.nolo_outer_step(h, 1, 1)
    torch.cuda.synchronize()
    nolo.nolo_destroy(h)
    for big, v in zip(bufs, views):
        assert bool((big[:band] == -123.0).all()) and bool((big[-band:] == -123.0).all()), "guard band written"
        assert bool((v[:, P:] == 7.0).all()), "padding written"
    assert not torch.equal(views[0][:, :P].cpu(), state[0][:, :P])       # and the step did run


def test_randomised_shapes(nolo):
    """Seeded random draw of (W, n, P, stride, dtype, hyper-parameters, seed, step): every kernel
    path meets odd sizes in combinations the hand-picked cases may miss."""
    rng = np.random.default_rng(2024)
    divisors = lambda w: [d for d in range(1, w + 1) if w % d == 0]  # noqa: E731
    for case in range(48):
        W = int(rng.choice([1, 2, 3, 4, 6, 8, 10, 12, 16, 18, 30, 36, 64, 70, 90, 96, 130, 144, 200, 260]))
        n = int(rng.choice(divisors(W)))
        P = int(rng.choice([1, 3, 6, 31, 127, 129, 640, 1021, 2050, 4097, 9000]))
        if W * P > 600_000:
            P = max(1, 600_000 // W)
        stride = synth.padded_stride(P, 8) + 8 * int(rng.integers(0, 3))
        dt = torch.bfloat16 if rng.integers(0, 2) else torch.float32
        hp = tuple(float(np.float32(x)) for x in (rng.uniform(0, 0.95), rng.uniform(0, 1.2), rng.uniform(0, 1.5)))
        run_both(nolo, W, n, P, int(rng.integers(0, 2**62)), int(rng.integers(0, 2**62)), dt, stride=stride,
                 hp=hp, state_seed=case)


def test_diloco_reduction_on_gpu(nolo):
    """n = W, gamma = 0, shared momentum: all replicas take the same global
    momentum step on the mean outer gradient (Section 3.2)."""
    W, P = 8, 4096
    phi, theta, delta = synth.make_state(W, P, 3)
    delta[:] = delta[0]
    want_d = 0.3 * delta[0].double() - 0.7 * (phi.double() - theta.double()).mean(0)
    d_phi, d_theta, d_delta = (x.cuda() for x in (phi, theta, delta))
    h = nolo.nolo_create(W, W, P, 1, 0.3, 0.7, 0.0)
    nolo.nolo_bind_state(h, d_phi, d_theta, d_delta)
    nolo.nolo_outer_step(h, 0, 0)
    torch.cuda.synchronize()
    for i in range(W):
        assert_close_f32(to_np(d_delta[i]), want_d.numpy(), "delta")
        assert torch.equal(d_delta[i], d_delta[0])
    nolo.nolo_destroy(h)


def test_ten_consecutive_steps_bf16(nolo):
    """Config-2 pattern at reduced P: 10 outer steps, call k uses (seed k,
    step k), fresh drift before each; every step is checked from the GPU's own
    pre-step state, and the final state against a pure-oracle run."""
    W, n, P = 16, 2, 50_000
    phi, theta, delta = synth.make_state(W, P, 11, torch.bfloat16)
    d_phi, d_theta, d_delta = (x.cuda() for x in (phi, theta, delta))
    o_phi, o_theta, o_delta = (to_np(x).copy() for x in (phi, theta, delta))
    h = nolo.nolo_create(W, n, P, 1, *F)
    nolo.nolo_bind_state(h, d_phi, d_theta, d_delta)
    for k in range(10):
        if k:
            synth.apply_drift_(d_phi, d_theta, P, 100 + k)
            # the pure-oracle trajectory sees the same fast weights (a bf16 rounding flip
            # in an input would be a different problem, not a rounding difference)
            o_theta = to_np(d_theta).copy()
        pre = [to_np(x).copy() for x in (d_phi, d_theta, d_delta)]
        nolo.nolo_outer_step(h, k, k)
        torch.cuda.synchronize()
        perm = O.draw_groups(k, k, W, n)
        assert np.array_equal(nolo.nolo_get_groups(h), perm)
        want = O.outer_step(pre[0], pre[1], pre[2], perm, n, *F, O.THETA_BF16)
        assert_close_f32(to_np(d_phi), want[0], f"phi step {k}")
        assert_close_f32(to_np(d_delta), want[1], f"delta step {k}")
        assert_bf16_within_1ulp(to_np(d_theta), want[2], f"theta step {k}")
        o_phi, o_delta, o_theta = O.outer_step(o_phi, o_theta, o_delta, perm, n, *F, O.THETA_BF16)
    nolo.nolo_destroy(h)
    # 10 steps of independent rounding: errors add, so 10x the one-step bound
    err = np.abs(to_np(d_phi).astype(np.float64) - o_phi)
    assert (err <= 10 * (1e-7 + 2e-6 * np.abs(o_phi))).all()


def test_resume_from_checkpoint_is_exact(nolo):
    """The draw depends only on (seed, step): a new handle continues exactly."""
    W, n, P = 8, 2, 10_000
    phi, theta, delta = synth.make_state(W, P, 5)

    def run(split):
        a, b, c = (x.clone().cuda() for x in (phi, theta, delta))
        h = nolo.nolo_create(W, n, P, 1, *F)
        nolo.nolo_bind_state(h, a, b, c)
        for k in range(6):
            if k == split:
                nolo.nolo_destroy(h)
                h = nolo.nolo_create(W, n, P, 1, *F)
                nolo.nolo_bind_state(h, a, b, c)
            nolo.nolo_outer_step(h, 9, k)
        torch.cuda.synchronize()
        nolo.nolo_destroy(h)
        return a.cpu(), c.cpu()

    a0, c0 = run(-1)
    a1, c1 = run(3)
    assert torch.equal(a0, a1) and torch.equal(c0, c1)


def test_host_state_path_matches_device_path(nolo):
    W, n, P = 16, 2, 3_000_001            # several column chunks, ragged tail
    for dt in (torch.float32, torch.bfloat16):
        phi, theta, delta = synth.make_state(W, P, 21, dt)
        stride = phi.stride(0)
        dev = [x.clone().cuda() for x in (phi, theta, delta)]
        h = nolo.nolo_create(W, n, P, 1, *F)
        nolo.nolo_bind_state(h, *dev)
        nolo.nolo_outer_step(h, 4, 2)
        torch.cuda.synchronize()
        want = [x.cpu() for x in dev]
        # page-locked buffers overlap the copies; ordinary pageable memory must work as well
        host = [x.clone().pin_memory() if dt == torch.float32 else x.clone() for x in (phi, theta, delta)]
        dev2 = [torch.zeros_like(x) for x in dev]
        nolo.nolo_bind_state(h, *dev2)
        nolo.nolo_outer_step_host(h, 4, 2, *host, host_stride=stride)
        for got, w, d2 in zip(host, want, dev2):
            assert torch.equal(got, w)
            assert torch.equal(d2.cpu()[:, :P], w[:, :P])
        nolo.nolo_destroy(h)


# ----------------------------------------------------------------- routing

@pytest.mark.parametrize("S,R,K,E,dt,pm", [
    (2, 4, 2, 2 * 128 * 256, torch.float32, False),      # config 1's routing
    (4, 8, 4, 4096 + 8, torch.bfloat16, False),
    (3, 8, 2, 5000, torch.bfloat16, True),
    (3, 4, 3, 1001, torch.bfloat16, False),              # 2002-byte blocks: element-wise path
    (2, 16, 1, 333, torch.float32, True),                # 1332-byte blocks: element-wise path
    (2, 1, 1, 64, torch.float32, False),
])
def test_route_bit_exact(nolo, S, R, K, E, dt, pm):
    acts = synth.make_acts(S - 1, R, K, E, 3, dt)
    d_acts = acts.cuda()
    d_out = torch.zeros_like(d_acts)
    h = nolo.nolo_create(R, 1, 8, S, *F)
    nolo.nolo_bind_route(h, R * K, E, d_out, pm)
    for seed, step in [(0, 0), (5, 9)]:
        nolo.nolo_route(h, seed, step, d_acts)
        torch.cuda.synchronize()
        table = O.draw_route(seed, step, S, R, K, pm)
        assert np.array_equal(nolo.nolo_get_route(h), table)
        want = O.route_forward(to_np(acts), table)
        assert np.array_equal(to_np(d_out), want)
        # gradients return along the same path
        d_back = torch.zeros_like(d_acts)
        nolo.nolo_route_backward(h, seed, step, d_out, d_back)
        torch.cuda.synchronize()
        assert np.array_equal(to_np(d_back), O.route_backward(want, table))
        assert torch.equal(d_back.view(torch.uint8), d_acts.view(torch.uint8))
    nolo.nolo_destroy(h)


@pytest.mark.parametrize("pm", [False, True])
def test_route_one_boundary_at_a_time(nolo, pm):
    S, R, K, E = 4, 8, 2, 3000
    acts = synth.make_acts(S - 1, R, K, E, 5, torch.bfloat16)
    d_acts = acts.cuda()
    d_out = torch.zeros_like(d_acts)
    h = nolo.nolo_create(R, 2, 8, S, *F)
    nolo.nolo_bind_route(h, R * K, E, torch.zeros_like(d_acts), pm)
    table = O.draw_route(6, 2, S, R, K, pm)
    want = O.route_forward(to_np(acts), table)
    for b in (2, 0, 1):
        nolo.nolo_route_boundary(h, 6, 2, b, d_acts[b], d_out[b])
        torch.cuda.synchronize()
        assert np.array_equal(to_np(d_out[b]), want[b])
    assert np.array_equal(nolo.nolo_get_route(h), table)
    with pytest.raises(nolo.NoloError) as e:
        nolo.nolo_route_boundary(h, 6, 2, 3, d_acts[0], d_out[0])
    assert e.value.status == nolo.NOLO_EINVAL
    nolo.nolo_destroy(h)


@pytest.mark.parametrize("E,dt", [(4096 + 8, torch.bfloat16), (1001, torch.bfloat16), (333, torch.float32)])
def test_route_guard_bands(nolo, E, dt):
    S, R, K, band = 3, 4, 2, 2048
    acts = synth.make_acts(S - 1, R, K, E, 4, dt).cuda()
    n_el = acts.numel()
    big = torch.full((2 * band + n_el,), -5.0, dtype=dt, device="cuda")
    out = big[band:band + n_el].view_as(acts)
    h = nolo.nolo_create(R, 2, 8, S, *F)
    nolo.nolo_bind_route(h, R * K, E, out)
    nolo.nolo_route(h, 1, 2, acts)
    big2 = torch.full((2 * band + n_el,), -5.0, dtype=dt, device="cuda")
    back = big2[band:band + n_el].view_as(acts)
    nolo.nolo_route_backward(h, 1, 2, out, back)
    torch.cuda.synchronize()
    nolo.nolo_destroy(h)
    for b in (big, big2):
        assert bool((b[:band] == -5.0).all()) and bool((b[-band:] == -5.0).all())
    assert torch.equal(back, acts)


def test_route_single_stage_is_a_noop(nolo):
    h = nolo.nolo_create(4, 2, 8, 1, *F)
    out = torch.zeros(8, device="cuda")
    nolo.nolo_bind_route(h, 4, 2, out)
    nolo.nolo_route(h, 0, 0, torch.ones(8, device="cuda"))
    torch.cuda.synchronize()
    assert not out.any()
    nolo.nolo_destroy(h)


def test_route_host_path(nolo):
    S, R, K, E = 3, 4, 2, 4096
    acts = synth.make_acts(S - 1, R, K, E, 8, torch.bfloat16)
    h = nolo.nolo_create(R, 2, 8, S, *F)
    d_out = torch.zeros_like(acts, device="cuda")
    stage = torch.zeros_like(acts, device="cuda")
    nolo.nolo_bind_route(h, R * K, E, d_out)
    src, dst = acts.pin_memory(), torch.zeros_like(acts).pin_memory()
    nolo.nolo_route_host(h, 2, 3, src, dst, stage)
    want = O.route_forward(to_np(acts), O.draw_route(2, 3, S, R, K))
    assert np.array_equal(to_np(dst), want)
    nolo.nolo_destroy(h)


# --------------------------------------------------------------- divergence

@pytest.mark.parametrize("W,P", [(1, 10), (2, 4099), (8, 1 << 16), (16, 300_001), (128, 5000), (1000, 513)])
def test_divergence_matches_oracle(nolo, W, P):
    phi, theta, delta = synth.make_state(W, P, 4, pad_value=float("nan"))
    phi[:, :P] = phi[:1, :P] + 0.05 * phi[:, :P]            # replicas close to a common point
    dev = [x.cuda() for x in (phi, theta, delta)]
    h = nolo.nolo_create(W, 1, P, 1, *F)
    nolo.nolo_bind_state(h, *dev)
    got = nolo.nolo_divergence(h)
    want = O.divergence(to_np(phi)[:, :P])
    assert got[0] == pytest.approx(want[0], rel=1e-5, abs=1e-12)
    assert got[1] == pytest.approx(want[1], rel=1e-5, abs=1e-12)
    assert nolo.nolo_divergence(h) == got                    # reproducible bit for bit
    assert torch.equal(dev[0].cpu().view(torch.int32), phi.view(torch.int32))     # read-only
    nolo.nolo_destroy(h)


def test_divergence_after_gossip_step_is_zero(nolo):
    """alpha = beta = 0, gamma = 1, n = W puts every replica on the mean."""
    W, P = 16, 70_000
    dev = [x.cuda() for x in synth.make_state(W, P, 6)]
    h = nolo.nolo_create(W, W, P, 1, 0.0, 0.0, 1.0)
    nolo.nolo_bind_state(h, *dev)
    before = nolo.nolo_divergence(h)
    nolo.nolo_outer_step(h, 0, 0)
    after = nolo.nolo_divergence(h)
    assert before[0] > 1e-2 and after[1] < 1e-8
    nolo.nolo_destroy(h)


# ----------------------------------------------------- boundary behaviour

def test_error_codes(nolo):
    h = nolo.nolo_create(4, 2, 100, 2, *F)
    with pytest.raises(nolo.NoloError) as e:
        nolo.nolo_outer_step(h, 0, 0)
    assert e.value.status == nolo.NOLO_ESTATE
    with pytest.raises(nolo.NoloError) as e:
        nolo.nolo_get_groups(h)
    assert e.value.status == nolo.NOLO_ESTATE
    with pytest.raises(nolo.NoloError) as e:
        nolo.nolo_route(h, 0, 0, torch.zeros(8, device="cuda"))
    assert e.value.status == nolo.NOLO_ESTATE
    big = torch.zeros(3 * 4 * 104 + 16, device="cuda")
    ok = [big[i * 416:(i + 1) * 416].view(4, 104) for i in range(3)]
    with pytest.raises(nolo.NoloError) as e:                    # stride < P
        nolo.nolo_bind_state(h, *ok, row_stride=96)
    assert e.value.status == nolo.NOLO_EINVAL
    with pytest.raises(nolo.NoloError) as e:                    # stride not a multiple of 8
        nolo.nolo_bind_state(h, *ok, row_stride=100)
    assert e.value.status == nolo.NOLO_EALIGN
    with pytest.raises(nolo.NoloError) as e:                    # misaligned pointer
        nolo.nolo_bind_state(h, big[1:417].view(4, 104), ok[1], ok[2])
    assert e.value.status == nolo.NOLO_EALIGN
    with pytest.raises(nolo.NoloError) as e:                    # overlapping buffers
        nolo.nolo_bind_state(h, ok[0], ok[0], ok[2])
    assert e.value.status == nolo.NOLO_EINVAL
    assert "overlap" in nolo.nolo_last_error(h)
    with pytest.raises(nolo.NoloError) as e:                    # M not a multiple of W
        nolo.nolo_bind_route(h, 6, 16, torch.zeros(64, device="cuda"))
    assert e.value.status == nolo.NOLO_EINVAL
    out = torch.zeros(4 * 16, device="cuda")
    nolo.nolo_bind_route(h, 4, 16, out)
    with pytest.raises(nolo.NoloError) as e:                    # input aliases output
        nolo.nolo_route(h, 0, 0, out)
    assert e.value.status == nolo.NOLO_EINVAL
    nolo.nolo_bind_state(h, *ok)                                # the handle is still usable
    nolo.nolo_outer_step(h, 0, 0)
    torch.cuda.synchronize()
    nolo.nolo_destroy(h)


def test_timing_and_launch_count(nolo):
    W, n, P = 4, 2, 1 << 16
    dev = [x.cuda() for x in synth.make_state(W, P, 0)]
    h = nolo.nolo_create(W, n, P, 2, *F)
    nolo.nolo_bind_state(h, *dev)
    acts = torch.zeros(1, W, 1, 1024, device="cuda")
    out = torch.zeros_like(acts)
    nolo.nolo_bind_route(h, W, 1024, out)
    nolo.nolo_timing_enable(h, True)
    for k in range(5):
        nolo.nolo_outer_step(h, 0, k)
        nolo.nolo_route(h, 0, k, acts)
    ms, cnt = nolo.nolo_timing_read(h, nolo.NOLO_KERNEL_OUTER)
    assert cnt == 5 and 0 < ms < 1000
    ms, cnt = nolo.nolo_timing_read(h, nolo.NOLO_KERNEL_ROUTE)
    assert cnt == 5 and 0 < ms < 1000
    assert nolo.nolo_timing_read(h, nolo.NOLO_KERNEL_OUTER)[1] == 0
    for k in range(4):
        nolo.nolo_outer_step(h, 0, k)
    st, cnt = nolo.nolo_timing_stats(h, nolo.NOLO_KERNEL_OUTER)
    assert cnt == 4 and 0 < st["min"] <= st["median"] <= st["max"] and st["min"] <= st["mean"] <= st["max"]
    assert nolo.nolo_timing_stats(h, nolo.NOLO_KERNEL_OUTER)[1] == 0
    assert nolo.nolo_launch_count(h) == 28       # (draw + step) + (draw + copy) per iteration, + 4 more steps
    nolo.nolo_destroy(h)


def test_copy_probe(nolo):
    src = torch.arange(1 << 22, dtype=torch.int32, device="cuda")
    dst = torch.zeros_like(src)
    gbs = nolo.nolo_copy_probe(src, dst, src.numel() * 4, 3)
    assert torch.equal(src, dst) and gbs > 10
    with pytest.raises(nolo.NoloError) as e:
        nolo.nolo_copy_probe(src, src, src.numel() * 4, 3)
    assert e.value.status == nolo.NOLO_EINVAL
    with pytest.raises(nolo.NoloError) as e:
        nolo.nolo_copy_probe(src, dst, 24, 3)
    assert e.value.status == nolo.NOLO_EINVAL


def test_non_default_stream(nolo):
    W, n, P = 4, 2, 10_000
    phi, theta, delta = synth.make_state(W, P, 2)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        dev = [x.cuda() for x in (phi, theta, delta)]
        h = nolo.nolo_create(W, n, P, 1, *F)
        nolo.nolo_bind_state(h, *dev, stream=s)
        nolo.nolo_outer_step(h, 1, 1)
    s.synchronize()
    perm = O.draw_groups(1, 1, W, n)
    want = O.outer_step(to_np(phi), to_np(theta), to_np(delta), perm, n, *F)
    assert_close_f32(to_np(dev[0]), want[0], "phi")
    nolo.nolo_destroy(h)
