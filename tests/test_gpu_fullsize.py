"""Parity at the full sizes of the five configurations, in the launch
configuration the benchmark uses.  The state (up to 141 GB) is generated on the
device; the oracle checks sampled column windows of all W rows -- the first and
last columns, windows straddling tile boundaries and random ones -- and
whole-buffer properties are checked on the device (theta' is phi' rounded;
columns outside the windows changed too)."""

import numpy as np
import pytest
import torch

from oracle import c_oracle as C
from oracle import nolo_oracle as O
from paper_2506_10911_b200 import synth
from tests.helpers import assert_bf16_within_1ulp, assert_close_f32, to_np

pytestmark = pytest.mark.gpu

F32 = lambda x: float(np.float32(x))  # noqa: E731


@pytest.fixture(scope="module")
def nolo():
    from paper_2506_10911_b200 import binding
    return binding


@pytest.fixture(autouse=True)
def release_device_memory():
    yield
    import gc
    gc.collect()
    torch.cuda.empty_cache()


def need_gb(gb):
    free, _ = torch.cuda.mem_get_info()
    if free < gb * 1e9:
        pytest.skip(f"needs {gb:.0f} GB of free device memory, {free / 1e9:.0f} GB available")


def sample_columns(P, W, seed, width=2048, budget=1 << 21):
    """Sorted unique column indices: head, tail, tile-boundary straddles, random windows."""
    rng = np.random.default_rng(seed)
    n_win = max(6, budget // (W * width))
    starts = [0, max(0, P - width), max(0, P - width // 2 - 1)]
    for tile in (1024, 2048, 4096):                         # straddle some tile edges
        t = int(rng.integers(1, max(2, P // tile)))
        starts.append(max(0, min(P - width, t * tile - width // 2)))
    while len(starts) < n_win:
        starts.append(int(rng.integers(0, max(1, P - width))))
    cols = np.unique(np.concatenate([np.arange(s, min(P, s + width)) for s in starts]))
    return torch.from_numpy(cols)


def gather(t, cols_dev):
    return to_np(t.index_select(1, cols_dev))


def run_config(nolo, W, n, P, theta_dtype, hp, steps, drift="normal", seed0=0):
    bf16 = theta_dtype == torch.bfloat16
    stride = synth.padded_stride(P)
    need_gb(W * stride * (8 + (2 if bf16 else 4)) / 1e9 + 3)
    dev = torch.device("cuda")
    phi = torch.empty((W, stride), dtype=torch.float32, device=dev)
    theta = torch.empty((W, stride), dtype=theta_dtype, device=dev)
    delta = torch.empty((W, stride), dtype=torch.float32, device=dev)
    synth.fill_state_(phi, theta, delta, P, seed=seed0, drift=drift)
    h = nolo.nolo_create(W, n, P, 1, *hp)
    nolo.nolo_bind_state(h, phi, theta, delta)
    cols = sample_columns(P, W, seed0 + 17).to(dev)
    # a sample sixteen times larger for the last step, judged by the C writing of the oracle
    # (which has been cross-checked against the NumPy one and is fast enough for it)
    wide = sample_columns(P, W, seed0 + 99, width=1 << 14, budget=1 << 25).to(dev)
    for k in range(steps):
        seed, step = seed0 + k, k
        if k:
            synth.apply_drift_(phi, theta, P, seed=1000 + seed, drift=drift)
        pre = [gather(x, cols) for x in (phi, theta, delta)]
        pre_wide = [gather(x, wide) for x in (phi, theta, delta)] if k == steps - 1 else None
        probe = phi[:, P // 3: P // 3 + 4096].clone()          # a window the oracle does not look at
        nolo.nolo_outer_step(h, seed, step)
        torch.cuda.synchronize()
        perm = O.draw_groups(seed, step, W, n)
        assert np.array_equal(nolo.nolo_get_groups(h), perm)
        want = O.outer_step(pre[0], pre[1], pre[2], perm, n, *hp, O.THETA_BF16 if bf16 else O.THETA_F32)
        assert_close_f32(gather(phi, cols), want[0], f"phi step {k}")
        assert_close_f32(gather(delta, cols), want[1], f"delta step {k}")
        if bf16:
            assert_bf16_within_1ulp(gather(theta, cols), want[2], f"theta step {k}")
        else:
            assert_close_f32(gather(theta, cols), want[2], f"theta step {k}")
        if pre_wide is not None:
            want = C.outer_step(pre_wide[0], pre_wide[1], pre_wide[2], perm, n, *hp, O.THETA_BF16 if bf16 else O.THETA_F32)
            assert_close_f32(gather(phi, wide), want[0], f"phi step {k}, wide sample")
            assert_close_f32(gather(delta, wide), want[1], f"delta step {k}, wide sample")
            if bf16:
                assert_bf16_within_1ulp(gather(theta, wide), want[2], f"theta step {k}, wide sample")
            else:
                assert_close_f32(gather(theta, wide), want[2], f"theta step {k}, wide sample")
        # whole-buffer properties
        assert not torch.equal(probe, phi[:, P // 3: P // 3 + 4096])
        for w in range(W):
            assert torch.equal(phi[w, :P].to(theta_dtype), theta[w, :P]), f"theta != round(phi) in row {w}"
    nolo.nolo_destroy(h)


def test_config2_125M_bf16_ten_steps(nolo):
    """W=16, n=2, 125M decoder, fp32 phi/delta, bf16 theta, seeds 0..9."""
    run_config(nolo, 16, 2, synth.model_params("125M"), torch.bfloat16, (F32(.5), F32(.7), F32(.5)), steps=10)


def test_config2_every_element_by_sum_and_difference_identities(nolo):
    """Full coverage at full size without a host copy.  For a pair (n = 2), Eq. 2-3 fix the sum and
    the difference of the two members' new slow weights:
        phi_a' + phi_b' = (phi_a + phi_b) + alpha (delta_a + delta_b) - beta (Delta_a + Delta_b)
        phi_a' - phi_b' = (1 - gamma) (phi_a - phi_b) + alpha (delta_a - delta_b)
    and the two together fix every element.  Checked on the device in float64 for all 2e9 elements
    of the 125M x 16 configuration, with delta' = phi' - phi and theta' = round(phi')."""
    W, n, P = 16, 2, synth.model_params("125M")
    a_, b_, c_ = F32(.5), F32(.7), F32(.5)
    stride = synth.padded_stride(P)
    need_gb(2 * W * stride * 10 / 1e9 + 12)
    dev = torch.device("cuda")
    phi = torch.empty((W, stride), dtype=torch.float32, device=dev)
    theta = torch.empty((W, stride), dtype=torch.bfloat16, device=dev)
    delta = torch.empty((W, stride), dtype=torch.float32, device=dev)
    synth.fill_state_(phi, theta, delta, P, seed=3)
    phi0, theta0, delta0 = phi.clone(), theta.clone(), delta.clone()
    h = nolo.nolo_create(W, n, P, 1, a_, b_, c_)
    nolo.nolo_bind_state(h, phi, theta, delta)
    nolo.nolo_outer_step(h, 3, 0)
    torch.cuda.synchronize()
    perm = O.draw_groups(3, 0, W, n)
    assert np.array_equal(nolo.nolo_get_groups(h), perm)
    nolo.nolo_destroy(h)
    chunk = 1 << 24
    for g in range(W // n):
        a, b = int(perm[2 * g]), int(perm[2 * g + 1])
        for c0 in range(0, P, chunk):
            sl = slice(c0, min(P, c0 + chunk))
            pa, pb = phi0[a, sl].double(), phi0[b, sl].double()
            da, db = delta0[a, sl].double(), delta0[b, sl].double()
            Da, Db = pa - theta0[a, sl].double(), pb - theta0[b, sl].double()
            na, nb = phi[a, sl].double(), phi[b, sl].double()
            want_sum = (pa + pb) + a_ * (da + db) - b_ * (Da + Db)
            want_dif = (1 - c_) * (pa - pb) + a_ * (da - db)
            tol = 2 * (1e-7 + 2e-6 * torch.maximum(pa.abs(), pb.abs()))
            assert bool(((na + nb - want_sum).abs() <= tol).all()), f"sum identity, group {g}"
            assert bool(((na - nb - want_dif).abs() <= tol).all()), f"difference identity, group {g}"
            for r, p0, pn in ((a, pa, na), (b, pb, nb)):
                d_new = delta[r, sl].double()
                assert bool(((d_new - (pn - p0)).abs() <= 1e-7 + 2e-6 * d_new.abs()).all()), "delta' != phi' - phi"
                assert torch.equal(phi[r, sl].to(torch.bfloat16), theta[r, sl])


@pytest.mark.parametrize("gamma", [0.0, 0.5])
def test_config3_1p3B_fp32_three_steps(nolo, gamma):
    """W=8, n=4, 1.3B decoder, all fp32 (about 126 GB resident)."""
    run_config(nolo, 8, 4, synth.model_params("1.3B"), torch.float32, (F32(.5), F32(.7), F32(gamma)), steps=3)


def test_config4_6p8B_stage_bf16_with_routing(nolo):
    """One of 4 stages of the 6.8B decoder x 8 replicas, bf16 theta, plus routing
    of 32 micro-batches of 4x2048x4096 bf16 over 4 stages (about 141 GB)."""
    W, S, M, E = 8, 4, 32, 4 * 2048 * 4096
    P = synth.stage_params("6.8B", 4)
    need_gb(W * synth.padded_stride(P) * 10 / 1e9 + 2 * (S - 1) * M * E * 2 / 1e9 + 4)
    run_config(nolo, W, 2, P, torch.bfloat16, (F32(.5), F32(.7), F32(.5)), steps=1)
    torch.cuda.empty_cache()
    K = M // W
    dev = torch.device("cuda")
    acts = torch.empty((S - 1, W, K, E), dtype=torch.bfloat16, device=dev)
    gen = torch.Generator(device=dev).manual_seed(5)
    for b in range(S - 1):
        for r in range(W):
            acts[b, r].view(torch.int16).random_(-32768, 32767, generator=gen)    # arbitrary bit patterns
    out = torch.zeros_like(acts)
    h = nolo.nolo_create(W, 2, P, S, .5, .7, .5)
    nolo.nolo_bind_route(h, M, E, out)
    nolo.nolo_route(h, 3, 1, acts)
    torch.cuda.synchronize()
    table = O.draw_route(3, 1, S, W, K)
    assert np.array_equal(nolo.nolo_get_route(h), table)
    rng = np.random.default_rng(0)
    a16, o16 = acts.view(torch.int16), out.view(torch.int16)
    for b in range(S - 1):
        for k in range(K):
            for r in range(W):
                src = int(table[b, k, r])
                # whole block on the device, sampled windows against the oracle's copy on the host
                assert torch.equal(o16[b, r, k], a16[b, src, k])
            e0 = int(rng.integers(0, E - 4096))
            win = slice(e0, e0 + 4096)
            sub = to_np(acts[b, :, k, win]).reshape(1, W, 1, -1)
            want = O.route_forward(sub, table[b:b + 1, k:k + 1])
            assert np.array_equal(to_np(out[b, :, k, win]).reshape(1, W, 1, -1), want)
    back = torch.zeros_like(acts)
    nolo.nolo_route_backward(h, 3, 1, out, back)
    torch.cuda.synchronize()
    assert torch.equal(back.view(torch.int16), a16)
    nolo.nolo_destroy(h)


@pytest.mark.parametrize("W", [8, 32, 128])
@pytest.mark.parametrize("n", [2, 4, 8])
def test_config5_sweep_student_t(nolo, W, n):
    """64M fp32 parameters per worker, heavy-tailed drift."""
    run_config(nolo, W, n, 1 << 26, torch.float32, (F32(.5), F32(.7), F32(.5)), steps=1, drift="student_t3",
               seed0=W + n)
