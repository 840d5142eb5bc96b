"""The outer step in two phases (Section 3.2, remark after Eq. 3): subgroup
means of phi prepared ahead, then the step that uses them.  Must give what the
fused step gives (the oracle's outer_step), must write exactly the oracle's
subgroup means into the carried buffer, and must refuse stale or mismatched
means."""

import numpy as np
import pytest
import torch

from oracle import nolo_oracle as O
from paper_2506_10911_b200 import synth
from tests.helpers import assert_outer_step_parity, to_np
from tests.test_gpu_magnitudes import step_and_compare

pytestmark = pytest.mark.gpu

HP = tuple(float(np.float32(x)) for x in (0.5, 0.7, 0.5))


@pytest.fixture(scope="module")
def nolo():
    from paper_2506_10911_b200 import binding
    return binding


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 8, 12, 20, 40, 64, 96, 128, 160, 256, 384, 700])
@pytest.mark.parametrize("bf16", [False, True])
def test_prepared_step_matches_oracle(nolo, n, bf16):
    W = 2 * n if n <= 256 else n
    step_and_compare(nolo, W, n, 6 * 150 + 2, torch.bfloat16 if bf16 else torch.float32, HP, seed=40 + n,
                     prepared=True)


def test_prepared_and_fused_steps_agree_over_consecutive_steps(nolo):
    """Three outer steps with fresh drift in between, run once fused and once split-phase
    (prepare issued right after the previous step, as a deployment would).  float32 theta, so
    that the two trajectories differ by accumulated float32 rounding only (with bfloat16 theta a
    last-bit difference in phi can flip the rounding of the next theta, a full bfloat16 ulp)."""
    W, n, P = 16, 2, 40_000
    state = synth.make_state(W, P, 21, torch.float32)
    fused = [x.clone().cuda() for x in state]
    split = [x.clone().cuda() for x in state]
    mean = torch.empty((W // n, synth.padded_stride(P, 8)), dtype=torch.float64, device="cuda")
    hf = nolo.nolo_create(W, n, P, 1, *HP)
    hs = nolo.nolo_create(W, n, P, 1, *HP)
    nolo.nolo_bind_state(hf, *fused)
    nolo.nolo_bind_state(hs, *split)
    nolo.nolo_bind_prepared(hs, mean)
    nolo.nolo_outer_prepare(hs, 9, 0)
    for k in range(3):
        for st in (fused, split):
            synth.apply_drift_(st[0], st[1], P, 300 + k)
        pre = [to_np(x).copy() for x in split]
        nolo.nolo_outer_step(hf, 9, k)
        nolo.nolo_outer_step_prepared(hs, 9, k)
        nolo.nolo_outer_prepare(hs, 9, k + 1)            # early exchange for the next step
        torch.cuda.synchronize()
        perm = O.draw_groups(9, k, W, n)
        want = O.outer_step(pre[0][:, :P], pre[1][:, :P], pre[2][:, :P], perm, n, *HP, O.THETA_F32)
        got = [to_np(x)[:, :P] for x in split]
        assert_outer_step_parity(got[0], got[2], got[1], want, False, f"step {k}: ")
        np.testing.assert_allclose(mean.cpu().numpy()[:, :P],
                                   O.subgroup_mean_phi(got[0], O.draw_groups(9, k + 1, W, n), n), rtol=1e-12,
                                   atol=1e-12 * float(np.abs(got[0]).max()))
        # the two forms differ by float32 rounding only; k + 1 steps of it have added up
        np.testing.assert_allclose(split[0].cpu().numpy(), fused[0].cpu().numpy(), rtol=(k + 1) * 2e-6,
                                   atol=(k + 1) * 1e-7)
    nolo.nolo_destroy(hf)
    nolo.nolo_destroy(hs)


@pytest.mark.parametrize("n", [2, 8])
def test_means_buffer_aligned_to_16_bytes_only(nolo, n):
    """The means are stored 32 bytes at a time when their rows allow it; a buffer that starts on
    a 16-byte boundary only takes the other store path and must give the same means."""
    W, P = 2 * n, 2051
    phi, theta, delta = synth.make_state(W, P, 77)
    dev = [x.cuda() for x in (phi, theta, delta)]
    stride = synth.padded_stride(P, 8)
    backing = torch.full((2 + (W // n) * stride,), float("nan"), dtype=torch.float64, device="cuda")
    mean = backing[2:].view(W // n, stride)
    assert mean.data_ptr() % 32 == 16
    h = nolo.nolo_create(W, n, P, 1, *HP)
    nolo.nolo_bind_state(h, *dev)
    nolo.nolo_bind_prepared(h, mean)
    nolo.nolo_outer_prepare(h, 3, 3)
    torch.cuda.synchronize()
    got = mean.cpu().numpy()
    want = O.subgroup_mean_phi(to_np(phi)[:, :P], O.draw_groups(3, 3, W, n), n)
    np.testing.assert_allclose(got[:, :P], want, rtol=1e-12, atol=1e-14)
    assert np.isnan(got[:, P:]).all() and np.isnan(backing[:2].cpu().numpy()).all()     # nothing else written
    nolo.nolo_destroy(h)


def test_prepared_means_are_refused_when_stale_or_mismatched(nolo):
    W, n, P = 8, 4, 1000
    dev = [x.cuda() for x in synth.make_state(W, P, 2)]
    keep = [x.clone() for x in dev]
    mean = torch.zeros((W // n, synth.padded_stride(P, 8)), dtype=torch.float64, device="cuda")
    h = nolo.nolo_create(W, n, P, 1, *HP)
    nolo.nolo_bind_state(h, *dev)

    def refused(seed, step):
        with pytest.raises(nolo.NoloError) as e:
            nolo.nolo_outer_step_prepared(h, seed, step)
        assert e.value.status == nolo.NOLO_ESTATE
        torch.cuda.synchronize()
        assert all(torch.equal(a, b) for a, b in zip(dev, keep)), "a refused call must not touch the state"
        return str(e.value)

    assert "nolo_bind_prepared" in refused(1, 1)          # no buffer bound
    with pytest.raises(nolo.NoloError) as e:
        nolo.nolo_outer_prepare(h, 1, 1)
    assert e.value.status == nolo.NOLO_ESTATE
    nolo.nolo_bind_prepared(h, mean)
    assert "nolo_outer_prepare" in refused(1, 1)          # bound but nothing prepared
    nolo.nolo_outer_prepare(h, 1, 1)
    assert "step 1" in refused(1, 2)                      # other step
    assert "seed 1" in refused(2, 1)                      # other seed
    nolo.nolo_outer_step_prepared(h, 1, 1)                # the matching call runs ...
    torch.cuda.synchronize()
    assert not torch.equal(dev[0], keep[0])
    keep = [x.clone() for x in dev]
    assert "nolo_outer_prepare" in refused(1, 1)          # ... and consumes the means (phi has changed)
    nolo.nolo_outer_prepare(h, 1, 2)
    nolo.nolo_outer_step(h, 1, 2)                         # a fused step changes phi as well
    torch.cuda.synchronize()
    keep = [x.clone() for x in dev]
    assert "nolo_outer_prepare" in refused(1, 2)
    # argument checks of the bind call
    for bad_stride, code in ((P - 8, nolo.NOLO_EINVAL), (synth.padded_stride(P, 8) + 4, nolo.NOLO_EALIGN)):
        with pytest.raises(nolo.NoloError) as e:
            nolo.nolo_bind_prepared(h, mean, bad_stride)
        assert e.value.status == code
    with pytest.raises(nolo.NoloError) as e:
        nolo.nolo_bind_prepared(h, dev[0], dev[0].stride(0))       # overlaps the state
    assert e.value.status == nolo.NOLO_EINVAL
    nolo.nolo_destroy(h)
