"""Parity of every outer-step kernel path on weights of any ordinary magnitude.

The state's columns cycle through six regimes (norm gains near 1, replicas close
around weights of size up to 4, replicas far apart at unit scale, the usual
0.02 initialisation scale, exactly zero drift, large momentum), so an
accumulation whose error grows with |phi| or with the subgroup size, rather
than with the pseudo-gradient, is seen -- element by element against the
float64 oracle, with the same tolerance for every path."""

import numpy as np
import pytest
import torch

from oracle import nolo_oracle as O
from paper_2506_10911_b200 import synth
from tests.helpers import assert_outer_step_parity, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nolo():
    from paper_2506_10911_b200 import binding
    return binding


def step_and_compare(nolo, W, n, P, theta_dtype, hp, seed, prepared=False):
    alpha, beta, gamma = (float(np.float32(x)) for x in hp)
    phi, theta, delta, band = synth.make_state_mixed(W, P, seed, theta_dtype, pad_value=float("nan"))
    ins = [to_np(x).copy() for x in (phi, theta, delta)]
    dev = [x.cuda() for x in (phi, theta, delta)]
    h = nolo.nolo_create(W, n, P, 1, alpha, beta, gamma)
    nolo.nolo_bind_state(h, *dev)
    if prepared:
        mean = torch.full((W // n, synth.padded_stride(P, 8)), float("nan"), dtype=torch.float64, device="cuda")
        nolo.nolo_bind_prepared(h, mean)
        nolo.nolo_outer_prepare(h, seed, 7)
        nolo.nolo_outer_step_prepared(h, seed, 7)
    else:
        nolo.nolo_outer_step(h, seed, 7)
    torch.cuda.synchronize()
    perm = nolo.nolo_get_groups(h)
    nolo.nolo_destroy(h)
    assert np.array_equal(perm, O.draw_groups(seed, 7, W, n))
    bf16 = theta_dtype == torch.bfloat16
    want = O.outer_step(ins[0][:, :P], ins[1][:, :P], ins[2][:, :P], perm, n, alpha, beta, gamma,
                        O.THETA_BF16 if bf16 else O.THETA_F32)
    got = [to_np(x)[:, :P] for x in dev]
    for b, name in enumerate(synth.MIXED_BANDS):       # band by band, so a failure names its regime
        c = band == b
        assert_outer_step_parity(got[0][:, c], got[2][:, c], got[1][:, c], [w[:, c] for w in want], bf16,
                                 f"n={n} {name}: ")
    if prepared:
        # the carried means hold about 46 bits (a float32 pair), stored as float64
        np.testing.assert_allclose(mean.cpu().numpy()[:, :P], O.subgroup_mean_phi(ins[0][:, :P], perm, n),
                                   rtol=1e-12, atol=1e-12 * float(np.abs(ins[0][:, :P]).max()))


# one subgroup size per dispatch path and per boundary between paths
SIZES = [1, 2, 3, 4, 8, 9, 12, 13, 24, 25, 48, 64, 65, 96, 97, 112, 128, 129, 192, 224, 225, 256, 257, 300, 512, 640, 641, 1024]


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("bf16", [False, True])
def test_every_path_on_mixed_magnitudes(nolo, n, bf16):
    """Two subgroups (one above 256 members, to bound the oracle's time), P spanning several
    tiles with a ragged tail, the paper's alpha/beta with gamma = 0.5."""
    W = 2 * n if n <= 256 else n
    P = 6 * 200 + 3 if n <= 256 else 6 * 70 + 3
    step_and_compare(nolo, W, n, P, torch.bfloat16 if bf16 else torch.float32, (0.5, 0.7, 0.5), seed=n)


@pytest.mark.parametrize("n", [8, 48, 96, 128, 192, 256, 300])
@pytest.mark.parametrize("gamma", [0.0, 1.0])
def test_replicas_close_around_large_weights(nolo, n, gamma):
    """gamma = 0 (DiLoCo's outer step when n = W) and gamma = 1 on the same mixed state."""
    step_and_compare(nolo, n, n, 6 * 100 + 1, torch.float32, (0.3, 0.7, gamma), seed=1000 + n)


def test_larger_state_register_path(nolo):
    """Pairs and fours over enough columns to meet the rare near-cancellations of phi + delta'."""
    for n, dt in ((2, torch.bfloat16), (4, torch.float32), (8, torch.bfloat16)):
        step_and_compare(nolo, 16, n, 300_001, dt, (0.5, 0.7, 0.5), seed=5 + n)
