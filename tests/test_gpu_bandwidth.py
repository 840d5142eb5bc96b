"""Bandwidth floor of each kernel path against a plain copy timed in the same process.

Not a benchmark (bench.py reports the figures): a guard that a change which halves a kernel's
bandwidth -- a spill, a lost coalescing, an extra pass over memory -- fails the suite.  The
floors sit well under the measured fractions (0.98 register-resident, 0.97-0.84 two-pass,
1.0 routing, 1.0 divergence on a B200) so that run-to-run noise cannot trip them."""

import pytest
import torch

from paper_2506_10911_b200 import synth

pytestmark = pytest.mark.gpu

HP = (0.5, 0.7, 0.5)


@pytest.fixture(scope="module")
def nolo():
    from paper_2506_10911_b200 import binding
    return binding


@pytest.fixture(scope="module")
def copy_gbs(nolo):
    nbytes = 1 << 30
    src = torch.ones(nbytes, dtype=torch.uint8, device="cuda")
    dst = torch.empty_like(src)
    gbs = nolo.nolo_copy_probe(src, dst, nbytes, 10)
    assert gbs > 1000, "the plain copy itself is implausibly slow"
    return gbs


def outer_step_gbs(nolo, W, n, P, theta_dtype, launches=6):
    stride = synth.padded_stride(P)
    dev = torch.device("cuda")
    phi = torch.empty((W, stride), dtype=torch.float32, device=dev).uniform_(-0.03, 0.03)
    theta = phi.to(theta_dtype, copy=True)
    delta = torch.empty((W, stride), dtype=torch.float32, device=dev).uniform_(-1e-4, 1e-4)
    h = nolo.nolo_create(W, n, P, 1, *HP)
    nolo.nolo_bind_state(h, phi, theta, delta)
    for k in range(2):
        nolo.nolo_outer_step(h, k, k)
    nolo.nolo_timing_enable(h, True)
    for k in range(launches):
        nolo.nolo_outer_step(h, 2 + k, 2 + k)
    stats, cnt = nolo.nolo_timing_stats(h, nolo.NOLO_KERNEL_OUTER)
    nolo.nolo_destroy(h)
    assert cnt == launches
    bpp = 20 if theta_dtype == torch.bfloat16 else 24
    return bpp * W * P / (stats["median"] * 1e-3) / 1e9


# (W, n, P, theta, floor as a fraction of the plain copy): every case holds 1.3-1.6 GB of state
CASES = [
    (16, 2, 1 << 23, torch.bfloat16, 0.85),     # register-resident, the benchmark's kernel
    (8, 4, 1 << 23, torch.float32, 0.85),
    (8, 8, 1 << 23, torch.float32, 0.82),
    (12, 12, 1 << 23, torch.float32, 0.82),     # two passes, second read of phi from L1 / L2: one slot
    (32, 32, 1 << 22, torch.float32, 0.82),     # slots of two warps
    (128, 128, 1 << 20, torch.bfloat16, 0.78),  # slots of one warp
    (192, 192, 699_072, torch.float32, 0.75),
    (512, 512, 1 << 18, torch.float32, 0.70),
    (1024, 1024, 1 << 17, torch.bfloat16, 0.65),
]


@pytest.mark.parametrize("W,n,P,theta,floor", CASES)
def test_outer_step_bandwidth_floor(nolo, copy_gbs, W, n, P, theta, floor):
    gbs = outer_step_gbs(nolo, W, n, P, theta)
    assert gbs >= floor * copy_gbs, f"{gbs:.0f} GB/s is under {floor:.2f} of the plain copy's {copy_gbs:.0f} GB/s"


def test_routing_and_divergence_bandwidth_floor(nolo, copy_gbs):
    W, K, E, S = 8, 2, 1 << 24, 3                               # 2 boundaries x 16 x 32 MiB = 1 GiB moved each way
    h = nolo.nolo_create(W, 2, 8, S, *HP)
    acts = torch.ones((S - 1, W, K, E), dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(acts)
    nolo.nolo_bind_route(h, W * K, E, out)
    Wd, Pd = 16, 1 << 24                                        # 1 GiB of phi for the divergence metric
    hd = nolo.nolo_create(Wd, 2, Pd, 1, *HP)
    phi = torch.empty((Wd, Pd), dtype=torch.float32, device="cuda").uniform_(-1, 1)
    nolo.nolo_bind_state(hd, phi, phi.clone(), torch.zeros_like(phi))
    nolo.nolo_route(h, 0, 0, acts)
    nolo.nolo_divergence(hd)
    nolo.nolo_timing_enable(h, True)
    nolo.nolo_timing_enable(hd, True)
    for k in range(6):
        nolo.nolo_route(h, k, k, acts)
        nolo.nolo_divergence(hd)
    r, _ = nolo.nolo_timing_stats(h, nolo.NOLO_KERNEL_ROUTE)
    d, _ = nolo.nolo_timing_stats(hd, nolo.NOLO_KERNEL_DIVERGENCE)
    nolo.nolo_destroy(h)
    nolo.nolo_destroy(hd)
    route_gbs = 2 * acts.numel() * 2 / (r["median"] * 1e-3) / 1e9
    div_gbs = 4 * Wd * Pd / (d["median"] * 1e-3) / 1e9          # read-only: 4 bytes per worker-parameter
    assert route_gbs >= 0.85 * copy_gbs, f"routing {route_gbs:.0f} GB/s vs copy {copy_gbs:.0f} GB/s"
    assert div_gbs >= 0.75 * copy_gbs, f"divergence {div_gbs:.0f} GB/s vs copy {copy_gbs:.0f} GB/s"
