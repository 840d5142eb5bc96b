"""nolo_outer_step_static -- the outer step for callers that cannot allocate
(their own pool owns the device, or cudaMalloc is off limits on their path).
It keeps the subgroup table in a fixed array inside the library instead of in
memory from cudaMalloc, so it must give exactly what nolo_outer_step gives.
Checked on two calls in a row, of different shapes, because the table is
shared between calls and keeps the previous call's contents."""

import gc

import pytest
import torch

from paper_2506_10911_b200 import synth

pytestmark = pytest.mark.gpu

HP = (0.5, 0.7, 0.5)


@pytest.fixture(scope="module")
def nolo():
    from paper_2506_10911_b200 import binding
    return binding


def reference_step(nolo, W, n, P, state, seed, step):
    dev = [x.clone().cuda() for x in state]
    h = nolo.nolo_create(W, n, P, 1, *HP)
    nolo.nolo_bind_state(h, *dev)
    nolo.nolo_outer_step(h, seed, step)
    torch.cuda.synchronize()
    nolo.nolo_destroy(h)
    return dev


def test_static_entry_point_matches_handle_path_twice(nolo):
    # The very first call on a device looks the table's address up, and the driver may load the
    # library's device code at that moment (as at any first launch), which takes device memory
    # once.  That set-up call comes first, on a small state; the two checked calls follow it.
    warm = [x.cuda() for x in synth.make_state(4, 64, 0)]
    warm_want = reference_step(nolo, 4, 2, 64, [x.cpu() for x in warm], 1, 1)
    nolo.nolo_outer_step_static(4, 2, 64, *HP, *warm, 1, 1)
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(warm, warm_want))
    calls = [(16, 2, 70_001, torch.bfloat16, 3, 0),     # larger W than the set-up call
             (8, 4, 33_333, torch.float32, 4, 1)]       # reuses the table: smaller W, other dtype
    for W, n, P, dt, seed, step in calls:
        state = synth.make_state(W, P, seed, dt)
        want = reference_step(nolo, W, n, P, state, seed, step)
        dev = [x.clone().cuda() for x in state]
        gc.collect()                                     # leftovers of earlier tests may be freed at any time
        torch.cuda.synchronize()
        pool_before = torch.cuda.memory_allocated()
        free_before = torch.cuda.mem_get_info()[0]       # the driver's own count: sees any cudaMalloc
        nolo.nolo_outer_step_static(W, n, P, *HP, *dev, seed, step)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() <= pool_before      # nothing taken from torch's pool
        # ... and nothing from the device behind torch's back (the driver hands memory out in
        # blocks of 2 MiB, so even a 4-byte cudaMalloc would show)
        assert free_before - torch.cuda.mem_get_info()[0] < (1 << 20)
        for got, w in zip(dev, want):
            # same kernels, same table: identical bits (tighter than the 2e-6 / 1e-7 parity tolerance)
            assert torch.equal(got, w)


def test_static_entry_point_rejects_more_workers_than_its_table_holds(nolo):
    W = nolo.NOLO_STATIC_MAX_WORKERS * 2
    phi, theta, delta = (x.cuda() for x in synth.make_state(W, 8, 0))
    keep = phi.clone()
    with pytest.raises(nolo.NoloError) as e:
        nolo.nolo_outer_step_static(W, 2, 8, *HP, phi, theta, delta, 0, 0)
    assert e.value.status == nolo.NOLO_EINVAL
    assert str(nolo.NOLO_STATIC_MAX_WORKERS) in str(e.value)
    torch.cuda.synchronize()
    assert torch.equal(phi, keep)                        # nothing ran
    # the limit itself is accepted
    W = nolo.NOLO_STATIC_MAX_WORKERS
    state = synth.make_state(W, 64, 1)
    want = reference_step(nolo, W, 4, 64, state, 9, 9)
    dev = [x.clone().cuda() for x in state]
    nolo.nolo_outer_step_static(W, 4, 64, *HP, *dev, 9, 9)
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(dev, want))
