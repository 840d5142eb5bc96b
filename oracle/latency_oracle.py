"""CPU oracle for the paper's latency simulations (Section 4.3, "Theoretical and
simulated speed-up", and the latency-analysis appendix).

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT: plain NumPy float64, used only
to check the CUDA simulation kernels.  Shares no code with them.

Two simulations, as the paper describes them:

* ``sim_tree_allreduce`` -- message times t ~ LogNormal(mu, sigma^2), i.i.d.
  A tree all-reduce over W = 2^L workers climbs a binary tree (a parent is
  ready when both children's messages have arrived: max over the two of
  child-ready + t) and then descends it again (a child has the result one
  message time after its parent).  With constant t_c this takes
  2 t_c log2(W), the paper's estimate; with W = 2 it is the paper's local
  averaging in pairs, max(t1, t2) + max(t3, t4), whose expectation
  2 (1 + erf(sigma/2)) exp(mu + sigma^2/2) is ``expected_pair_exchange``.
* ``sim_straggler`` -- every inner step of every worker takes
  LogNormal(mu, sigma^2) time (the paper uses mu = 1, sigma^2 = 0.5); no
  communication cost.  DiLoCo meets at a global barrier after every H inner
  steps; NoLoCo only waits for the members of its random subgroup of n.
  Returns the time for all workers to finish T outer iterations under each.

Random numbers (the paper gives none; the library defines them).  One Philox
block of four 64-bit words gives four log-normal times: uniform
u = ((x >> 11) + 0.5) 2^-53 from each word; Box-Muller on the word pairs (0, 1)
and (2, 3): r = sqrt(-2 ln u_a), z = r cos(2 pi u_b) and r sin(2 pi u_b), so the
block's four normals are [r01 cos, r01 sin, r23 cos, r23 sin]; t = exp(mu + sigma z).
Sample number j of a stream lives in block j // 4, position j % 4.
  tree:       stream index = heap index of the child end of the edge
              (2 .. 2W-1); counter (node // 4, trial, phase, 3), key (seed, 0);
              phase 0 up / 1 down
  straggler:  stream index = inner step k; counter (k // 4, worker w, outer step t, 4),
              key (seed, trial); subgroups of outer step t: the library's
              permutation draw with (seed, step = t, boundary = trial).
"""

from __future__ import annotations

import math

import numpy as np

from . import nolo_oracle as O

DOMAIN_TREE = 3
DOMAIN_STRAGGLER = 4

_M32 = np.uint64(0xFFFFFFFF)


def _mulhilo(a: int, b: np.ndarray):
    """(hi, lo) of the 128-bit product of the constant a and the uint64 array b."""
    a_lo, a_hi = np.uint64(a & 0xFFFFFFFF), np.uint64(a >> 32)
    b_lo, b_hi = b & _M32, b >> np.uint64(32)
    ll = a_lo * b_lo
    lh = a_lo * b_hi
    hl = a_hi * b_lo
    hh = a_hi * b_hi
    mid = (ll >> np.uint64(32)) + (lh & _M32) + (hl & _M32)
    lo = (mid << np.uint64(32)) | (ll & _M32)
    hi = hh + (lh >> np.uint64(32)) + (hl >> np.uint64(32)) + (mid >> np.uint64(32))
    return hi, lo


def philox4x64_10_np(c0, c1, c2, c3, k0: int, k1: int):
    """Vectorised Philox-4x64-10: counters are uint64 arrays (broadcast), the key two ints."""
    c0, c1, c2, c3 = np.broadcast_arrays(*(np.asarray(c, dtype=np.uint64) for c in (c0, c1, c2, c3)))
    c0, c1, c2, c3 = c0.copy(), c1.copy(), c2.copy(), c3.copy()
    with np.errstate(over="ignore"):
        for r in range(10):
            if r > 0:
                k0 = (k0 + O.PHILOX_W0) & O.MASK64
                k1 = (k1 + O.PHILOX_W1) & O.MASK64
            hi0, lo0 = _mulhilo(O.PHILOX_M0, c0)
            hi1, lo1 = _mulhilo(O.PHILOX_M1, c2)
            c0, c1, c2, c3 = hi1 ^ c1 ^ np.uint64(k0), lo1, hi0 ^ c3 ^ np.uint64(k1), lo0
    return c0, c1, c2, c3


def uniform_open(x):
    """Uniform in (0, 1) from 64-bit words: the top 53 bits plus one half, times 2^-53."""
    return ((np.asarray(x, dtype=np.uint64) >> np.uint64(11)).astype(np.float64) + 0.5) * 2.0 ** -53


def lognormal4_from_block(w0, w1, w2, w3, mu, sigma):
    """The four log-normal times of one Philox block (arrays broadcast): stacked on a new last
    axis in the order [cos of pair (0,1), sin of pair (0,1), cos of pair (2,3), sin of pair (2,3)]."""
    z = []
    for a, b in ((w0, w1), (w2, w3)):
        r = np.sqrt(-2.0 * np.log(uniform_open(a)))
        ang = 2.0 * np.pi * uniform_open(b)
        z += [r * np.cos(ang), r * np.sin(ang)]
    return np.exp(mu + sigma * np.stack(z, axis=-1))


def stream_times(count, c1, c2, domain, mu, sigma, k0, k1):
    """Samples 0 .. count-1 of the stream with counter words (block, c1, c2, domain) and key
    (k0, k1); c1 may be an array (one stream per entry, result [len(c1), count])."""
    blocks = np.arange((count + 3) // 4, dtype=np.uint64)
    c1 = np.asarray(c1, dtype=np.uint64)
    w = philox4x64_10_np(blocks if c1.ndim == 0 else blocks[None, :], c1 if c1.ndim == 0 else c1[:, None],
                         c2, domain, k0, k1)
    t = lognormal4_from_block(*w, mu, sigma)                  # [..., blocks, 4]
    return t.reshape(t.shape[:-2] + (-1,))[..., :count]


def expected_pair_exchange(mu, sigma):
    """E[max(t1,t2) + max(t3,t4)] = 2 (1 + erf(sigma/2)) exp(mu + sigma^2/2)
    for i.i.d. log-normal message times (the appendix's closed form, doubled
    for the two directions of the exchange)."""
    return 2.0 * (1.0 + math.erf(sigma / 2.0)) * math.exp(mu + sigma * sigma / 2.0)


def message_times(W, trial, phase, mu, sigma, seed):
    """Times of the 2W-2 messages of one phase of one trial, indexed by child node (2..2W-1)."""
    return stream_times(2 * W, trial, phase, DOMAIN_TREE, mu, sigma, seed, 0)


def sim_tree_allreduce(W, mu, sigma, trials, seed):
    """Completion time of a binary-tree all-reduce, one value per trial."""
    if W < 2 or W & (W - 1):
        raise ValueError("W must be a power of two >= 2")
    out = np.empty(trials, dtype=np.float64)
    for s in range(trials):
        up = message_times(W, s, 0, mu, sigma, seed)
        down = message_times(W, s, 1, mu, sigma, seed)
        ready = np.zeros(2 * W)
        for p in range(W - 1, 0, -1):                      # parents, bottom level first
            ready[p] = max(ready[2 * p] + up[2 * p], ready[2 * p + 1] + up[2 * p + 1])
        arrive = np.zeros(2 * W)
        arrive[1] = ready[1]
        for c in range(2, 2 * W):                          # top-down
            arrive[c] = arrive[c // 2] + down[c]
        out[s] = arrive[W:].max()
    return out


def sim_straggler(W, n, H, T, mu, sigma, trials, seed):
    """[trials, 2]: time for all workers to finish T outer iterations of H inner
    steps under (global barrier every outer step, wait only for the subgroup)."""
    out = np.empty((trials, 2), dtype=np.float64)
    w = np.arange(W, dtype=np.uint64)
    for s in range(trials):
        barrier_clock = 0.0
        clock = np.zeros(W)
        for t in range(T):
            steps = stream_times(H, w, t, DOMAIN_STRAGGLER, mu, sigma, seed, s)      # [W, H]
            work = np.zeros(W)
            for kk in range(H):                                   # same summation order as a loop
                work = work + steps[:, kk]
            barrier_clock += work.max()
            perm = O.draw_perm(seed, t, O.DOMAIN_GROUPS, s, 0, W)
            done = clock + work
            new = np.empty(W)
            for g in range(W // n):
                members = perm[g * n:(g + 1) * n]
                new[members] = done[members].max()
            clock = new
        out[s] = (barrier_clock, clock.max())
    return out
