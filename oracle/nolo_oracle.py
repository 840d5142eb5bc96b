"""CPU oracle for the NoLoCo outer synchronisation step and random pipeline routing.

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, float64
restatement of the method, written from the paper, used only to check the CUDA
path (tests, the smoke check and the benchmark's CPU-baseline leg).  It shares
no code with the CUDA library and imports nothing from it.

What follows the paper directly (pinned by the tests against hand-computed
values, closed forms and invariants):

* ``outer_step``      -- Eq. 1 (outer gradient), Eq. 2 (modified Nesterov
                         momentum over a subgroup of n workers) and Eq. 3
                         (slow-weight update), then the reset of the fast
                         weights to the new slow weights (Section 3.2).
* ``subgroup_mean_phi`` -- the subgroup mean of the slow weights inside Eq. 2,
                         on its own (the part Section 3.2 says can be
                         exchanged ahead of the step).
* ``divergence``      -- the replica spread plotted in Fig. 3b (standard
                         deviation of the weights across the data-parallel
                         replicas).
* ``route_forward`` / ``route_backward`` -- Section 3.1 and Algorithm 1: every
                         step each stage boundary gets a fresh random
                         permutation of the replicas; activations follow it
                         forward, gradients return along the same path.

What the paper leaves open and this library fixes (the paper only says
"random" and "seed"); the *choice* of generator is therefore
"parity unpinned" by the paper itself -- the generator is pinned against
numpy's independent Philox implementation, and the tables built from it
against structural properties (bijection, determinism, uniformity):

* ``philox4x64_10``   -- the counter-based generator of Salmon, Moraes, Dror
                         and Shaw, "Parallel random numbers: as easy as 1, 2, 3"
                         (SC'11), 4 words of 64 bits, 10 rounds.
* ``draw_perm``       -- a permutation of 0..N-1 obtained by sorting N random
                         64-bit keys, ties broken by the smaller index.

Sign convention.  Eq. 1 prints Delta = theta - phi while Eq. 2 subtracts
(beta/n) * sum(Delta); taken together the slow weights would move away from
the fast weights.  The convergence analysis (Appendix D) uses
E(delta) = alpha E(delta) + beta E(theta - phi), which moves phi toward theta.
The oracle therefore uses Delta = phi - theta with Eq. 2 exactly as printed,
which is the convergent reading and DiLoCo's convention.
"""

from __future__ import annotations

import numpy as np

MASK64 = (1 << 64) - 1

# Philox4x64 constants as published by Salmon et al. (SC'11): two multipliers
# and the two Weyl-sequence key increments (golden ratio, sqrt(3) - 1).
PHILOX_M0 = 0xD2E7470EE14C6C93
PHILOX_M1 = 0xCA5A826395121157
PHILOX_W0 = 0x9E3779B97F4A7C15
PHILOX_W1 = 0xBB67AE8584CAA73B

# Counter word 3 separates the two uses of the generator.
DOMAIN_GROUPS = 1   # subgroup draw of the outer step (Section 3.2)
DOMAIN_ROUTE = 2    # pipeline routing permutations (Section 3.1)

THETA_F32 = 0
THETA_BF16 = 1


# --------------------------------------------------------------------------
# Counter-based random numbers and permutations
# --------------------------------------------------------------------------

def philox4x64_10(ctr, key):
    """Philox-4x64 with 10 rounds (Salmon et al., SC'11, Section 3.3 / Fig. 1).

    ``ctr`` is 4 and ``key`` 2 unsigned 64-bit integers; returns 4 words.
    One round maps (c0, c1, c2, c3) to
    (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0));
    the key is bumped by the Weyl constants between rounds.
    """
    c0, c1, c2, c3 = (int(x) & MASK64 for x in ctr)
    k0, k1 = (int(x) & MASK64 for x in key)
    for r in range(10):
        if r > 0:
            k0 = (k0 + PHILOX_W0) & MASK64
            k1 = (k1 + PHILOX_W1) & MASK64
        p0 = PHILOX_M0 * c0
        p1 = PHILOX_M1 * c2
        hi0, lo0 = p0 >> 64, p0 & MASK64
        hi1, lo1 = p1 >> 64, p1 & MASK64
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return (c0, c1, c2, c3)


def draw_keys(seed, step, domain, boundary, slot, N):
    """The N 64-bit sort keys of one permutation draw.

    Element i uses counter (i, boundary, slot, domain) under key (seed, step)
    and takes output word 0.  (Library-defined: the paper only names a seed.)
    """
    return [philox4x64_10((i, boundary, slot, domain), (seed, step))[0] for i in range(N)]


def draw_perm(seed, step, domain, boundary, slot, N):
    """A uniformly random permutation of 0..N-1 as an int32 array.

    Indices sorted ascending by (key_i, i): a sort of i.i.d. uniform keys is a
    uniform permutation (up to the 2^-64 mass of ties, which the index breaks).
    """
    keys = draw_keys(seed, step, domain, boundary, slot, N)
    order = sorted(range(N), key=lambda i: (keys[i], i))
    return np.asarray(order, dtype=np.int32)


def draw_groups(seed, step, W, n):
    """Random partition of the W workers into W/n subgroups of n (Section 3.2:
    a randomly chosen local subgroup of n instances, re-sampled every outer
    iteration).  Returns ``perm`` (int32, length W); group g is
    ``perm[g*n:(g+1)*n]``.  One permutation gives disjoint groups, so every
    worker takes part in exactly one exchange per outer step.
    """
    if W < 1 or n < 1 or n > W or W % n != 0:
        raise ValueError("need 1 <= n <= W and n dividing W")
    return draw_perm(seed, step, DOMAIN_GROUPS, 0, 0, W)


# --------------------------------------------------------------------------
# bfloat16 helpers (bit patterns held in uint16)
# --------------------------------------------------------------------------

def bf16_bits_to_f32(bits):
    """Widen bfloat16 bit patterns (uint16) to float32; exact."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32)


def f32_to_bf16_bits(x):
    """Round float32 to bfloat16 bit patterns, round-to-nearest-even.
    NaN stays NaN (quiet bit forced so the payload cannot round to Inf)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = ((u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        r = np.where(nan, ((u >> np.uint64(16)) | np.uint64(0x0040)).astype(np.uint16), r)
    return r


# --------------------------------------------------------------------------
# Outer step (Eq. 1-3)
# --------------------------------------------------------------------------

def outer_step(phi, theta, delta, perm, n, alpha, beta, gamma, theta_dtype=THETA_F32):
    """One NoLoCo outer step for W workers, out of place, in float64.

    phi, delta : float32 [W, P]   slow weights phi_{t,i}, outer momentum delta_{t-1,i}
    theta      : float32 [W, P], or uint16 [W, P] holding bfloat16 bits
                 (fast weights theta_{t+1,i} after the inner phase)
    perm       : int32 [W]; subgroup g is perm[g*n:(g+1)*n]
    Returns (phi', delta', theta') in the input dtypes.

    For each subgroup G and each member i of it:
        Delta_j  = phi_j - theta_j                                  (Eq. 1, sign as in the module header)
        delta_i' = alpha*delta_i - (beta/n) * sum_{j in G} Delta_j
                   - gamma * (phi_i - (1/n) * sum_{j in G} phi_j)   (Eq. 2)
        phi_i'   = phi_i + delta_i'                                 (Eq. 3)
        theta_i' = phi_i'        (next inner phase starts from the new slow weights)
    Both sums run over all n members, i included, and use the slow weights
    from before the update.  phi' and delta' are rounded to float32 once, at
    the end; a bfloat16 theta' is the float32 phi' rounded to nearest-even.
    """
    phi = np.asarray(phi)
    delta = np.asarray(delta)
    theta = np.asarray(theta)
    W, P = phi.shape
    assert phi.dtype == np.float32 and delta.dtype == np.float32
    if theta_dtype == THETA_BF16:
        assert theta.dtype == np.uint16
        theta_f = bf16_bits_to_f32(theta).astype(np.float64)
    else:
        assert theta.dtype == np.float32
        theta_f = theta.astype(np.float64)
    perm = np.asarray(perm)
    assert perm.shape == (W,) and W % n == 0

    phi_new = np.empty((W, P), dtype=np.float32)
    delta_new = np.empty((W, P), dtype=np.float32)
    for g in range(W // n):
        members = [int(w) for w in perm[g * n:(g + 1) * n]]
        phi_g = phi[members].astype(np.float64)            # [n, P]
        Delta_g = phi_g - theta_f[members]                 # Eq. 1
        mean_Delta = Delta_g.sum(axis=0) / n
        mean_phi = phi_g.sum(axis=0) / n
        for row, i in enumerate(members):
            d = (alpha * delta[i].astype(np.float64)
                 - beta * mean_Delta
                 - gamma * (phi_g[row] - mean_phi))        # Eq. 2
            delta_new[i] = d.astype(np.float32)
            phi_new[i] = (phi_g[row] + d).astype(np.float32)   # Eq. 3
    if theta_dtype == THETA_BF16:
        theta_new = f32_to_bf16_bits(phi_new)
    else:
        theta_new = phi_new.copy()
    return phi_new, delta_new, theta_new


def subgroup_mean_phi(phi, perm, n):
    """The part of Eq. 2 that depends on the slow weights alone: for every
    subgroup g, mean_g[p] = (1/n) * sum_{j in G_g} phi_j[p], float64 [W/n, P].

    Section 3.2 (the remark after Eq. 3) points out that these slow weights
    are known when the previous outer step ends and can be exchanged then.
    """
    phi = np.asarray(phi)
    W, P = phi.shape
    perm = np.asarray(perm)
    out = np.empty((W // n, P), dtype=np.float64)
    for g in range(W // n):
        members = [int(w) for w in perm[g * n:(g + 1) * n]]
        out[g] = phi[members].astype(np.float64).sum(axis=0) / n
    return out


def outer_step_seeded(phi, theta, delta, seed, step, n, alpha, beta, gamma,
                      theta_dtype=THETA_F32):
    """``outer_step`` with the subgroups drawn from (seed, step)."""
    perm = draw_groups(seed, step, phi.shape[0], n)
    out = outer_step(phi, theta, delta, perm, n, alpha, beta, gamma, theta_dtype)
    return out + (perm,)


# --------------------------------------------------------------------------
# Replica divergence (Fig. 3b)
# --------------------------------------------------------------------------

def divergence(phi):
    """Spread of the slow weights across the W data-parallel replicas (the
    quantity of Fig. 3b, before its normalisation by the run's maximum).

    For every parameter p: mean_p = (1/W) sum_w phi[w, p] and the population
    variance var_p = (1/W) sum_w (phi[w, p] - mean_p)^2.  Returns
    (mean_p sqrt(var_p), sqrt(mean_p var_p)); the paper does not say which
    scalar it plots, so both are given.
    """
    x = np.asarray(phi).astype(np.float64)
    W = x.shape[0]
    mean = x.sum(axis=0) / W
    var = ((x - mean) ** 2).sum(axis=0) / W
    return float(np.sqrt(var).sum() / var.size), float(np.sqrt(var.sum() / var.size))


# --------------------------------------------------------------------------
# Random pipeline routing (Section 3.1, Algorithm 1)
# --------------------------------------------------------------------------

def draw_route(seed, step, stages, R, K, per_microbatch=False):
    """Routing tables, int32 [stages-1, K, R].

    ``table[b, k, r]`` is the replica of stage b whose micro-batch slot k is
    received by replica r of stage b+1.  Each (b, k) row is a permutation of
    the R replicas, so every sender feeds exactly one receiver (the load
    balance Section 3.1 asks of the random groups).  By default one
    permutation per (step, boundary) serves all K slots; with
    ``per_microbatch`` every slot draws its own, as Algorithm 1's loop over
    the batch permits.
    """
    table = np.empty((max(stages - 1, 0), K, R), dtype=np.int32)
    for b in range(stages - 1):
        for k in range(K):
            slot = k if per_microbatch else 0
            table[b, k] = draw_perm(seed, step, DOMAIN_ROUTE, b, slot, R)
    return table


def route_forward(acts, table):
    """Forward routing: ``out[b, r, k] = acts[b, table[b, k, r], k]``.

    acts : [stages-1, R, K, E] outputs of stage b's replicas, any dtype;
    returns the inputs of stage b+1's replicas in the same layout (bit copy).
    """
    acts = np.asarray(acts)
    B, R, K = acts.shape[:3]
    out = np.empty_like(acts)
    for b in range(B):
        for r in range(R):
            for k in range(K):
                out[b, r, k] = acts[b, table[b, k, r], k]
    return out


def route_backward(grads, table):
    """Backward routing: gradients return along the forward path (Algorithm 1,
    backward pass): ``out[b, table[b, k, r], k] = grads[b, r, k]``.
    """
    grads = np.asarray(grads)
    B, R, K = grads.shape[:3]
    out = np.empty_like(grads)
    for b in range(B):
        for r in range(R):
            for k in range(K):
                out[b, table[b, k, r], k] = grads[b, r, k]
    return out
