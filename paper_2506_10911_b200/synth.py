"""Seeded synthetic inputs shaped like the paper's workloads.

This module only *generates inputs* (random state and activations, model
shapes); it holds none of the method's arithmetic and is the one module that
both the CUDA path's callers and the CPU checker's callers may use.

State of W data-parallel workers, each a flat vector of P parameters
(Section 3.2): slow weights phi ~ N(0, 0.02^2), fast weights
theta = phi + drift with drift ~ N(0, (1e-3)^2) or Student-t(3) * 1e-3, and
outer momentum delta ~ N(0, (1e-4)^2).  theta is float32 or bfloat16.

Model shapes follow the paper's Table 3 (hidden size, layers, intermediate
size) with a 50k-entry tied embedding: P = V*d + L*(4*d*d + 2*d*ff + 2*d) + d.
"""

from __future__ import annotations

import torch

PHI_STD = 0.02
DRIFT_STD = 1e-3
DELTA_STD = 1e-4

# name -> (hidden d, layers L, intermediate ff, heads)   [paper, Table 3]
MODEL_SHAPES = {
    "125M": (768, 12, 3072, 12),
    "1.3B": (2048, 24, 8192, 32),
    "6.8B": (4096, 32, 16384, 32),
}
VOCAB = 50_000


def layer_params(d: int, ff: int) -> int:
    """Parameters of one decoder layer: q,k,v,o projections, a 2-matrix MLP
    and two norm vectors."""
    return 4 * d * d + 2 * d * ff + 2 * d


def model_params(name: str, vocab: int = VOCAB) -> int:
    """Flattened parameter count of a whole model (tied embedding + final norm)."""
    d, L, ff, _ = MODEL_SHAPES[name]
    return vocab * d + L * layer_params(d, ff) + d


def stage_params(name: str, stages: int) -> int:
    """Parameters of one middle pipeline stage (layers only) when the model
    is cut into ``stages`` equal runs of layers."""
    d, L, ff, _ = MODEL_SHAPES[name]
    assert L % stages == 0
    return (L // stages) * layer_params(d, ff)


def padded_stride(P: int, multiple: int = 64) -> int:
    """Row stride in elements: P rounded up to a multiple of ``multiple`` (64 elements: every
    row starts on a 256-byte boundary).  A stride that comes out as a multiple of 2^17 elements
    (512 KiB rows or a multiple) gets 1024 more: rows that far apart by an exact power of two map
    the same column of every row to the same memory channels, which measured 4-8 % slower when
    hundreds of rows are streamed side by side; any smaller offset between rows removes it."""
    stride = (P + multiple - 1) // multiple * multiple
    if multiple >= 64 and stride % (1 << 17) == 0:
        stride += 1024
    return stride


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _student_t3_(out: torch.Tensor, gen: torch.Generator) -> torch.Tensor:
    """Fill ``out`` (float32) with Student-t(3) draws: Z / sqrt(chi2_3 / 3)."""
    z = torch.empty_like(out).normal_(generator=gen)
    s = torch.zeros_like(out)
    for _ in range(3):
        s += torch.empty_like(out).normal_(generator=gen) ** 2
    out.copy_(z / torch.sqrt(s / 3.0))
    return out


def fill_state_(phi: torch.Tensor, theta: torch.Tensor, delta: torch.Tensor,
                P: int, seed: int, drift: str = "normal",
                chunk: int = 1 << 24) -> None:
    """Fill the first P columns of the [W, stride] state tensors in place.

    Works on CPU or CUDA tensors; large rows are filled in column chunks so
    the temporaries stay small.  ``theta`` may be float32 or bfloat16.
    Padding columns (>= P) are left untouched.
    """
    W = phi.shape[0]
    gen = _gen(phi.device, seed)
    for w in range(W):
        for c0 in range(0, P, chunk):
            c1 = min(P, c0 + chunk)
            p = phi[w, c0:c1]
            p.normal_(0.0, PHI_STD, generator=gen)
            d = torch.empty(c1 - c0, dtype=torch.float32, device=phi.device)
            if drift == "normal":
                d.normal_(0.0, DRIFT_STD, generator=gen)
            elif drift == "student_t3":
                _student_t3_(d, gen).mul_(DRIFT_STD)
            else:
                raise ValueError(drift)
            theta[w, c0:c1].copy_(p + d)          # casts when theta is bfloat16
            delta[w, c0:c1].normal_(0.0, DELTA_STD, generator=gen)


def apply_drift_(phi: torch.Tensor, theta: torch.Tensor, P: int, seed: int,
                 drift: str = "normal", chunk: int = 1 << 24) -> None:
    """Stand-in for an inner optimisation phase between two outer steps:
    theta <- cast(phi + fresh drift)."""
    W = phi.shape[0]
    gen = _gen(phi.device, seed)
    for w in range(W):
        for c0 in range(0, P, chunk):
            c1 = min(P, c0 + chunk)
            d = torch.empty(c1 - c0, dtype=torch.float32, device=phi.device)
            if drift == "normal":
                d.normal_(0.0, DRIFT_STD, generator=gen)
            else:
                _student_t3_(d, gen).mul_(DRIFT_STD)
            theta[w, c0:c1].copy_(phi[w, c0:c1] + d)


def make_state(W: int, P: int, seed: int, theta_dtype=torch.float32,
               drift: str = "normal", stride: int | None = None,
               device="cpu", pad_value: float = 0.0):
    """Allocate and fill (phi, theta, delta) as [W, stride] tensors."""
    stride = padded_stride(P, 8) if stride is None else stride
    phi = torch.full((W, stride), pad_value, dtype=torch.float32, device=device)
    theta = torch.full((W, stride), pad_value, dtype=theta_dtype, device=device)
    delta = torch.full((W, stride), pad_value, dtype=torch.float32, device=device)
    fill_state_(phi, theta, delta, P, seed, drift)
    return phi, theta, delta


MIXED_BANDS = ("near_one", "shared_base", "unit_normal", "init_scale", "zero_drift", "large_momentum")


def make_state_mixed(W: int, P: int, seed: int, theta_dtype=torch.float32, stride: int | None = None,
                     pad_value: float = 0.0):
    """State whose columns cycle through six value regimes, for checking that the
    arithmetic holds its tolerance at any ordinary weight magnitude (CPU tensors).

    Column p belongs to band p % 6:
      0 near_one        phi = 1 + N(0, 0.02^2) per worker (norm gains);
      1 shared_base     phi = b_p + N(0, (1e-3)^2), b_p ~ U(-4, 4) common to all workers
                        (replicas that have stayed close around weights of any size);
      2 unit_normal     phi ~ N(0, 1) per worker (replicas far apart);
      3 init_scale      phi ~ N(0, 0.02^2) per worker (the usual initialisation scale);
      4 zero_drift      as band 3 but theta == phi exactly (Delta = 0; phi is made
                        representable in theta's type);
      5 large_momentum  as band 3 with delta ~ N(0, 1).
    Elsewhere theta = cast(phi + N(0, (1e-3)^2)) and delta ~ N(0, (1e-4)^2).
    Returns (phi, theta, delta) as [W, stride] tensors and the band index per column.
    """
    stride = padded_stride(P, 8) if stride is None else stride
    gen = _gen("cpu", seed)
    band = torch.arange(P) % len(MIXED_BANDS)
    noise = lambda std: torch.empty((W, P), dtype=torch.float32).normal_(0.0, std, generator=gen)  # noqa: E731
    base = torch.empty(P, dtype=torch.float32).uniform_(-4.0, 4.0, generator=gen)
    cols = {
        0: 1.0 + noise(PHI_STD),
        1: base.unsqueeze(0) + noise(DRIFT_STD),
        2: noise(1.0),
    }
    phi_v = noise(PHI_STD)
    for b, v in cols.items():
        phi_v = torch.where(band == b, v, phi_v)
    zero = band == 4
    if theta_dtype != torch.float32:
        phi_v = torch.where(zero, phi_v.to(theta_dtype).to(torch.float32), phi_v)
    theta_v = torch.where(zero, phi_v, phi_v + noise(DRIFT_STD)).to(theta_dtype)
    delta_v = torch.where(band == 5, noise(1.0), noise(DELTA_STD))
    phi = torch.full((W, stride), pad_value, dtype=torch.float32)
    theta = torch.full((W, stride), pad_value, dtype=theta_dtype)
    delta = torch.full((W, stride), pad_value, dtype=torch.float32)
    phi[:, :P], theta[:, :P], delta[:, :P] = phi_v, theta_v, delta_v
    return phi, theta, delta, band.numpy()


def make_acts(boundaries: int, R: int, K: int, E: int, seed: int,
              dtype=torch.float32, device="cpu") -> torch.Tensor:
    """Activations at the stage boundaries, [boundaries, R, K, E], N(0, 1)."""
    gen = _gen(device, seed)
    out = torch.empty((boundaries, R, K, E), dtype=dtype, device=device)
    for b in range(boundaries):
        for r in range(R):
            out[b, r].copy_(torch.empty((K, E), dtype=torch.float32,
                                        device=device).normal_(generator=gen))
    return out
