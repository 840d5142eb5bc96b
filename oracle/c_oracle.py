"""Loader of the plain-C writing of the oracle (``nolo_oracle_c.c``).

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Compiles the C file with gcc into
``libnolo_oracle_c.so`` beside it (no CUDA, no dependency on the CUDA library) and exposes
its functions on numpy arrays with the argument order of ``nolo_oracle.py``, so that the two
writings can be compared call by call.  Imported only by the tests and by the benchmark's
CPU-baseline leg.
"""

from __future__ import annotations

import ctypes
import os
import shutil
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_HERE, "nolo_oracle_c.c")
LIB = os.path.join(_HERE, "libnolo_oracle_c.so")

THETA_F32 = 0
THETA_BF16 = 1


def build(force: bool = False) -> str:
    """Compile the C oracle if it is missing or older than its source; return the path."""
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    gcc = shutil.which("gcc") or shutil.which("cc")
    if gcc is None:
        raise RuntimeError("no C compiler found for the C oracle")
    tmp = LIB + f".{os.getpid()}.tmp"
    cmd = [gcc, "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-o", tmp, SRC, "-lm"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("gcc failed:\n" + res.stdout + res.stderr)
    os.replace(tmp, LIB)
    return LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, i32, i64, u64, f64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint64, ctypes.c_double
        L.oc_threads.restype = i32
        L.oc_set_threads.argtypes = [i32]
        L.oc_philox4x64_10.argtypes = [vp, vp, vp]
        L.oc_draw_perm.argtypes = [u64, u64, u64, u64, u64, i32, vp]
        L.oc_outer_step.argtypes = [vp, vp, vp, vp, i32, i32, i64, i64, f64, f64, f64, i32, vp, vp, vp]
        L.oc_subgroup_mean_phi.argtypes = [vp, vp, i32, i32, i64, i64, vp, i64]
        L.oc_route.argtypes = [vp, vp, vp, i32, i32, i32, i64, i32]
        L.oc_divergence.argtypes = [vp, i32, i64, i64, vp]
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def threads() -> int:
    return int(lib().oc_threads())


def set_threads(t: int) -> None:
    lib().oc_set_threads(int(t))


def philox4x64_10(ctr, key):
    c = np.asarray([int(x) & (2**64 - 1) for x in ctr], dtype=np.uint64)
    k = np.asarray([int(x) & (2**64 - 1) for x in key], dtype=np.uint64)
    out = np.empty(4, dtype=np.uint64)
    lib().oc_philox4x64_10(_p(c), _p(k), _p(out))
    return tuple(int(x) for x in out)


def draw_perm(seed, step, domain, boundary, slot, N):
    perm = np.empty(N, dtype=np.int32)
    rc = lib().oc_draw_perm(int(seed), int(step), int(domain), int(boundary), int(slot), int(N), _p(perm))
    if rc != 0:
        raise ValueError(f"oc_draw_perm failed ({rc})")
    return perm


def _rows(a: np.ndarray):
    """A [W, P] array whose rows are contiguous (a column slice of a larger array is fine):
    returns (array, row stride in elements)."""
    a = np.asarray(a)
    if a.ndim != 2 or (a.shape[1] > 1 and a.strides[1] != a.itemsize) or a.strides[0] % a.itemsize:
        a = np.ascontiguousarray(a)
    return a, a.strides[0] // a.itemsize


def outer_step(phi, theta, delta, perm, n, alpha, beta, gamma, theta_dtype=THETA_F32):
    phi, s0 = _rows(phi)
    theta, s1 = _rows(theta)
    delta, s2 = _rows(delta)
    if not (s0 == s1 == s2):
        phi, theta, delta = (np.ascontiguousarray(x) for x in (phi, theta, delta))
        s0 = phi.shape[1]
    W, P = phi.shape
    assert phi.dtype == np.float32 and delta.dtype == np.float32
    assert theta.dtype == (np.uint16 if theta_dtype == THETA_BF16 else np.float32)
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    # outputs share the inputs' row stride, so one index serves all six arrays
    outs = [np.empty((W, s0), dtype=x.dtype) for x in (phi, delta, theta)]
    rc = lib().oc_outer_step(_p(phi), _p(theta), _p(delta), _p(perm), W, int(n), P, s0,
                             float(alpha), float(beta), float(gamma), int(theta_dtype),
                             _p(outs[0]), _p(outs[1]), _p(outs[2]))
    if rc != 0:
        raise ValueError(f"oc_outer_step failed ({rc})")
    return tuple(o[:, :P] for o in outs)


def subgroup_mean_phi(phi, perm, n):
    phi, s = _rows(phi)
    W, P = phi.shape
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    out = np.empty((W // n, P), dtype=np.float64)
    rc = lib().oc_subgroup_mean_phi(_p(phi), _p(perm), W, int(n), P, s, _p(out), P)
    if rc != 0:
        raise ValueError(f"oc_subgroup_mean_phi failed ({rc})")
    return out


def _route(acts, table, backward):
    acts = np.ascontiguousarray(acts)
    B, R, K = acts.shape[:3]
    table = np.ascontiguousarray(table, dtype=np.int32)
    out = np.empty_like(acts)
    block = int(np.prod(acts.shape[3:], dtype=np.int64)) * acts.itemsize
    rc = lib().oc_route(_p(acts), _p(out), _p(table), B, R, K, block, backward)
    if rc != 0:
        raise ValueError(f"oc_route failed ({rc})")
    return out


def route_forward(acts, table):
    return _route(acts, table, 0)


def route_backward(grads, table):
    return _route(grads, table, 1)


def divergence(phi):
    phi, s = _rows(phi)
    assert phi.dtype == np.float32
    out = np.empty(2, dtype=np.float64)
    rc = lib().oc_divergence(_p(phi), phi.shape[0], phi.shape[1], s, _p(out))
    if rc != 0:
        raise ValueError(f"oc_divergence failed ({rc})")
    return float(out[0]), float(out[1])
