"""ctypes binding of ``libnolo.so`` (the C ABI declared in ``include/nolo.h``).

Argument marshalling only: the functions here have the names and argument
order of the C entry points, take ``torch`` tensors (or raw addresses) where
the C side takes pointers, and raise :class:`NoloError` on a non-zero status.
There is no fallback: if the shared library is missing, importing this module
fails.
"""

from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnolo.so")

NOLO_OK, NOLO_EINVAL, NOLO_ESTATE, NOLO_EALIGN, NOLO_ECUDA, NOLO_ENOMEM = 0, -1, -2, -3, -4, -5
NOLO_F32, NOLO_BF16 = 0, 1
NOLO_KERNEL_OUTER, NOLO_KERNEL_ROUTE, NOLO_KERNEL_DIVERGENCE, NOLO_KERNEL_PREPARE = 0, 1, 2, 3
NOLO_MAX_WORKERS = 4096
NOLO_STATIC_MAX_WORKERS = 1024


class NoloError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        msg = f"{where}: {_lib.nolo_strerror(status).decode()} ({status})"
        if detail:
            msg += f": {detail}"
        super().__init__(msg)


if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2506_10911_b200.build` "
        "(there is no CPU or PyTorch fallback for the CUDA path)")

_lib = ctypes.CDLL(LIB_PATH)

_H = ctypes.c_void_p
_u64, _i64, _i32, _f32, _vp = ctypes.c_uint64, ctypes.c_int64, ctypes.c_int, ctypes.c_float, ctypes.c_void_p

# name -> argtypes; every entry point of include/nolo.h
SIGNATURES = {
    "nolo_create": [_i32, _i32, _i64, _i32, _f32, _f32, _f32, ctypes.POINTER(_H)],
    "nolo_bind_state": [_H, _vp, _vp, _vp, _i32, _i64, _vp],
    "nolo_outer_step": [_H, _u64, _u64],
    "nolo_bind_prepared": [_H, _vp, _i64],
    "nolo_outer_prepare": [_H, _u64, _u64],
    "nolo_outer_step_prepared": [_H, _u64, _u64],
    "nolo_outer_step_static": [_i32, _i32, _i64, _f32, _f32, _f32, _vp, _vp, _vp, _i32, _i64, _u64, _u64, _vp,
                               ctypes.c_char_p, _i32],
    "nolo_outer_step_host": [_H, _u64, _u64, _vp, _vp, _vp, _i64],
    "nolo_bind_route": [_H, _i32, _i64, _i32, _vp, _i32],
    "nolo_route": [_H, _u64, _u64, _vp],
    "nolo_route_boundary": [_H, _u64, _u64, _i32, _vp, _vp],
    "nolo_route_backward": [_H, _u64, _u64, _vp, _vp],
    "nolo_route_host": [_H, _u64, _u64, _vp, _vp, _vp],
    "nolo_get_groups": [_H, _vp],
    "nolo_get_route": [_H, _vp],
    "nolo_divergence": [_H, ctypes.POINTER(ctypes.c_double)],
    "nolo_copy_probe": [_vp, _vp, _i64, _i32, _vp, ctypes.POINTER(ctypes.c_double)],
    "nolo_sim_tree_allreduce": [_i32, ctypes.c_double, ctypes.c_double, _i64, _u64, _vp, _vp, _vp],
    "nolo_expected_pair_exchange": [ctypes.c_double, ctypes.c_double],
    "nolo_sim_straggler": [_i32, _i32, _i32, _i32, ctypes.c_double, ctypes.c_double, _i64, _u64, _vp, _vp, _vp],
    "nolo_timing_enable": [_H, _i32],
    "nolo_timing_read": [_H, _i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(_i64)],
    "nolo_timing_stats": [_H, _i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(_i64)],
    "nolo_launch_count": [_H, ctypes.POINTER(_i64)],
    "nolo_destroy": [_H],
    "nolo_strerror": [_i32],
    "nolo_last_error": [_H],
    "nolo_version": [],
}
for _name, _args in SIGNATURES.items():
    _fn = getattr(_lib, _name)
    _fn.argtypes = _args
    _fn.restype = (ctypes.c_char_p if _name in ("nolo_strerror", "nolo_last_error")
                   else ctypes.c_double if _name == "nolo_expected_pair_exchange" else ctypes.c_int)


def _ptr(x) -> int:
    """Address of a torch tensor / numpy array, or an int passed through."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return NOLO_F32
    if t.dtype == torch.bfloat16:
        return NOLO_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


class Handle:
    """Owns a ``nolo_handle*``; keeps references to bound tensors alive."""

    def __init__(self, ptr: int, W: int, n: int, P: int, stages: int):
        self.ptr = ptr
        self.W, self.n, self.P, self.stages = W, n, P, stages
        self.K = 0
        self._keep = {}

    def __del__(self):
        try:
            nolo_destroy(self)
        except Exception:
            pass


def _check(status: int, where: str, h: Handle | None = None):
    if status != NOLO_OK:
        detail = _lib.nolo_last_error(h.ptr).decode() if h is not None and h.ptr else ""
        raise NoloError(status, where, detail)


def nolo_create(W: int, n: int, P: int, stages: int, alpha: float, beta: float, gamma: float) -> Handle:
    out = _H()
    _check(_lib.nolo_create(W, n, P, stages, alpha, beta, gamma, ctypes.byref(out)), "nolo_create")
    return Handle(out.value, W, n, P, stages)


def nolo_bind_state(h: Handle, phi, theta, delta, stream=None, theta_dtype=None, row_stride=None):
    """phi/theta/delta: CUDA tensors of shape [W, row_stride]; stream: a
    ``torch.cuda.Stream`` (default: the current stream)."""
    import torch
    if theta_dtype is None:
        theta_dtype = _dtype_code(theta)
    if row_stride is None:
        row_stride = phi.stride(0)
    if stream is None:
        stream = torch.cuda.current_stream()
    sp = stream if isinstance(stream, int) else stream.cuda_stream
    _check(_lib.nolo_bind_state(h.ptr, _ptr(phi), _ptr(theta), _ptr(delta), theta_dtype, row_stride, sp),
           "nolo_bind_state", h)
    h._keep["state"] = (phi, theta, delta, stream)


def nolo_outer_step(h: Handle, seed: int, step: int):
    _check(_lib.nolo_outer_step(h.ptr, seed, step), "nolo_outer_step", h)


def nolo_bind_prepared(h: Handle, mean_phi, mean_stride=None):
    """mean_phi: CUDA float64 tensor [W/n, mean_stride] that carries the subgroup means of phi
    from nolo_outer_prepare to nolo_outer_step_prepared."""
    if mean_stride is None:
        mean_stride = mean_phi.stride(0)
    _check(_lib.nolo_bind_prepared(h.ptr, _ptr(mean_phi), mean_stride), "nolo_bind_prepared", h)
    h._keep["prepared"] = mean_phi


def nolo_outer_prepare(h: Handle, seed: int, next_step: int):
    _check(_lib.nolo_outer_prepare(h.ptr, seed, next_step), "nolo_outer_prepare", h)


def nolo_outer_step_prepared(h: Handle, seed: int, step: int):
    _check(_lib.nolo_outer_step_prepared(h.ptr, seed, step), "nolo_outer_step_prepared", h)


def nolo_outer_step_static(W: int, n: int, P: int, alpha: float, beta: float, gamma: float,
                           phi, theta, delta, seed: int, step: int, stream=None,
                           theta_dtype=None, row_stride=None):
    """Outer step without a handle and without any allocation (for callers whose device memory
    is entirely owned by their own pool, or who may not call cudaMalloc for other reasons).
    W is limited to NOLO_STATIC_MAX_WORKERS.  Call it once on each device before any stream
    capture; do not let two calls overlap on the GPU."""
    import torch
    if theta_dtype is None:
        theta_dtype = _dtype_code(theta)
    if row_stride is None:
        row_stride = phi.stride(0)
    if stream is None:
        stream = torch.cuda.current_stream()
    sp = stream if isinstance(stream, int) else stream.cuda_stream
    err = ctypes.create_string_buffer(256)
    status = _lib.nolo_outer_step_static(W, n, P, alpha, beta, gamma, _ptr(phi), _ptr(theta), _ptr(delta),
                                         theta_dtype, row_stride, seed, step, sp, err, len(err))
    if status != NOLO_OK:
        raise NoloError(status, "nolo_outer_step_static", err.value.decode())


def nolo_outer_step_host(h: Handle, seed: int, step: int, phi_host, theta_host, delta_host, host_stride=None):
    if host_stride is None:
        host_stride = phi_host.stride(0)
    _check(_lib.nolo_outer_step_host(h.ptr, seed, step, _ptr(phi_host), _ptr(theta_host), _ptr(delta_host),
                                     host_stride), "nolo_outer_step_host", h)


def nolo_bind_route(h: Handle, M: int, E: int, acts_out, per_microbatch: bool = False, act_dtype=None):
    if act_dtype is None:
        act_dtype = _dtype_code(acts_out)
    _check(_lib.nolo_bind_route(h.ptr, M, E, act_dtype, _ptr(acts_out), int(per_microbatch)),
           "nolo_bind_route", h)
    h.K = M // h.W
    h._keep["route"] = acts_out


def nolo_route(h: Handle, seed: int, step: int, acts):
    _check(_lib.nolo_route(h.ptr, seed, step, _ptr(acts)), "nolo_route", h)


def nolo_route_boundary(h: Handle, seed: int, step: int, boundary: int, acts_b, out_b):
    _check(_lib.nolo_route_boundary(h.ptr, seed, step, boundary, _ptr(acts_b), _ptr(out_b)),
           "nolo_route_boundary", h)


def nolo_route_backward(h: Handle, seed: int, step: int, grads, grads_out):
    _check(_lib.nolo_route_backward(h.ptr, seed, step, _ptr(grads), _ptr(grads_out)), "nolo_route_backward", h)


def nolo_route_host(h: Handle, seed: int, step: int, acts_host, out_host, acts_dev):
    _check(_lib.nolo_route_host(h.ptr, seed, step, _ptr(acts_host), _ptr(out_host), _ptr(acts_dev)),
           "nolo_route_host", h)


def nolo_get_groups(h: Handle) -> np.ndarray:
    out = np.empty(h.W, dtype=np.int32)
    _check(_lib.nolo_get_groups(h.ptr, out.ctypes.data), "nolo_get_groups", h)
    return out


def nolo_get_route(h: Handle) -> np.ndarray:
    out = np.empty((max(h.stages - 1, 0), h.K, h.W), dtype=np.int32)
    _check(_lib.nolo_get_route(h.ptr, out.ctypes.data), "nolo_get_route", h)
    return out


def nolo_divergence(h: Handle):
    """(mean per-parameter std across workers, root of the mean variance) of the bound phi."""
    out = (ctypes.c_double * 2)()
    _check(_lib.nolo_divergence(h.ptr, out), "nolo_divergence", h)
    return out[0], out[1]


def _stream_ptr(stream):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream if isinstance(stream, int) else stream.cuda_stream


def nolo_copy_probe(src, dst, nbytes: int, iters: int = 10, stream=None) -> float:
    """GB/s (read + write bytes) of a plain copy of nbytes from src to dst."""
    ms = ctypes.c_double()
    _check(_lib.nolo_copy_probe(_ptr(src), _ptr(dst), nbytes, iters, _stream_ptr(stream), ctypes.byref(ms)),
           "nolo_copy_probe")
    return 2.0 * nbytes / (ms.value * 1e-3) / 1e9


def nolo_sim_tree_allreduce(W: int, mu: float, sigma: float, trials: int, seed: int, stream=None,
                            return_trials: bool = False):
    """Returns (mean completion time, standard error[, per-trial times])."""
    stats = np.empty(2, dtype=np.float64)
    per = np.empty(trials, dtype=np.float64) if return_trials else None
    _check(_lib.nolo_sim_tree_allreduce(W, mu, sigma, trials, seed, _stream_ptr(stream), stats.ctypes.data,
                                        per.ctypes.data if return_trials else None), "nolo_sim_tree_allreduce")
    return (stats[0], stats[1], per) if return_trials else (stats[0], stats[1])


def nolo_expected_pair_exchange(mu: float, sigma: float) -> float:
    return _lib.nolo_expected_pair_exchange(mu, sigma)


def nolo_sim_straggler(W: int, n: int, H: int, T: int, mu: float, sigma: float, trials: int, seed: int,
                       stream=None, return_trials: bool = False):
    """Returns (mean barrier time, mean subgroup time, their standard errors[, per-trial [trials, 2]])."""
    stats = np.empty(4, dtype=np.float64)
    per = np.empty((trials, 2), dtype=np.float64) if return_trials else None
    _check(_lib.nolo_sim_straggler(W, n, H, T, mu, sigma, trials, seed, _stream_ptr(stream), stats.ctypes.data,
                                   per.ctypes.data if return_trials else None), "nolo_sim_straggler")
    return tuple(stats) + ((per,) if return_trials else ())


def nolo_timing_enable(h: Handle, enable: bool = True):
    _check(_lib.nolo_timing_enable(h.ptr, int(enable)), "nolo_timing_enable", h)


def nolo_timing_read(h: Handle, kernel: int):
    """Returns (total milliseconds, launches) since the last read."""
    ms, cnt = ctypes.c_double(), _i64()
    _check(_lib.nolo_timing_read(h.ptr, kernel, ctypes.byref(ms), ctypes.byref(cnt)), "nolo_timing_read", h)
    return ms.value, cnt.value


def nolo_timing_stats(h: Handle, kernel: int):
    """Returns ({'mean','min','median','max'} in milliseconds, launches) since the last read."""
    st, cnt = (ctypes.c_double * 4)(), _i64()
    _check(_lib.nolo_timing_stats(h.ptr, kernel, st, ctypes.byref(cnt)), "nolo_timing_stats", h)
    return dict(mean=st[0], min=st[1], median=st[2], max=st[3]), cnt.value


def nolo_launch_count(h: Handle) -> int:
    cnt = _i64()
    _check(_lib.nolo_launch_count(h.ptr, ctypes.byref(cnt)), "nolo_launch_count", h)
    return cnt.value


def nolo_destroy(h: Handle):
    if h is not None and h.ptr:
        p, h.ptr = h.ptr, 0
        _lib.nolo_destroy(p)
        h._keep.clear()


def nolo_strerror(status: int) -> str:
    return _lib.nolo_strerror(status).decode()


def nolo_last_error(h: Handle) -> str:
    return _lib.nolo_last_error(h.ptr if h else None).decode()


def nolo_version() -> int:
    return _lib.nolo_version()
