"""Python face of the CPU oracle (test infrastructure only).

Compiles ``odsgd_oracle.cpp`` with g++ into ``libodsgd_oracle.so`` next to this
file (on first use, or when the source is newer) and wraps each rule as a
function over contiguous numpy arrays.  Nothing here touches CUDA, torch or
the product package; only tests, the smoke check and the benchmark's CPU
baseline call it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "odsgd_oracle.cpp")
_LIB = os.path.join(_HERE, "libodsgd_oracle.so")
# One rounding per operator: no contraction into FMA, no value-changing optimisation.
CXXFLAGS = ["-O2", "-std=c++17", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math"]

_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compile the oracle if it is missing or older than its source; return the .so path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["g++", *CXXFLAGS, "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        f32p, f64p = ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_double)
        pp32, pp64 = ctypes.POINTER(f32p), ctypes.POINTER(f64p)
        cf, cd, ci, sz = ctypes.c_float, ctypes.c_double, ctypes.c_int, ctypes.c_size_t
        sig = {
            "oracle_global_update": [pp32, ci, sz, f32p, f32p, f32p, cf, cf, cf],
            "oracle_ssgd_step": [pp32, ci, sz, f32p, f32p, cf, cf, cf],
            "oracle_local_update": [f32p, f32p, sz, f32p, cf],
            "oracle_asgd_step": [f32p, sz, f32p, f32p, cf, cf, cf],
            "oracle_local_update_dc_c": [f32p, f32p, f32p, sz, f32p, cf, cf],
            "oracle_local_update_dc_a": [f32p, f32p, f32p, f32p, sz, f32p, cf, cf, cf, cf],
            "oracle_local_update_momentum": [f32p, f32p, f32p, sz, f32p, cf, cf, cf],
            "oracle_global_update_mult": [pp32, ci, sz, f32p, f32p, f32p, cf, cf, cf,
                                          ctypes.POINTER(sz), sz, f32p, f32p],
            "oracle_dcasgd_step_c": [f32p, sz, f32p, f32p, cf, cf],
            "oracle_dcasgd_step_a": [f32p, sz, f32p, f32p, f32p, cf, cf, cf, cf],
            "oracle_global_update_f64": [pp64, ci, sz, f64p, f64p, f64p, cd, cd, cd],
            "oracle_local_update_f64": [f64p, f64p, sz, f64p, cd],
            "oracle_asgd_step_f64": [f64p, sz, f64p, f64p, cd, cd, cd],
        }
        for name, argtypes in sig.items():
            fn = getattr(_lib, name)
            fn.argtypes = argtypes
            fn.restype = ci
    return _lib


def _chk(a: np.ndarray, dtype, name: str, n: Optional[int] = None) -> np.ndarray:
    if not isinstance(a, np.ndarray) or a.dtype != dtype or not a.flags["C_CONTIGUOUS"] or a.ndim != 1:
        raise TypeError(f"{name}: need a contiguous 1-D {np.dtype(dtype).name} numpy array")
    if n is not None and a.shape[0] != n:
        raise ValueError(f"{name}: length {a.shape[0]} != {n}")
    return a


def _ptr(a: Optional[np.ndarray], ct):
    if a is None:
        return ctypes.cast(None, ctypes.POINTER(ct))
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _ptr_table(arrs: Sequence[np.ndarray], ct):
    tab = (ctypes.POINTER(ct) * len(arrs))()
    for i, a in enumerate(arrs):
        tab[i] = _ptr(a, ct)
    return tab


def global_update(grads: Sequence[np.ndarray], w: np.ndarray, v: np.ndarray, *, lr: float,
                  momentum: float, wd: float, w_prev: Optional[np.ndarray] = None) -> None:
    """Algorithm 1's update, in place on ``w`` and ``v``; ``w_prev`` receives the old weights."""
    n = _chk(w, np.float32, "w").shape[0]
    _chk(v, np.float32, "v", n)
    for m, g in enumerate(grads):
        _chk(g, np.float32, f"grads[{m}]", n)
    if w_prev is not None:
        _chk(w_prev, np.float32, "w_prev", n)
    rc = lib().oracle_global_update(_ptr_table(grads, ctypes.c_float), len(grads), n,
                                    _ptr(w, ctypes.c_float), _ptr(v, ctypes.c_float),
                                    _ptr(w_prev, ctypes.c_float), lr, momentum, wd)
    if rc != 0:
        raise ValueError("oracle_global_update: need at least one worker")


def ssgd_step(grads: Sequence[np.ndarray], w: np.ndarray, v: np.ndarray, *, lr: float,
              momentum: float, wd: float) -> None:
    """SSGD server step (Section 3.1: same as the OD-SGD server), in place."""
    n = _chk(w, np.float32, "w").shape[0]
    _chk(v, np.float32, "v", n)
    for m, g in enumerate(grads):
        _chk(g, np.float32, f"grads[{m}]", n)
    rc = lib().oracle_ssgd_step(_ptr_table(grads, ctypes.c_float), len(grads), n,
                                _ptr(w, ctypes.c_float), _ptr(v, ctypes.c_float),
                                lr, momentum, wd)
    if rc != 0:
        raise ValueError("oracle_ssgd_step: need at least one worker")


def local_update(w_bak: np.ndarray, g: np.ndarray, *, local_lr: float,
                 out: Optional[np.ndarray] = None) -> np.ndarray:
    """Algorithm 2's local update (SGD flavour): returns w_bak - local_lr * g."""
    n = _chk(w_bak, np.float32, "w_bak").shape[0]
    _chk(g, np.float32, "g", n)
    x = np.empty(n, np.float32) if out is None else _chk(out, np.float32, "out", n)
    lib().oracle_local_update(_ptr(w_bak, ctypes.c_float), _ptr(g, ctypes.c_float), n,
                              _ptr(x, ctypes.c_float), local_lr)
    return x


def asgd_step(g: np.ndarray, w: np.ndarray, v: np.ndarray, *, lr: float, momentum: float,
              wd: float) -> None:
    """ASGD server step: one worker's gradient applied at once, in place."""
    n = _chk(w, np.float32, "w").shape[0]
    _chk(v, np.float32, "v", n)
    _chk(g, np.float32, "g", n)
    lib().oracle_asgd_step(_ptr(g, ctypes.c_float), n, _ptr(w, ctypes.c_float),
                           _ptr(v, ctypes.c_float), lr, momentum, wd)


def local_update_dc_c(w_bak: np.ndarray, g: np.ndarray, x_prev: np.ndarray, *, local_lr: float,
                      lam: float, out: Optional[np.ndarray] = None) -> np.ndarray:
    """Eq. 4 as the local updater."""
    n = _chk(w_bak, np.float32, "w_bak").shape[0]
    _chk(g, np.float32, "g", n)
    _chk(x_prev, np.float32, "x_prev", n)
    x = np.empty(n, np.float32) if out is None else _chk(out, np.float32, "out", n)
    lib().oracle_local_update_dc_c(_ptr(w_bak, ctypes.c_float), _ptr(g, ctypes.c_float),
                                   _ptr(x_prev, ctypes.c_float), n, _ptr(x, ctypes.c_float),
                                   local_lr, lam)
    return x


def local_update_dc_a(w_bak: np.ndarray, g: np.ndarray, x_prev: np.ndarray,
                      mean_square: np.ndarray, *, local_lr: float, lam: float, m: float,
                      eps: float, out: Optional[np.ndarray] = None) -> np.ndarray:
    """Eq. 5 with Eq. 6's running mean square (updated in place) as the local updater."""
    n = _chk(w_bak, np.float32, "w_bak").shape[0]
    _chk(g, np.float32, "g", n)
    _chk(x_prev, np.float32, "x_prev", n)
    _chk(mean_square, np.float32, "mean_square", n)
    x = np.empty(n, np.float32) if out is None else _chk(out, np.float32, "out", n)
    lib().oracle_local_update_dc_a(_ptr(w_bak, ctypes.c_float), _ptr(g, ctypes.c_float),
                                   _ptr(x_prev, ctypes.c_float),
                                   _ptr(mean_square, ctypes.c_float), n,
                                   _ptr(x, ctypes.c_float), local_lr, lam, m, eps)
    return x


def local_update_momentum(w_bak: np.ndarray, g: np.ndarray, u: np.ndarray, *, local_lr: float,
                          momentum: float, wd: float, out: Optional[np.ndarray] = None) -> np.ndarray:
    """Local SGD with momentum (Section 4.1's MNIST run); the velocity ``u`` is updated in place."""
    n = _chk(w_bak, np.float32, "w_bak").shape[0]
    _chk(g, np.float32, "g", n)
    _chk(u, np.float32, "u", n)
    x = np.empty(n, np.float32) if out is None else _chk(out, np.float32, "out", n)
    lib().oracle_local_update_momentum(_ptr(w_bak, ctypes.c_float), _ptr(g, ctypes.c_float),
                                       _ptr(u, ctypes.c_float), n, _ptr(x, ctypes.c_float),
                                       local_lr, momentum, wd)
    return x


def global_update_mult(grads: Sequence[np.ndarray], w: np.ndarray, v: np.ndarray, *, lr: float,
                       momentum: float, wd: float, offsets: Sequence[int], lr_mult: np.ndarray,
                       wd_mult: np.ndarray, w_prev: Optional[np.ndarray] = None) -> None:
    """Algorithm 1's update with per-tensor learning-rate and weight-decay multipliers, in place."""
    n = _chk(w, np.float32, "w").shape[0]
    _chk(v, np.float32, "v", n)
    for m, g in enumerate(grads):
        _chk(g, np.float32, f"grads[{m}]", n)
    nt = len(offsets) - 1
    _chk(lr_mult, np.float32, "lr_mult", nt)
    _chk(wd_mult, np.float32, "wd_mult", nt)
    if w_prev is not None:
        _chk(w_prev, np.float32, "w_prev", n)
    offs = (ctypes.c_size_t * len(offsets))(*[int(o) for o in offsets])
    rc = lib().oracle_global_update_mult(_ptr_table(grads, ctypes.c_float), len(grads), n,
                                         _ptr(w, ctypes.c_float), _ptr(v, ctypes.c_float),
                                         _ptr(w_prev, ctypes.c_float), lr, momentum, wd, offs, nt,
                                         _ptr(lr_mult, ctypes.c_float), _ptr(wd_mult, ctypes.c_float))
    if rc != 0:
        raise ValueError("oracle_global_update_mult: bad worker count or offsets")


def dcasgd_step_c(g: np.ndarray, w: np.ndarray, w_bak_m: np.ndarray, *, lr: float, lam: float) -> None:
    """Eq. 4 applied at the server to one arriving gradient; w and the worker's backup in place."""
    n = _chk(w, np.float32, "w").shape[0]
    _chk(g, np.float32, "g", n)
    _chk(w_bak_m, np.float32, "w_bak_m", n)
    lib().oracle_dcasgd_step_c(_ptr(g, ctypes.c_float), n, _ptr(w, ctypes.c_float),
                               _ptr(w_bak_m, ctypes.c_float), lr, lam)


def dcasgd_step_a(g: np.ndarray, w: np.ndarray, w_bak_m: np.ndarray, mean_square: np.ndarray, *,
                  lr: float, lam: float, m: float, eps: float) -> None:
    """Eq. 6 then Eq. 5 applied at the server to one arriving gradient, in place."""
    n = _chk(w, np.float32, "w").shape[0]
    _chk(g, np.float32, "g", n)
    _chk(w_bak_m, np.float32, "w_bak_m", n)
    _chk(mean_square, np.float32, "mean_square", n)
    lib().oracle_dcasgd_step_a(_ptr(g, ctypes.c_float), n, _ptr(w, ctypes.c_float),
                               _ptr(w_bak_m, ctypes.c_float), _ptr(mean_square, ctypes.c_float),
                               lr, lam, m, eps)


def global_update_f64(grads: Sequence[np.ndarray], w: np.ndarray, v: np.ndarray, *, lr: float,
                      momentum: float, wd: float, w_prev: Optional[np.ndarray] = None) -> None:
    n = _chk(w, np.float64, "w").shape[0]
    _chk(v, np.float64, "v", n)
    for m, g in enumerate(grads):
        _chk(g, np.float64, f"grads[{m}]", n)
    if w_prev is not None:
        _chk(w_prev, np.float64, "w_prev", n)
    rc = lib().oracle_global_update_f64(_ptr_table(grads, ctypes.c_double), len(grads), n,
                                        _ptr(w, ctypes.c_double), _ptr(v, ctypes.c_double),
                                        _ptr(w_prev, ctypes.c_double), lr, momentum, wd)
    if rc != 0:
        raise ValueError("oracle_global_update_f64: need at least one worker")


def local_update_f64(w_bak: np.ndarray, g: np.ndarray, *, local_lr: float) -> np.ndarray:
    n = _chk(w_bak, np.float64, "w_bak").shape[0]
    _chk(g, np.float64, "g", n)
    x = np.empty(n, np.float64)
    lib().oracle_local_update_f64(_ptr(w_bak, ctypes.c_double), _ptr(g, ctypes.c_double), n,
                                  _ptr(x, ctypes.c_double), local_lr)
    return x


def asgd_step_f64(g: np.ndarray, w: np.ndarray, v: np.ndarray, *, lr: float, momentum: float,
                  wd: float) -> None:
    n = _chk(w, np.float64, "w").shape[0]
    _chk(v, np.float64, "v", n)
    _chk(g, np.float64, "g", n)
    lib().oracle_asgd_step_f64(_ptr(g, ctypes.c_double), n, _ptr(w, ctypes.c_double),
                               _ptr(v, ctypes.c_double), lr, momentum, wd)
