"""Thin ctypes binding of libodsgd.so: argument marshalling only.

Every arithmetic step runs inside the CUDA library; this module turns torch
tensors into raw device pointers, keeps the tensors alive while the context
borrows them, and maps error codes to exceptions.  There is no CPU fallback:
if the shared library is missing or fails to load, importing the symbols
raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libodsgd.so")

MAX_WORKERS = 64
FLAG_DETERMINISTIC = 0x1
FLAG_ALLOW_UNALIGNED = 0x2
FLAG_ALLOW_FMA = 0x4
FLAG_WORKER_ONLY = 0x8
MAX_BINDINGS = 16
MAX_MIRRORS = 15
LOCAL_SGD, LOCAL_DC_C, LOCAL_DC_A, LOCAL_MOMENTUM = 0, 1, 2, 3

OK, ERR_ARG, ERR_ALIGN, ERR_OVERLAP, ERR_STATE, ERR_CUDA, ERR_UNSUPPORTED = 0, -1, -2, -3, -4, -5, -6

# Every entry point include/odsgd.h declares.
EXPORTS = (
    "odsgd_version", "odsgd_strerror", "odsgd_create", "odsgd_destroy", "odsgd_global_update",
    "odsgd_local_update", "odsgd_fused_update", "odsgd_fused_update_host", "odsgd_ssgd_step",
    "odsgd_asgd_step", "odsgd_set_lr", "odsgd_set_local_lr", "odsgd_set_momentum", "odsgd_set_wd",
    "odsgd_set_local_rule", "odsgd_get_weights", "odsgd_get_step", "odsgd_set_step",
    "odsgd_set_launch_config", "odsgd_get_launch_count", "odsgd_last_error",
    "odsgd_set_tensor_multipliers", "odsgd_dcasgd_step", "odsgd_set_server_mean_square", "odsgd_set_warmup",
    "odsgd_step", "odsgd_get_train_weights", "odsgd_lr_step_decay", "odsgd_lr_linear_ramp",
    "odsgd_lr_poly_decay", "odsgd_fused_update_mult_static", "odsgd_get_iteration", "odsgd_set_iteration",
    "odsgd_bind_grads", "odsgd_unbind_grads", "odsgd_global_update_bound", "odsgd_fused_update_bound",
    "odsgd_ssgd_step_bound", "odsgd_step_bound", "odsgd_worker_local_update", "odsgd_shard_range",
    "odsgd_set_weight_mirrors",
)


class OdsgdError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"odsgd error {code}: {message}")
        self.code = code


class _Desc(ctypes.Structure):
    _fields_ = [
        ("w_a", ctypes.c_void_p), ("w_b", ctypes.c_void_p), ("w_delayed", ctypes.c_void_p),
        ("v", ctypes.c_void_p), ("local", ctypes.POINTER(ctypes.c_void_p)),
        ("n_params", ctypes.c_size_t), ("tensor_offsets", ctypes.POINTER(ctypes.c_size_t)),
        ("n_tensors", ctypes.c_size_t), ("n_workers", ctypes.c_int),
        ("lr", ctypes.c_float), ("local_lr", ctypes.c_float), ("momentum", ctypes.c_float),
        ("wd", ctypes.c_float), ("flags", ctypes.c_uint32),
    ]


_lib: Optional[ctypes.CDLL] = None


def load_library(path: str = LIB_PATH) -> ctypes.CDLL:
    """Loads libodsgd.so and declares its signatures.  Raises if it is not there."""
    global _lib
    if _lib is not None and path == LIB_PATH:
        return _lib
    if not os.path.exists(path):
        raise RuntimeError(
            f"{path} not found: build the CUDA library first (python -m paper_2005_06728_b200.build); "
            "there is no fallback path")
    lib = ctypes.CDLL(path)
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    pvp = ctypes.POINTER(ctypes.c_void_p)
    u64p = ctypes.POINTER(ctypes.c_uint64)
    sig = {
        "odsgd_version": ([], ci),
        "odsgd_strerror": ([ci], ctypes.c_char_p),
        "odsgd_create": ([ctypes.POINTER(vp), ctypes.POINTER(_Desc)], ci),
        "odsgd_destroy": ([vp], ci),
        "odsgd_global_update": ([vp, pvp, vp], ci),
        "odsgd_local_update": ([vp, ci, vp], ci),
        "odsgd_fused_update": ([vp, pvp, ci, vp], ci),
        "odsgd_fused_update_host": ([vp, pvp, pvp, ci, vp, vp, vp], ci),
        "odsgd_ssgd_step": ([vp, pvp, vp], ci),
        "odsgd_asgd_step": ([vp, ci, vp, vp], ci),
        "odsgd_set_lr": ([vp, cf], ci),
        "odsgd_set_local_lr": ([vp, cf], ci),
        "odsgd_set_momentum": ([vp, cf], ci),
        "odsgd_set_wd": ([vp, cf], ci),
        "odsgd_set_local_rule": ([vp, ci, cf, cf, cf, pvp], ci),
        "odsgd_get_weights": ([vp, ctypes.POINTER(vp), ctypes.POINTER(vp)], ci),
        "odsgd_get_step": ([vp, u64p], ci),
        "odsgd_set_step": ([vp, ctypes.c_uint64], ci),
        "odsgd_set_launch_config": ([vp, ci, ci], ci),
        "odsgd_get_launch_count": ([vp, u64p], ci),
        "odsgd_last_error": ([vp], ctypes.c_char_p),
        "odsgd_set_tensor_multipliers": ([vp, ctypes.POINTER(cf), ctypes.POINTER(cf), vp], ci),
        "odsgd_dcasgd_step": ([vp, ci, vp, vp], ci),
        "odsgd_set_server_mean_square": ([vp, vp], ci),
        "odsgd_set_warmup": ([vp, ctypes.c_uint64], ci),
        "odsgd_step": ([vp, pvp, vp], ci),
        "odsgd_get_train_weights": ([vp, ci, ctypes.POINTER(vp)], ci),
        "odsgd_lr_step_decay": ([cf, cf, u64p, ctypes.c_size_t, ctypes.c_uint64], cf),
        "odsgd_lr_linear_ramp": ([cf, cf, ctypes.c_uint64, ctypes.c_uint64], cf),
        "odsgd_lr_poly_decay": ([cf, cf, cf, ctypes.c_uint64, ctypes.c_uint64], cf),
        "odsgd_get_iteration": ([vp, u64p], ci),
        "odsgd_set_iteration": ([vp, ctypes.c_uint64], ci),
        "odsgd_fused_update_mult_static": ([vp, pvp, ci, ctypes.POINTER(cf), ctypes.POINTER(cf), vp], ci),
        "odsgd_bind_grads": ([vp, pvp, ctypes.POINTER(ci)], ci),
        "odsgd_unbind_grads": ([vp, ci], ci),
        "odsgd_global_update_bound": ([vp, ci, vp], ci),
        "odsgd_fused_update_bound": ([vp, ci, ci, vp], ci),
        "odsgd_ssgd_step_bound": ([vp, ci, vp], ci),
        "odsgd_step_bound": ([vp, ci, vp], ci),
        "odsgd_worker_local_update": ([vp, ci, vp, vp, ci, vp], ci),
        "odsgd_shard_range": ([ctypes.c_size_t, ci, ci, ctypes.POINTER(ctypes.c_size_t),
                               ctypes.POINTER(ctypes.c_size_t)], ci),
        "odsgd_set_weight_mirrors": ([vp, pvp, pvp, ci], ci),
    }
    for name, (argtypes, restype) in sig.items():
        fn = getattr(lib, name)  # AttributeError if the library lacks a declared symbol
        fn.argtypes = argtypes
        fn.restype = restype
    if path == LIB_PATH:
        _lib = lib
    return lib


def _dev_ptr(t: Optional[torch.Tensor], name: str, n: Optional[int] = None) -> Optional[int]:
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise TypeError(f"{name}: need a contiguous float32 CUDA tensor")
    if n is not None and t.numel() != n:
        raise ValueError(f"{name}: {t.numel()} elements, expected {n}")
    return t.data_ptr()


def _ptr_table(ptrs: Sequence[Optional[int]]):
    tab = (ctypes.c_void_p * len(ptrs))()
    for i, p in enumerate(ptrs):
        tab[i] = p
    return tab


def _stream_handle(stream: Optional[torch.cuda.Stream]) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


class GradTable:
    """The host array of device pointers the update calls take, built once from tensors that
    stay alive (and are not reallocated) as long as the table is used."""

    def __init__(self, grads: Sequence[torch.Tensor], n_workers: int, n_params: int):
        if len(grads) != n_workers:
            raise ValueError(f"need {n_workers} gradient tensors, got {len(grads)}")
        self.tensors = list(grads)
        self.n_workers, self.n_params = n_workers, n_params
        self.table = _ptr_table([_dev_ptr(g, f"grads[{i}]", n_params) for i, g in enumerate(grads)])

    def __len__(self) -> int:
        return self.n_workers

    def __iter__(self):
        return iter(self.tensors)


class BoundGrads:
    """A gradient table the library has checked once (odsgd_bind_grads): passing it to the update
    calls skips the per-call validation.  Keeps the tensors alive; `unbind()` frees the slot."""

    def __init__(self, ctx: "Odsgd", grads: Sequence[torch.Tensor], slot: int):
        self.ctx, self.tensors, self.slot = ctx, list(grads), slot

    def unbind(self) -> None:
        if self.slot >= 0:
            self.ctx._check(self.ctx._lib.odsgd_unbind_grads(self.ctx._h, self.slot))
            self.slot = -1

    def __del__(self):
        try:  # give the slot back when the table is dropped while its context is still alive
            if self.slot >= 0 and self.ctx._h:
                self.ctx._lib.odsgd_unbind_grads(self.ctx._h, self.slot)
        except Exception:
            pass

    def __len__(self) -> int:
        return len(self.tensors)

    def __iter__(self):
        return iter(self.tensors)


class Odsgd:
    """One context of the CUDA library (see include/odsgd.h for the semantics of each call)."""

    def __init__(self, w_a: torch.Tensor, v: Optional[torch.Tensor], *, n_workers: int, lr: float, local_lr: float,
                 momentum: float, wd: float, w_b: Optional[torch.Tensor] = None,
                 w_delayed: Optional[torch.Tensor] = None,
                 local: Optional[Sequence[Optional[torch.Tensor]]] = None,
                 tensor_offsets: Optional[Sequence[int]] = None, flags: int = 0):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        n = w_a.numel()
        self.n_params = n
        self.n_workers = n_workers
        self._keep: List[object] = [w_a, v, w_b, w_delayed, list(local) if local is not None else None]
        offs = list(tensor_offsets) if tensor_offsets is not None else [0, n]
        off_arr = (ctypes.c_size_t * len(offs))(*offs)
        d = _Desc()
        d.w_a = _dev_ptr(w_a, "w_a")
        d.w_b = _dev_ptr(w_b, "w_b", n)
        d.w_delayed = _dev_ptr(w_delayed, "w_delayed", n)
        d.v = _dev_ptr(v, "v", n)
        if local is not None:
            if len(local) != n_workers:
                raise ValueError("local: need one entry (tensor or None) per worker")
            tab = _ptr_table([_dev_ptr(t, f"local[{i}]", n) for i, t in enumerate(local)])
            d.local = ctypes.cast(tab, ctypes.POINTER(ctypes.c_void_p))
        d.n_params = n
        d.tensor_offsets = ctypes.cast(off_arr, ctypes.POINTER(ctypes.c_size_t))
        d.n_tensors = len(offs) - 1
        d.n_workers = n_workers
        d.lr, d.local_lr, d.momentum, d.wd = lr, local_lr, momentum, wd
        d.flags = flags
        with torch.cuda.device(w_a.device):
            rc = self._lib.odsgd_create(ctypes.byref(self._h), ctypes.byref(d))
        if rc != OK:
            msg = self._lib.odsgd_last_error(None).decode()
            self._h = ctypes.c_void_p()
            raise OdsgdError(rc, msg)
        self._device = w_a.device
        self._by_ptr = {t.data_ptr(): t for t in (w_a, w_b, w_delayed) if t is not None}
        if local is not None:
            self._by_ptr.update({t.data_ptr(): t for t in local if t is not None})
        self.n_tensors = len(offs) - 1

    # -- plumbing
    def _check(self, rc: int) -> None:
        if rc != OK:
            raise OdsgdError(rc, self._lib.odsgd_last_error(self._h).decode())

    def _grad_table(self, grads):
        if isinstance(grads, GradTable):
            if grads.n_workers != self.n_workers or grads.n_params != self.n_params:
                raise ValueError("gradient table was built for another context shape")
            return grads.table
        if len(grads) != self.n_workers:
            raise ValueError(f"need {self.n_workers} gradient tensors, got {len(grads)}")
        return _ptr_table([_dev_ptr(g, f"grads[{i}]", self.n_params) for i, g in enumerate(grads)])

    def grad_table(self, grads: Sequence[torch.Tensor]) -> "GradTable":
        """Checks the gradient tensors once and keeps their pointer table, for loops that pass
        the same buffers every iteration (saves the per-call marshalling, which dominates the
        cost of a step on small parameter sets)."""
        return GradTable(grads, self.n_workers, self.n_params)

    def bind_grads(self, grads: Sequence[torch.Tensor]) -> "BoundGrads":
        """odsgd_bind_grads: the library validates the table once; global_update / fused_update /
        ssgd_step / step_update then take the returned object in place of the tensor list."""
        slot = ctypes.c_int(-1)
        self._check(self._lib.odsgd_bind_grads(self._h, self._grad_table(grads), ctypes.byref(slot)))
        return BoundGrads(self, grads, slot.value)

    def _slot(self, grads: "BoundGrads") -> int:
        if grads.ctx is not self or grads.slot < 0:
            raise ValueError("gradient table is bound to another context, or was unbound")
        return grads.slot

    def close(self) -> None:
        if self._h:
            self._lib.odsgd_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the update calls
    def global_update(self, grads: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None) -> None:
        if isinstance(grads, BoundGrads):
            self._check(self._lib.odsgd_global_update_bound(self._h, self._slot(grads), _stream_handle(stream)))
        else:
            self._check(self._lib.odsgd_global_update(self._h, self._grad_table(grads), _stream_handle(stream)))
        self._bound = grads

    def local_update(self, worker_id: int, stream: Optional[torch.cuda.Stream] = None) -> None:
        self._check(self._lib.odsgd_local_update(self._h, worker_id, _stream_handle(stream)))

    def fused_update(self, grads: Sequence[torch.Tensor], worker_id: int,
                     stream: Optional[torch.cuda.Stream] = None) -> None:
        if isinstance(grads, BoundGrads):
            self._check(self._lib.odsgd_fused_update_bound(self._h, self._slot(grads), worker_id,
                                                           _stream_handle(stream)))
        else:
            self._check(self._lib.odsgd_fused_update(self._h, self._grad_table(grads), worker_id,
                                                     _stream_handle(stream)))
        self._bound = grads

    def fused_update_bound_raw(self, slot: int, worker_id: int, stream_handle: int) -> int:
        """odsgd_fused_update_bound with nothing around it: slot index and raw stream handle in,
        error code out (check it with `check`).  For loops where the marshalling of the regular
        wrapper is comparable to the kernel itself."""
        return self._lib.odsgd_fused_update_bound(self._h, slot, worker_id, stream_handle)

    def check(self, rc: int) -> None:
        self._check(rc)

    def worker_local_update(self, worker_id: int, w_bak: torch.Tensor, grad: torch.Tensor, no_delay: bool = False,
                            stream: Optional[torch.cuda.Stream] = None) -> None:
        """odsgd_worker_local_update: local[worker_id] = LocalRule(w_bak, grad) on explicit inputs."""
        self._check(self._lib.odsgd_worker_local_update(self._h, worker_id, _dev_ptr(w_bak, "w_bak", self.n_params),
                                                        _dev_ptr(grad, "grad", self.n_params), int(bool(no_delay)),
                                                        _stream_handle(stream)))

    def fused_update_host(self, host_grads: Sequence[torch.Tensor], dev_staging: Sequence[torch.Tensor],
                          worker_id: int, host_local_out: Optional[torch.Tensor] = None,
                          stream: Optional[torch.cuda.Stream] = None,
                          copy_stream: Optional[torch.cuda.Stream] = None) -> None:
        if len(host_grads) != self.n_workers:
            raise ValueError(f"need {self.n_workers} host gradient tensors")
        hp = []
        for i, t in enumerate(host_grads):
            if t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous() or t.numel() != self.n_params:
                raise TypeError(f"host_grads[{i}]: need a contiguous float32 CPU tensor of n_params elements")
            hp.append(t.data_ptr())
        out_ptr = None
        if host_local_out is not None:
            t = host_local_out
            if t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous() or t.numel() != self.n_params:
                raise TypeError("host_local_out: need a contiguous float32 CPU tensor of n_params elements")
            out_ptr = t.data_ptr()
        self._check(self._lib.odsgd_fused_update_host(self._h, _ptr_table(hp), self._grad_table(dev_staging),
                                                      worker_id, out_ptr, _stream_handle(stream),
                                                      copy_stream.cuda_stream if copy_stream is not None else None))
        self._bound = list(dev_staging)

    def ssgd_step(self, grads: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None) -> None:
        if isinstance(grads, BoundGrads):
            self._check(self._lib.odsgd_ssgd_step_bound(self._h, self._slot(grads), _stream_handle(stream)))
        else:
            self._check(self._lib.odsgd_ssgd_step(self._h, self._grad_table(grads), _stream_handle(stream)))

    def asgd_step(self, worker_id: int, grad: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
        self._check(self._lib.odsgd_asgd_step(self._h, worker_id, _dev_ptr(grad, "grad", self.n_params),
                                              _stream_handle(stream)))

    def dcasgd_step(self, worker_id: int, grad: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
        self._check(self._lib.odsgd_dcasgd_step(self._h, worker_id, _dev_ptr(grad, "grad", self.n_params),
                                                _stream_handle(stream)))

    def step_update(self, grads: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None) -> None:
        """odsgd_step: one iteration of Algorithm 2's state machine (warm-up SSGD, then OD-SGD)."""
        if isinstance(grads, BoundGrads):
            self._check(self._lib.odsgd_step_bound(self._h, self._slot(grads), _stream_handle(stream)))
        else:
            self._check(self._lib.odsgd_step(self._h, self._grad_table(grads), _stream_handle(stream)))
        self._bound = grads

    def set_warmup(self, wp: int) -> None:
        self._check(self._lib.odsgd_set_warmup(self._h, wp))

    def train_weights(self, worker_id: int) -> torch.Tensor:
        """The tensor worker `worker_id` computes its next gradient on."""
        p = ctypes.c_void_p()
        self._check(self._lib.odsgd_get_train_weights(self._h, worker_id, ctypes.byref(p)))
        return self._by_ptr[p.value]

    def set_tensor_multipliers(self, lr_mult: Optional[Sequence[float]], wd_mult: Optional[Sequence[float]],
                               stream: Optional[torch.cuda.Stream] = None) -> None:
        def arr(x):
            if x is None:
                return None
            if len(x) != self.n_tensors:
                raise ValueError(f"need {self.n_tensors} multipliers, got {len(x)}")
            return (ctypes.c_float * len(x))(*[float(t) for t in x])

        self._check(self._lib.odsgd_set_tensor_multipliers(self._h, arr(lr_mult), arr(wd_mult), _stream_handle(stream)))

    def fused_update_mult_static(self, grads: Sequence[torch.Tensor], worker_id: int,
                                 lr_mult: Optional[Sequence[float]], wd_mult: Optional[Sequence[float]],
                                 stream: Optional[torch.cuda.Stream] = None) -> None:
        """odsgd_fused_update_mult_static: the fused update with per-tensor multipliers for callers
        that may not allocate device memory.  The multiplier table goes into a fixed array inside
        the library instead of a cudaMalloc'ed one; all calls on a device share that array, so
        calls whose GPU work could overlap must be serialised.  Make the first call on a device
        outside any stream capture (it looks up the array's address)."""
        def arr(x):
            if x is None:
                return None
            if len(x) != self.n_tensors:
                raise ValueError(f"need {self.n_tensors} multipliers, got {len(x)}")
            return (ctypes.c_float * len(x))(*[float(t) for t in x])

        self._check(self._lib.odsgd_fused_update_mult_static(self._h, self._grad_table(grads), worker_id,
                                                             arr(lr_mult), arr(wd_mult), _stream_handle(stream)))
        self._bound = grads

    def set_weight_mirrors(self, mirrors_a: Optional[Sequence[torch.Tensor]],
                           mirrors_b: Optional[Sequence[torch.Tensor]] = None) -> None:
        """odsgd_set_weight_mirrors: tensors (n_params elements each; local or peer-mapped memory)
        that receive every weight the server pass writes into w_a (mirrors_a) / w_b (mirrors_b).
        None or an empty list switches the feature off."""
        if not mirrors_a:
            self._check(self._lib.odsgd_set_weight_mirrors(self._h, None, None, 0))
            self._mirrors = None
            return
        if mirrors_b is not None and len(mirrors_b) != len(mirrors_a):
            raise ValueError("mirrors_a and mirrors_b need the same number of entries")
        ta = _ptr_table([_dev_ptr(t, f"mirrors_a[{i}]", self.n_params) for i, t in enumerate(mirrors_a)])
        tb = None
        if mirrors_b is not None:
            tb = _ptr_table([_dev_ptr(t, f"mirrors_b[{i}]", self.n_params) for i, t in enumerate(mirrors_b)])
        self._check(self._lib.odsgd_set_weight_mirrors(self._h, ta, tb, len(mirrors_a)))
        self._mirrors = (list(mirrors_a), list(mirrors_b) if mirrors_b is not None else None)

    def set_server_mean_square(self, ms: Optional[torch.Tensor]) -> None:
        self._check(self._lib.odsgd_set_server_mean_square(self._h, _dev_ptr(ms, "mean_square", self.n_params)))
        self._keep.append(ms)

    # -- settings
    def set_lr(self, lr: float) -> None:
        self._check(self._lib.odsgd_set_lr(self._h, lr))

    def set_local_lr(self, local_lr: float) -> None:
        self._check(self._lib.odsgd_set_local_lr(self._h, local_lr))

    def set_momentum(self, momentum: float) -> None:
        self._check(self._lib.odsgd_set_momentum(self._h, momentum))

    def set_wd(self, wd: float) -> None:
        self._check(self._lib.odsgd_set_wd(self._h, wd))

    def set_local_rule(self, rule: int, lam: float = 0.0, m: float = 0.0, eps: float = 0.0,
                       mean_square: Optional[Sequence[Optional[torch.Tensor]]] = None) -> None:
        tab = None
        if mean_square is not None:
            if len(mean_square) != self.n_workers:
                raise ValueError("mean_square: need one entry (tensor or None) per worker")
            tab = _ptr_table([_dev_ptr(t, f"mean_square[{i}]", self.n_params) for i, t in enumerate(mean_square)])
        self._check(self._lib.odsgd_set_local_rule(self._h, rule, lam, m, eps, tab))
        self._keep.append(list(mean_square) if mean_square is not None else None)

    def set_launch_config(self, block_threads: int = 0, ctas_per_sm: int = 0) -> None:
        self._check(self._lib.odsgd_set_launch_config(self._h, block_threads, ctas_per_sm))

    # -- queries
    def weights(self) -> torch.Tensor:
        """The tensor that currently holds the global weights."""
        cur = ctypes.c_void_p()
        self._check(self._lib.odsgd_get_weights(self._h, ctypes.byref(cur), None))
        return self._by_ptr[cur.value]

    def delayed_weights(self) -> Optional[torch.Tensor]:
        """The tensor that holds the weights from before the latest global update, if kept."""
        dl = ctypes.c_void_p()
        self._check(self._lib.odsgd_get_weights(self._h, None, ctypes.byref(dl)))
        return self._by_ptr[dl.value] if dl.value else None

    @property
    def step(self) -> int:
        s = ctypes.c_uint64()
        self._check(self._lib.odsgd_get_step(self._h, ctypes.byref(s)))
        return s.value

    @step.setter
    def step(self, value: int) -> None:
        self._check(self._lib.odsgd_set_step(self._h, value))

    @property
    def iteration(self) -> int:
        """Iteration index of the Algorithm 2 state machine (odsgd_step calls so far)."""
        s = ctypes.c_uint64()
        self._check(self._lib.odsgd_get_iteration(self._h, ctypes.byref(s)))
        return s.value

    @iteration.setter
    def iteration(self, value: int) -> None:
        self._check(self._lib.odsgd_set_iteration(self._h, value))

    @property
    def launch_count(self) -> int:
        s = ctypes.c_uint64()
        self._check(self._lib.odsgd_get_launch_count(self._h, ctypes.byref(s)))
        return s.value


def version() -> int:
    return load_library().odsgd_version()


def shard_range(n_params: int, n_ranks: int, rank: int) -> tuple:
    """odsgd_shard_range: the slice [begin, end) of the arena that rank `rank` of `n_ranks` owns."""
    b, e = ctypes.c_size_t(), ctypes.c_size_t()
    rc = load_library().odsgd_shard_range(n_params, n_ranks, rank, ctypes.byref(b), ctypes.byref(e))
    if rc != OK:
        raise OdsgdError(rc, "odsgd_shard_range: n_ranks >= 1 and 0 <= rank < n_ranks are required")
    return b.value, e.value


# The C entry points under their own names, for callers that prefer the flat C style.
def odsgd_create(*args, **kwargs) -> Odsgd:
    return Odsgd(*args, **kwargs)


def odsgd_destroy(ctx: Odsgd) -> None:
    ctx.close()


def odsgd_global_update(ctx: Odsgd, worker_grads, stream=None) -> None:
    ctx.global_update(worker_grads, stream)


def odsgd_local_update(ctx: Odsgd, worker_id: int, stream=None) -> None:
    ctx.local_update(worker_id, stream)


def odsgd_fused_update(ctx: Odsgd, worker_grads, worker_id: int, stream=None) -> None:
    ctx.fused_update(worker_grads, worker_id, stream)


def odsgd_fused_update_host(ctx: Odsgd, host_grads, dev_staging, worker_id: int, host_local_out=None,
                            stream=None, copy_stream=None) -> None:
    ctx.fused_update_host(host_grads, dev_staging, worker_id, host_local_out, stream, copy_stream)


def odsgd_ssgd_step(ctx: Odsgd, worker_grads, stream=None) -> None:
    ctx.ssgd_step(worker_grads, stream)


def odsgd_asgd_step(ctx: Odsgd, worker_id: int, grad, stream=None) -> None:
    ctx.asgd_step(worker_id, grad, stream)


def odsgd_dcasgd_step(ctx: Odsgd, worker_id: int, grad, stream=None) -> None:
    ctx.dcasgd_step(worker_id, grad, stream)


def odsgd_step(ctx: Odsgd, worker_grads, stream=None) -> None:
    ctx.step_update(worker_grads, stream)


def odsgd_lr_step_decay(base_lr: float, factor: float, boundaries: Sequence[int], step: int) -> float:
    b = (ctypes.c_uint64 * len(boundaries))(*[int(x) for x in boundaries])
    return load_library().odsgd_lr_step_decay(base_lr, factor, b, len(boundaries), step)


def odsgd_lr_linear_ramp(start_lr: float, end_lr: float, ramp_steps: int, step: int) -> float:
    return load_library().odsgd_lr_linear_ramp(start_lr, end_lr, ramp_steps, step)


def odsgd_lr_poly_decay(base_lr: float, end_lr: float, power: float, total_steps: int, step: int) -> float:
    return load_library().odsgd_lr_poly_decay(base_lr, end_lr, power, total_steps, step)
