"""Helpers shared by the GPU tests: the CUDA library behind the pins' interface, guard bands,
and the floating-point comparison used when fused multiply-add is allowed."""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

from paper_2005_06728_b200 import binding
from pins import Impl

DEV = "cuda:0"
POISON = float.fromhex("0x1.fffffcp+100")  # a value no update produces by accident
GUARD = 64  # floats of guard band on each side of every arena

# Tolerance of the opt-in ODSGD_FLAG_ALLOW_FMA flavour, derived from its arithmetic.  It
# differs from the default one-rounding-per-operator evaluation only where the compiler contracts a
# multiply with the following add or subtract; each contraction removes one rounding of
# relative size 2**-24 of the product it swallows.  The server rule has three candidates
# (wd*w into d, lr*d or momentum*v into v', nothing into w' = w + v' but v' carries over), the
# local rule one.  So |gpu - oracle| <= 4 * 2**-24 * (sum of the magnitudes of the terms the
# element is built from) < 1e-6 * that sum.  Relative to the result itself the same
# difference is unbounded when the terms cancel (momentum*v against lr*d), which is why the
# scale is the sum of the terms, not the result.
REL_TOL = 1e-6


def dev_arena(x, guard: bool = True) -> Tuple[torch.Tensor, Optional[torch.Tensor]]:
    """Copies x to the device inside a poisoned guard band; returns (view, whole buffer)."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)) if not isinstance(x, torch.Tensor) else x
    t = t.reshape(-1).to(torch.float32)
    if not guard:
        return t.to(DEV).contiguous(), None
    n = t.numel()
    pad = (-n) % 4
    whole = torch.full((GUARD + n + pad + GUARD,), POISON, dtype=torch.float32, device=DEV)
    view = whole[GUARD:GUARD + n]
    view.copy_(t)
    return view, whole


def guards_intact(whole: Optional[torch.Tensor], n: int) -> bool:
    if whole is None:
        return True
    head, tail = whole[:GUARD], whole[GUARD + n:]
    return bool(torch.all(head == POISON)) and bool(torch.all(tail == POISON))


class GpuImpl(Impl):
    """The CUDA library driven through its C ABI, one fresh context per call."""

    def __init__(self, deterministic: bool = True, pingpong: bool = True, fused: bool = False):
        self.flags = binding.FLAG_DETERMINISTIC if deterministic else binding.FLAG_ALLOW_FMA
        self.pingpong = pingpong
        self.fused = fused

    def _ctx(self, w, v, n_workers, lr=0.0, local_lr=0.0, momentum=0.0, wd=0.0, local=None, keep_prev=True):
        self.bufs = []
        wa, b0 = dev_arena(w)
        va, b1 = dev_arena(v)
        self.bufs += [(b0, wa.numel()), (b1, va.numel())]
        wb = wd_ = None
        if keep_prev:
            other, b2 = dev_arena(np.zeros(wa.numel(), np.float32))
            self.bufs.append((b2, other.numel()))
            if self.pingpong:
                wb = other
            else:
                wd_ = other
        ctx = binding.Odsgd(wa, va, n_workers=n_workers, lr=lr, local_lr=local_lr, momentum=momentum,
                            wd=wd, w_b=wb, w_delayed=wd_, local=local, flags=self.flags)
        return ctx, va

    def _done(self):
        torch.cuda.synchronize()
        for whole, n in self.bufs:
            assert guards_intact(whole, n), "a kernel wrote outside its arena"

    def _grads(self, grads):
        out = []
        for g in grads:
            t, whole = dev_arena(g)
            self.bufs.append((whole, t.numel()))
            out.append(t)
        return out

    def global_update(self, grads, w, v, lr, momentum, wd):
        ctx, va = self._ctx(w, v, len(grads), lr=lr, momentum=momentum, wd=wd)
        gd = self._grads(grads)
        ctx.global_update(gd)
        self._done()
        res = (ctx.weights().cpu().numpy().copy(), va.cpu().numpy().copy(),
               ctx.delayed_weights().cpu().numpy().copy())
        assert all(np.array_equal(g.cpu().numpy(), np.asarray(h, np.float32), equal_nan=True)
                   for g, h in zip(gd, grads)), "gradients are read-only"
        ctx.close()
        return res

    def ssgd_step(self, grads, w, v, lr, momentum, wd):
        ctx, va = self._ctx(w, v, len(grads), lr=lr, momentum=momentum, wd=wd, keep_prev=False)
        ctx.ssgd_step(self._grads(grads))
        self._done()
        res = (ctx.weights().cpu().numpy().copy(), va.cpu().numpy().copy())
        ctx.close()
        return res

    def asgd_step(self, g, w, v, lr, momentum, wd):
        ctx, va = self._ctx(w, v, 3, lr=lr, momentum=momentum, wd=wd, keep_prev=False)
        ctx.asgd_step(1, self._grads([g])[0])
        self._done()
        res = (ctx.weights().cpu().numpy().copy(), va.cpu().numpy().copy())
        ctx.close()
        return res

    def _local(self, w_bak, g, local_lr, rule, x_prev=None, ms=None, lam=0.0, m=0.0, eps=0.0):
        # The library's local update always follows a global update: run one with lr = 0,
        # momentum = 0, wd = 0 and v = 0 (which leaves finite weights unchanged) and read the
        # local result, computed from the weights of before that update.
        n = np.asarray(w_bak).size
        x0 = np.zeros(n, np.float32) if x_prev is None else x_prev
        xl, bx = dev_arena(x0)
        local = [None, xl]
        ctx, _ = self._ctx(w_bak, np.zeros(n, np.float32), 2, local_lr=local_lr, local=local)
        self.bufs.append((bx, n))
        msd = None
        if rule != binding.LOCAL_SGD:
            if ms is not None:
                msd, bm = dev_arena(ms)
                self.bufs.append((bm, n))
            ctx.set_local_rule(rule, lam, m, eps, [None, msd] if msd is not None else None)
        gd = self._grads([np.zeros(n, np.float32), g])
        if self.fused:
            ctx.fused_update(gd, 1)
        else:
            ctx.global_update(gd)
            ctx.local_update(1)
        self._done()
        x = xl.cpu().numpy().copy()
        ms_out = msd.cpu().numpy().copy() if msd is not None else None
        ctx.close()
        return x, ms_out

    def local_update(self, w_bak, g, local_lr):
        return self._local(w_bak, g, local_lr, binding.LOCAL_SGD)[0]

    def local_update_dc_c(self, w_bak, g, x_prev, local_lr, lam):
        return self._local(w_bak, g, local_lr, binding.LOCAL_DC_C, x_prev=x_prev, lam=lam)[0]

    def local_update_dc_a(self, w_bak, g, x_prev, ms, local_lr, lam, m, eps):
        return self._local(w_bak, g, local_lr, binding.LOCAL_DC_A, x_prev=x_prev, ms=ms, lam=lam, m=m, eps=eps)


    def local_update_momentum(self, w_bak, g, u, local_lr, momentum, wd):
        return self._local(w_bak, g, local_lr, binding.LOCAL_MOMENTUM, ms=u, lam=wd, m=momentum)

    def global_update_mult(self, grads, w, v, lr, momentum, wd, offsets, lr_mult, wd_mult):
        self.bufs = []
        wa, b0 = dev_arena(w)
        va, b1 = dev_arena(v)
        other, b2 = dev_arena(np.zeros(wa.numel(), np.float32))
        self.bufs += [(b0, wa.numel()), (b1, wa.numel()), (b2, wa.numel())]
        vec_ok = all(int(o) % 4 == 0 for o in offsets)
        ctx = binding.Odsgd(wa, va, n_workers=len(grads), lr=lr, local_lr=0.0, momentum=momentum, wd=wd,
                            w_b=other if self.pingpong else None, w_delayed=None if self.pingpong else other,
                            tensor_offsets=[int(o) for o in offsets],
                            flags=self.flags | (0 if vec_ok else binding.FLAG_ALLOW_UNALIGNED))
        ctx.set_tensor_multipliers(list(map(float, lr_mult)), list(map(float, wd_mult)))
        ctx.global_update(self._grads(grads))
        self._done()
        res = (ctx.weights().cpu().numpy().copy(), va.cpu().numpy().copy(),
               ctx.delayed_weights().cpu().numpy().copy())
        ctx.close()
        return res

    def _dcasgd(self, g, w, bak, rule, lr, lam, ms=None, m=0.0, eps=0.0):
        self.bufs = []
        n = np.asarray(w).size
        wa, b0 = dev_arena(w)
        va, b1 = dev_arena(np.zeros(n, np.float32))
        bk, b2 = dev_arena(bak)
        self.bufs += [(b0, n), (b1, n), (b2, n)]
        ctx = binding.Odsgd(wa, va, n_workers=2, lr=lr, local_lr=123.0, momentum=0.9, wd=0.1,
                            local=[None, bk], flags=self.flags)
        ctx.set_local_rule(rule, lam, m, eps, None)
        msd = None
        if ms is not None:
            msd, b3 = dev_arena(ms)
            self.bufs.append((b3, n))
            ctx.set_server_mean_square(msd)
        ctx.dcasgd_step(1, self._grads([g])[0])
        self._done()
        res = (wa.cpu().numpy().copy(), bk.cpu().numpy().copy(),
               msd.cpu().numpy().copy() if msd is not None else None)
        ctx.close()
        return res

    def dcasgd_step_c(self, g, w, bak, lr, lam):
        return self._dcasgd(g, w, bak, binding.LOCAL_DC_C, lr, lam)[:2]

    def dcasgd_step_a(self, g, w, bak, ms, lr, lam, m, eps):
        return self._dcasgd(g, w, bak, binding.LOCAL_DC_A, lr, lam, ms=ms, m=m, eps=eps)


def same_bits(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    return (a.view(np.uint32) == b.view(np.uint32)) | (np.isnan(a) & np.isnan(b))


def assert_bits(a, b, what: str) -> None:
    ok = same_bits(np.asarray(a), np.asarray(b))
    if not ok.all():
        i = int(np.nonzero(~ok)[0][0])
        raise AssertionError(f"{what}: {int((~ok).sum())} of {ok.size} elements differ; first at {i}: "
                             f"{np.asarray(a)[i]!r} vs {np.asarray(b)[i]!r}")


def server_scales(grads: Sequence[np.ndarray], w, v, lr, momentum, wd) -> Tuple[np.ndarray, np.ndarray]:
    """Sum of the magnitudes of the terms v' and w' are built from (fp64), per element."""
    s = np.zeros(w.size, np.float64)
    for g in grads:
        s += np.abs(g.astype(np.float64))
    gbar = s / len(grads)
    sv = np.abs(momentum * v.astype(np.float64)) + lr * (gbar + np.abs(wd * w.astype(np.float64)))
    sw = np.abs(w.astype(np.float64)) + sv
    return sw, sv


def assert_close_scaled(got, ref, scale, what: str, tol: float = REL_TOL) -> float:
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    denom = np.maximum(np.abs(ref), scale)
    denom = np.where(denom == 0, 1.0, denom)
    err = np.abs(got - ref) / denom
    worst = float(np.max(err)) if err.size else 0.0
    assert worst <= tol, f"{what}: max scaled error {worst:.3e} > {tol:.1e}"
    return worst


def plain_relative_error(got, ref, offsets: Sequence[int]) -> Tuple[float, int]:
    """Error relative to max(|ref|, 1e-3 * RMS of the tensor the element belongs to); returns
    (maximum, number of elements above 1e-6).  Reported, not gated: see REL_TOL above."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    worst, over = 0.0, 0
    for a, b in zip(offsets[:-1], offsets[1:]):
        r = ref[a:b]
        rms = float(np.sqrt(np.mean(r * r))) if b > a else 0.0
        floor = 1e-3 * rms if rms > 0 else 1e-12
        e = np.abs(got[a:b] - r) / np.maximum(np.abs(r), floor)
        if e.size:
            worst = max(worst, float(e.max()))
            over += int((e > 1e-6).sum())
    return worst, over
