"""Checks that pin an implementation of the update rules to facts fixed outside it.

Each ``pin_*`` function takes an *implementation* (an object with the methods of
``Impl`` below) and raises AssertionError when the implementation disagrees with

* hand-worked examples stored under tests/golden/,
* closed forms of the trajectories on a diagonal quadratic objective,
* invariants that follow from the paper's description,
* an exact rational re-evaluation with explicit fp32 rounding.

The same pins run on the CPU oracle (tests/test_oracle_pins.py), on deliberately
wrong variants (which must fail), and on the CUDA library (tests/test_gpu_parity.py,
tests/test_gpu_ext.py).
"""
from __future__ import annotations

import os
from fractions import Fraction
from typing import Dict, List, Sequence, Tuple

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
F32 = np.float32


class Impl:
    """Functional interface every pinned implementation offers (numpy fp32 in, numpy fp32 out)."""

    def global_update(self, grads: Sequence[np.ndarray], w, v, lr, momentum, wd
                      ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """returns (w_new, v_new, w_prev)"""
        raise NotImplementedError

    def ssgd_step(self, grads, w, v, lr, momentum, wd) -> Tuple[np.ndarray, np.ndarray]:
        raise NotImplementedError

    def local_update(self, w_bak, g, local_lr) -> np.ndarray:
        raise NotImplementedError

    def asgd_step(self, g, w, v, lr, momentum, wd) -> Tuple[np.ndarray, np.ndarray]:
        raise NotImplementedError

    def local_update_dc_c(self, w_bak, g, x_prev, local_lr, lam) -> np.ndarray:
        raise NotImplementedError

    def local_update_dc_a(self, w_bak, g, x_prev, ms, local_lr, lam, m, eps
                          ) -> Tuple[np.ndarray, np.ndarray]:
        """returns (x, ms_new)"""
        raise NotImplementedError

    def local_update_momentum(self, w_bak, g, u, local_lr, momentum, wd) -> Tuple[np.ndarray, np.ndarray]:
        """returns (x, u_new)"""
        raise NotImplementedError

    def global_update_mult(self, grads, w, v, lr, momentum, wd, offsets, lr_mult, wd_mult
                           ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """returns (w_new, v_new, w_prev)"""
        raise NotImplementedError

    def dcasgd_step_c(self, g, w, bak, lr, lam) -> Tuple[np.ndarray, np.ndarray]:
        """returns (w_new, bak_new)"""
        raise NotImplementedError

    def dcasgd_step_a(self, g, w, bak, ms, lr, lam, m, eps) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """returns (w_new, bak_new, ms_new)"""
        raise NotImplementedError


def a32(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x, dtype=np.float32).reshape(-1))


def read_golden(name: str) -> Dict[str, np.ndarray]:
    out: Dict[str, np.ndarray] = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            key, vals = line.split(":", 1)
            out[key.strip()] = np.array([float(t) for t in vals.split()], dtype=np.float64)
    return out


def _same_bits(a: np.ndarray, b: np.ndarray) -> bool:
    a, b = a32(a), a32(b)
    nan = np.isnan(a) & np.isnan(b)
    return bool(np.all((a.view(np.uint32) == b.view(np.uint32)) | nan))


def assert_same_bits(a, b, what: str) -> None:
    if not _same_bits(a, b):
        a, b = a32(a), a32(b)
        bad = np.nonzero(~((a.view(np.uint32) == b.view(np.uint32)) | (np.isnan(a) & np.isnan(b))))[0]
        i = int(bad[0])
        raise AssertionError(f"{what}: {bad.size} elements differ, first at {i}: {a[i]!r} vs {b[i]!r}")


# ----------------------------------------------------------------- hand-worked example

def pin_worked_example(impl: Impl) -> None:
    g = read_golden("worked_example_p8.txt")
    lr1, lr2 = float(g["lr1"][0]), float(g["lr2"][0])
    llr, mu, wd = float(g["local_lr"][0]), float(g["momentum"][0]), float(g["wd"][0])
    w, v, g0, g1 = a32(g["w"]), a32(g["v"]), a32(g["g0"]), a32(g["g1"])
    w1, v1, wprev = impl.global_update([g0, g1], w.copy(), v.copy(), lr1, mu, wd)
    assert np.array_equal(w1, a32(g["w1"])), ("w after step 1", w1)
    assert np.array_equal(v1, a32(g["v1"])), ("v after step 1", v1)
    assert np.array_equal(wprev, w), ("weights kept for the workers", wprev)
    assert np.array_equal(impl.local_update(wprev, g0, llr), a32(g["x0"]))
    assert np.array_equal(impl.local_update(wprev, g1, llr), a32(g["x1"]))
    w2, v2, wprev2 = impl.global_update([g0, g1], w1.copy(), v1.copy(), lr2, mu, wd)
    assert np.array_equal(w2, a32(g["w2"])), ("w after step 2", w2)
    assert np.array_equal(v2, a32(g["v2"])), ("v after step 2", v2)
    assert np.array_equal(wprev2, w1)
    ws, vs = impl.ssgd_step([g0, g1], w.copy(), v.copy(), lr1, mu, wd)
    assert np.array_equal(ws, a32(g["w1"])) and np.array_equal(vs, a32(g["v1"]))
    wa, va = impl.asgd_step(g0, w.copy(), np.zeros(8, F32), 0.5, 0.0, 0.0)
    wa, va = impl.asgd_step(g1, wa, va, 0.5, 0.0, 0.0)
    assert np.array_equal(wa, a32(g["asgd_w"])), ("asgd w", wa)
    assert np.array_equal(va, a32(g["asgd_v"])), ("asgd v", va)


def pin_rounding_order(impl: Impl) -> None:
    g = read_golden("rounding_order.txt")
    z = np.zeros(1, F32)
    # A: four workers, fixed order, result 0
    grads = [a32([x]) for x in g["A_g"]]
    w1, v1, _ = impl.global_update(grads, z.copy(), z.copy(), 1.0, 0.0, 0.0)
    assert float(w1[0]) == -0.25 * float(g["A_sum"][0]), ("worker order / sum tree", w1)
    # B
    grads = [a32([x]) for x in g["B_g"]]
    w1, v1, _ = impl.global_update(grads, z.copy(), z.copy(), 1.0, 0.0, 0.0)
    assert float(w1[0]) == -0.5 * float(g["B_sum"][0])
    # C: wd*w rounds before it is added
    w = a32(g["C_w"])
    w1, v1, _ = impl.global_update([a32(g["C_g"])], w.copy(), z.copy(), 1.0, 0.0, float(g["C_wd"][0]))
    assert float(v1[0]) == 0.0 and float(w1[0]) == float(w[0]), ("separate rounding of wd*w", v1)
    wa, va = impl.asgd_step(a32(g["C_g"]), w.copy(), z.copy(), 1.0, 0.0, float(g["C_wd"][0]))
    assert float(va[0]) == 0.0 and float(wa[0]) == float(w[0])
    # E: sum first, scale once
    grads = [a32([x]) for x in g["E_g"]]
    w1, v1, _ = impl.global_update(grads, z.copy(), z.copy(), 1.0, 0.0, 0.0)
    assert w1[0] == -a32(g["E_mean"])[0] and w1[0] != 0.0, ("sum, then one multiply by 1/M", w1)
    # D: local_lr*g rounds before it is subtracted
    x = impl.local_update(a32(g["D_w_bak"]), a32(g["D_g"]), float(g["D_local_lr"][0]))
    assert float(x[0]) == float(g["D_x"][0]), ("separate rounding of local_lr*g", x)


def pin_dc_worked_example(impl: Impl) -> None:
    g = read_golden("dc_local_update.txt")
    x = impl.local_update_dc_c(a32(g["c_w_bak"]), a32(g["c_g"]), a32(g["c_x_prev"]),
                               float(g["c_eta"][0]), float(g["c_lambda"][0]))
    assert np.array_equal(x, a32(g["c_x"])), ("Eq. 4", x)
    x, ms = impl.local_update_dc_a(a32(g["a_w_bak"]), a32(g["a_g"]), a32(g["a_x_prev"]),
                                   a32(g["a_ms"]), float(g["a_eta"][0]), float(g["a_lambda"][0]),
                                   float(g["a_m"][0]), float(g["a_eps"][0]))
    assert np.array_equal(ms, a32(g["a_ms_new"])), ("Eq. 6", ms)
    assert np.array_equal(x, a32(g["a_x"])), ("Eq. 5", x)


# ----------------------------------------------------------------- closed forms on a quadratic
# Objective f(w) = 1/2 * sum_i a_i w_i^2, gradient a_i w_i; every worker sees the same gradient.

def _quadratic_setup(n: int = 64, seed: int = 5):
    rng = np.random.default_rng(seed)
    # curvatures and start point exactly representable in fp32, so that the closed forms
    # (evaluated in double) start from the very numbers the implementation sees
    a = rng.uniform(0.2, 3.0, n).astype(np.float32).astype(np.float64)
    w0 = rng.uniform(-2.0, 2.0, n).astype(np.float32).astype(np.float64)
    return a, w0


def pin_ssgd_quadratic_closed_form(impl: Impl, n_workers: int = 4, steps: int = 8) -> None:
    """Momentum SGD on a quadratic is a two-term linear recurrence,
    w_{k+1} = (1 + mu - eta*c) w_k - mu w_{k-1}, c = a + wd, w_1 = (1 - eta*c) w_0.
    Its solution is A r1^k + B r2^k with r1, r2 the roots of r^2 - (1+mu-eta*c) r + mu."""
    a, w0 = _quadratic_setup()
    for (eta, mu, wd) in ((0.1, 0.9, 0.01), (0.3, 0.5, 0.0), (0.05, 0.0, 0.1)):
        c = a + wd
        b = 1.0 + mu - eta * c
        disc = np.sqrt((b * b - 4.0 * mu).astype(np.complex128))
        r1, r2 = (b + disc) / 2.0, (b - disc) / 2.0
        assert np.all(np.abs(r1 - r2) > 1e-6)
        w = a32(w0)
        v = np.zeros_like(w)
        w0_32 = w.astype(np.float64)
        scale = np.abs(w0_32)
        for k in range(1, steps + 1):
            grad = a32(a.astype(F32) * w)
            w, v, _ = impl.global_update([grad] * n_workers, w, v, eta, mu, wd)
            Bk = ((1.0 - eta * c) * w0_32 - r1 * w0_32) / (r2 - r1)
            Ak = w0_32 - Bk
            expect = (Ak * r1 ** k + Bk * r2 ** k).real
            err = np.max(np.abs(w.astype(np.float64) - expect) / np.maximum(scale, 1e-3))
            assert err < 4e-6 * k, f"SSGD closed form, eta={eta} mu={mu} wd={wd}, step {k}: {err}"


def pin_odsgd_quadratic_matrix_form(impl: Impl, n_workers: int = 2, steps: int = 6) -> None:
    """OD-SGD with the gradient taken at the worker's local weights x (g = a*x):
        V' = mu V - eta (a x + wd W);  W' = W + V';  x' = W - eta_l a x
    (the worker's next weights start from W, the weights from BEFORE this server step).
    The state (W, V, x) therefore advances by a fixed 3x3 matrix per coordinate."""
    a, w0 = _quadratic_setup(seed=6)
    for (eta, eta_l, mu, wd) in ((0.1, 0.05, 0.9, 0.01), (0.2, 0.2, 0.5, 0.0), (0.15, 0.0, 0.3, 0.05)):
        W = a32(w0)
        V = np.zeros_like(W)
        x = W.copy()
        s0 = np.stack([W.astype(np.float64), np.zeros(W.size), W.astype(np.float64)])  # 3 x n
        for k in range(1, steps + 1):
            grad = a32(a.astype(F32) * x)
            W, V, Wprev = impl.global_update([grad] * n_workers, W, V, eta, mu, wd)
            x = impl.local_update(Wprev, grad, eta_l)
            for i in (0, 7, 31, 63):
                M = np.array([[1 - eta * wd, mu, -eta * a[i]],
                              [-eta * wd, mu, -eta * a[i]],
                              [1.0, 0.0, -eta_l * a[i]]])
                e = np.linalg.matrix_power(M, k) @ s0[:, i]
                got = np.array([W[i], V[i], x[i]], dtype=np.float64)
                tol = 6e-6 * k * max(1.0, abs(s0[0, i]))
                assert np.all(np.abs(got - e) < tol), \
                    f"OD-SGD matrix form (eta={eta}, eta_l={eta_l}) step {k} coord {i}: {got} vs {e}"


def pin_odsgd_special_cases(impl: Impl, steps: int = 6) -> None:
    a, w0 = _quadratic_setup(seed=8)
    # (i) mu = 0, wd = 0, eta_l = eta, one worker: the local prediction IS the new global
    # weight, so OD-SGD is plain gradient descent: W_k = (1 - eta a)^k W_0 and x_k = W_k.
    eta = 0.2
    W = a32(w0)
    V = np.zeros_like(W)
    x = W.copy()
    for k in range(1, steps + 1):
        grad = a32(a.astype(F32) * x)
        W, V, Wprev = impl.global_update([grad], W, V, eta, 0.0, 0.0)
        x = impl.local_update(Wprev, grad, eta)
        assert_same_bits(x, W, "eta_l = eta, mu = wd = 0, M = 1: local weights equal global weights")
        expect = (1.0 - eta * a) ** k * a32(w0).astype(np.float64)
        assert np.max(np.abs(W - expect)) < 2e-6 * k * 2.0
    # (ii) eta_l = 0: the worker trains on the one-step-old global weights,
    # W_{k+1} = W_k - eta a W_{k-1} (delayed gradient descent), x_{k+1} = W_k.
    W = a32(w0)
    V = np.zeros_like(W)
    x = W.copy()
    hist = [W.astype(np.float64), W.astype(np.float64)]  # W_{-1} := W_0 (x_0 = W_0)
    for k in range(1, steps + 1):
        grad = a32(a.astype(F32) * x)
        Wold = W.copy()
        W, V, Wprev = impl.global_update([grad, grad], W, V, eta, 0.0, 0.0)
        x = impl.local_update(Wprev, grad, 0.0)
        assert np.array_equal(x, Wold), "eta_l = 0 must hand back the delayed weights"
        expect = hist[-1] - eta * a * hist[-2]
        hist.append(expect)
        assert np.max(np.abs(W - expect)) < 4e-6 * k * 2.0


# ----------------------------------------------------------------- invariants

def pin_invariants(impl: Impl, seed: int = 21) -> None:
    rng = np.random.default_rng(seed)
    n = 257
    w = a32(rng.normal(0, 1, n))
    v = a32(rng.normal(0, 0.1, n))
    grads = [a32(rng.normal(0, 0.5, n)) for _ in range(5)]
    lr, mu, wd = 0.07, 0.9, 3e-3
    # one worker: the server step is plain momentum SGD on that gradient == the ASGD step
    w1, v1, wp = impl.global_update(grads[:1], w.copy(), v.copy(), lr, mu, wd)
    wa, va = impl.asgd_step(grads[0], w.copy(), v.copy(), lr, mu, wd)
    assert_same_bits(w1, wa, "M = 1 server step vs ASGD step (w)")
    assert_same_bits(v1, va, "M = 1 server step vs ASGD step (v)")
    assert_same_bits(wp, w, "backup weights are the weights before the update")
    # SSGD server == OD-SGD server
    w5, v5, _ = impl.global_update(grads, w.copy(), v.copy(), lr, mu, wd)
    ws, vs = impl.ssgd_step(grads, w.copy(), v.copy(), lr, mu, wd)
    assert_same_bits(w5, ws, "SSGD step vs OD-SGD server step (w)")
    assert_same_bits(v5, vs, "SSGD step vs OD-SGD server step (v)")
    # the update never moves the input gradients and depends on them: changing one worker changes w
    g2 = [g.copy() for g in grads]
    g2[3] = g2[3] + F32(1.0)
    w6, _, _ = impl.global_update(g2, w.copy(), v.copy(), lr, mu, wd)
    np.testing.assert_allclose(w6 - w5, -lr / 5.0, rtol=2e-4)
    # mean, not sum: M identical dyadic gradients give the same step as one
    gd = a32(np.round(rng.normal(0, 4, n) * 16) / 16)
    w8, v8, _ = impl.global_update([gd] * 8, w.copy(), v.copy(), lr, mu, wd)
    w1b, v1b, _ = impl.global_update([gd], w.copy(), v.copy(), lr, mu, wd)
    assert_same_bits(w8, w1b, "8 identical dyadic gradients vs one")
    # no momentum, no decay: M ASGD steps at lr/M == one SSGD step at lr (dyadic data: exactly)
    wq = a32(np.round(rng.normal(0, 4, n) * 16) / 16)
    gq = [a32(np.round(rng.normal(0, 4, n) * 16) / 16) for _ in range(4)]
    wsync, _, _ = impl.global_update(gq, wq.copy(), np.zeros(n, F32), 0.5, 0.0, 0.0)
    wasync, vasync = wq.copy(), np.zeros(n, F32)
    for gm in gq:
        wasync, vasync = impl.asgd_step(gm, wasync, vasync, 0.125, 0.0, 0.0)
    assert np.array_equal(wsync, wasync), "4 ASGD steps at lr/4 vs one SSGD step (dyadic)"
    # local update: zero local learning rate returns the delayed weights; it is linear in g
    x0 = impl.local_update(w, grads[0], 0.0)
    assert np.array_equal(x0, w)
    xa = impl.local_update(w, grads[0], 0.25)
    xb = impl.local_update(w, a32(-grads[0]), 0.25)
    np.testing.assert_allclose((xa.astype(np.float64) + xb) / 2, w, rtol=0, atol=2e-7 * 4)
    assert np.all((xa < w) == (grads[0] > 0)), "a positive gradient must lower the weight"
    # worker order matters only through rounding
    wr, _, _ = impl.global_update(grads[::-1], w.copy(), v.copy(), lr, mu, wd)
    assert np.max(np.abs(wr - w5)) < 1e-6


def pin_special_values(impl: Impl) -> None:
    inf, nan = np.inf, np.nan
    den = 1e-40  # subnormal in fp32; must not be flushed to zero
    w = a32([den, -den, 0.0, -0.0, 1.0, 1.0, inf, 1.0])
    v = a32([0.0, 0.0, 0.0, 0.0, 0.0, nan, 0.0, 0.0])
    g = a32([0.0, 0.0, 0.0, 0.0, nan, 0.0, 0.0, -inf])
    w1, v1, _ = impl.global_update([g, g], w.copy(), v.copy(), 1.0, 1.0, 0.0)
    assert w1[0] == F32(den) and w1[1] == F32(-den), "subnormal weights must survive"
    assert w1[0] != 0.0
    assert np.isnan(w1[4]) and np.isnan(w1[5]) and np.isnan(v1[4]) and np.isnan(v1[5])
    assert np.isnan(w1[6]), "wd * inf with wd = 0 is NaN in IEEE arithmetic"
    assert w1[7] == inf
    x = impl.local_update(w, a32([den] * 8), 0.5)
    half = F32(den) * F32(0.5)
    assert x[2] == -half and x[0] == F32(den) - half and x[0] != 0.0
    wa, va = impl.asgd_step(g, w.copy(), v.copy(), 1.0, 1.0, 0.0)
    assert wa[0] == F32(den) and np.isnan(wa[4]) and np.isnan(wa[5]) and wa[7] == inf


# ----------------------------------------------------------------- exact rational re-evaluation

def round_to_f32(q: Fraction) -> np.float32:
    """Correctly rounded (nearest, ties to even) binary32 value of an exact rational."""
    if q == 0:
        return F32(0.0)
    c = F32(float(q))  # close; may be off by one step through double rounding
    best = None
    for cand in (np.nextafter(c, F32(-np.inf)), c, np.nextafter(c, F32(np.inf))):
        if not np.isfinite(cand):
            continue
        err = abs(Fraction(float(cand)) - q)
        even = (int(np.array(cand, dtype=F32).view(np.uint32)) & 1) == 0
        key = (err, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, cand)
    return F32(best[1])


def _fr(x) -> Fraction:
    return Fraction(float(x))


def exact_global_update(grads, w, v, lr, mu, wd):
    """One op, one rounding, in the pinned order, on exact rationals."""
    lr, mu, wd = F32(lr), F32(mu), F32(wd)
    inv = round_to_f32(Fraction(1, len(grads)))
    wn, vn = np.empty_like(w), np.empty_like(v)
    for i in range(w.size):
        s = grads[0][i]
        for m in range(1, len(grads)):
            s = round_to_f32(_fr(s) + _fr(grads[m][i]))
        gbar = round_to_f32(_fr(s) * _fr(inv))
        decay = round_to_f32(_fr(wd) * _fr(w[i]))
        d = round_to_f32(_fr(gbar) + _fr(decay))
        keep = round_to_f32(_fr(mu) * _fr(v[i]))
        step = round_to_f32(_fr(lr) * _fr(d))
        vn[i] = round_to_f32(_fr(keep) - _fr(step))
        wn[i] = round_to_f32(_fr(w[i]) + _fr(vn[i]))
    return wn, vn


def pin_exact_rational(impl: Impl, seed: int = 33) -> None:
    rng = np.random.default_rng(seed)
    n = 48
    for M in (1, 3, 4, 7):
        w = a32(rng.normal(0, 1, n))
        v = a32(rng.normal(0, 0.1, n))
        grads = [a32(rng.normal(0, 0.3, n) * 10.0 ** rng.integers(-3, 2)) for _ in range(M)]
        lr, mu, wd = 0.1, 0.9, 1e-4
        wn, vn = exact_global_update(grads, w, v, lr, mu, wd)
        w1, v1, _ = impl.global_update(grads, w.copy(), v.copy(), lr, mu, wd)
        assert_same_bits(w1, wn, f"server step vs exact rationals (M={M}, w)")
        assert_same_bits(v1, vn, f"server step vs exact rationals (M={M}, v)")
    w = a32(rng.normal(0, 1, n))
    g = a32(rng.normal(0, 0.3, n))
    llr = F32(0.037)
    xe = np.array([round_to_f32(_fr(w[i]) - _fr(round_to_f32(_fr(llr) * _fr(g[i])))) for i in range(n)], F32)
    assert_same_bits(impl.local_update(w, g, float(llr)), xe, "local update vs exact rationals")


def pin_fp64_agreement(impl: Impl, f64_global, f64_local, seed: int = 44) -> None:
    """fp32 rules stay within a few fp32 ulps of the same rules evaluated in fp64."""
    rng = np.random.default_rng(seed)
    n = 4096
    w = a32(rng.normal(0, 1, n))
    v = a32(rng.normal(0, 0.01, n))
    grads = [a32(rng.normal(0, 1e-2, n)) for _ in range(8)]
    lr, mu, wd = 0.1, 0.9, 1e-4
    w1, v1, wp = impl.global_update(grads, w.copy(), v.copy(), lr, mu, wd)
    w64, v64 = w.astype(np.float64), v.astype(np.float64)
    f64_global([g.astype(np.float64) for g in grads], w64, v64, lr, mu, wd)
    assert np.max(np.abs(w1 - w64) / np.maximum(np.abs(w64), 1e-3)) < 1e-6
    assert np.max(np.abs(v1 - v64)) < 1e-6 * max(1e-3, np.max(np.abs(v64)))
    x = impl.local_update(w, grads[0], 0.1)
    x64 = f64_local(w.astype(np.float64), grads[0].astype(np.float64), 0.1)
    assert np.max(np.abs(x - x64) / np.maximum(np.abs(x64), 1e-3)) < 1e-6


# ----------------------------------------------------------------- delay-compensated updaters

def pin_dc_reductions(impl: Impl, seed: int = 55) -> None:
    rng = np.random.default_rng(seed)
    n = 300
    w = a32(rng.normal(0, 1, n))
    xp = a32(w + rng.normal(0, 0.05, n))
    g = a32(rng.normal(0, 0.5, n))
    ms = a32(rng.uniform(0.01, 1, n))
    # lambda = 0 -> plain SGD local update
    base = impl.local_update(w, g, 0.1)
    assert_same_bits(impl.local_update_dc_c(w, g, xp, 0.1, 0.0), base, "Eq. 4 with lambda = 0")
    xa, ms1 = impl.local_update_dc_a(w, g, xp, ms.copy(), 0.1, 0.0, 0.95, 1e-7)
    assert_same_bits(xa, base, "Eq. 5 with lambda = 0")
    # gradient computed on the very weights being updated -> no compensation
    assert_same_bits(impl.local_update_dc_c(w, g, w.copy(), 0.1, 2.0), base, "Eq. 4 with no delay")
    # Eq. 6 is a convex combination of the old mean square and g^2
    expect = 0.95 * ms.astype(np.float64) + 0.05 * g.astype(np.float64) ** 2
    np.testing.assert_allclose(ms1, expect, rtol=3e-7)
    # m = 0: mean square is g^2; with eps = 0, lambda/sqrt(g^2) * g*g = lambda*|g|
    xa0, ms0 = impl.local_update_dc_a(w, g, xp, ms.copy(), 0.1, 2.0, 0.0, 0.0)
    np.testing.assert_allclose(ms0, g.astype(np.float64) ** 2, rtol=2e-7)
    diff = w.astype(np.float64) - xp
    e = w - 0.1 * (g + 2.0 * np.abs(g.astype(np.float64)) * diff)
    np.testing.assert_allclose(xa0, e, rtol=0, atol=1e-6)
    # the compensation term points along (w_bak - x_prev): Taylor correction of the gradient
    xc = impl.local_update_dc_c(w, g, xp, 0.1, 2.0).astype(np.float64)
    e = w - 0.1 * (g + 2.0 * g.astype(np.float64) ** 2 * diff)
    np.testing.assert_allclose(xc, e, rtol=0, atol=1e-6)


# ----------------------------------------------------------------- per-tensor multipliers

def pin_multipliers(impl: Impl, seed: int = 66) -> None:
    """impl.global_update_mult(grads, w, v, lr, mu, wd, offsets, lr_mult, wd_mult) -> (w, v, w_prev)"""
    g = read_golden("per_tensor_multipliers.txt")
    offs = [int(o) for o in g["offsets"]]
    w1, v1, wp = impl.global_update_mult([a32(g["g0"]), a32(g["g1"])], a32(g["w"]), a32(g["v"]),
                                         float(g["lr"][0]), float(g["momentum"][0]), float(g["wd"][0]),
                                         offs, a32(g["lr_mult"]), a32(g["wd_mult"]))
    assert np.array_equal(w1, a32(g["w1"])), ("hand example, w", w1)
    assert np.array_equal(v1, a32(g["v1"])), ("hand example, v", v1)
    assert np.array_equal(wp, a32(g["w"]))
    # all multipliers 1: the plain rule, bit for bit; in general: tensor by tensor the plain
    # rule with that tensor's scaled hyper-parameters
    rng = np.random.default_rng(seed)
    sizes = [5, 64, 1, 300, 7, 2048]
    offs = np.concatenate([[0], np.cumsum(sizes)]).tolist()
    n = offs[-1]
    w, v = a32(rng.normal(0, 1, n)), a32(rng.normal(0, 0.1, n))
    grads = [a32(rng.normal(0, 0.3, n)) for _ in range(3)]
    lr, mu, wd = 0.07, 0.9, 2e-3
    ones = np.ones(len(sizes), F32)
    wa, va, _ = impl.global_update_mult(grads, w.copy(), v.copy(), lr, mu, wd, offs, ones, ones)
    wb, vb, _ = impl.global_update(grads, w.copy(), v.copy(), lr, mu, wd)
    assert_same_bits(wa, wb, "multipliers all 1 (w)")
    assert_same_bits(va, vb, "multipliers all 1 (v)")
    lm = a32([1.0, 0.5, 2.0, 0.1, 0.0, 1.5])
    wm = a32([1.0, 0.0, 0.0, 3.0, 1.0, 0.25])
    wa, va, _ = impl.global_update_mult(grads, w.copy(), v.copy(), lr, mu, wd, offs, lm, wm)
    for t, (a, b) in enumerate(zip(offs[:-1], offs[1:])):
        lr_t = float(F32(lr) * lm[t])
        wd_t = float(F32(wd) * wm[t])
        ws, vs, _ = impl.global_update([x[a:b].copy() for x in grads], w[a:b].copy(), v[a:b].copy(), lr_t, mu, wd_t)
        assert_same_bits(wa[a:b], ws, f"tensor {t} against the plain rule (w)")
        assert_same_bits(va[a:b], vs, f"tensor {t} against the plain rule (v)")
    a, b = offs[4], offs[5]  # lr_mult = 0: only momentum moves the weights
    np.testing.assert_array_equal(va[a:b], F32(mu) * v[a:b])


# ----------------------------------------------------------------- local SGD with momentum

def pin_local_momentum(impl: Impl, seed: int = 88) -> None:
    """impl.local_update_momentum(w_bak, g, u, local_lr, momentum, wd) -> (x, u_new)"""
    # the hand-worked server example, read as a local update: same rule, one gradient (gbar)
    g = read_golden("worked_example_p8.txt")
    gbar = a32((g["g0"] + g["g1"]) / 2)
    x, u1 = impl.local_update_momentum(a32(g["w"]), gbar, a32(g["v"]), float(g["lr1"][0]),
                                       float(g["momentum"][0]), float(g["wd"][0]))
    assert np.array_equal(x, a32(g["w1"])) and np.array_equal(u1, a32(g["v1"]))
    rng = np.random.default_rng(seed)
    n = 400
    w = a32(rng.normal(0, 1, n))
    u = a32(rng.normal(0, 0.05, n))
    gr = a32(rng.normal(0, 0.3, n))
    # it IS the server's rule on one gradient: the ASGD step on (w_bak, u)
    x, u1 = impl.local_update_momentum(w, gr, u.copy(), 0.07, 0.9, 2e-3)
    wa, va = impl.asgd_step(gr, w.copy(), u.copy(), 0.07, 0.9, 2e-3)
    assert_same_bits(x, wa, "local momentum rule vs the server rule on one gradient (weights)")
    assert_same_bits(u1, va, "local momentum rule vs the server rule on one gradient (velocity)")
    # no momentum, no decay: the plain compensation
    x0, u0 = impl.local_update_momentum(w, gr, u.copy(), 0.07, 0.0, 0.0)
    assert_same_bits(x0, impl.local_update(w, gr, 0.07), "momentum = wd = 0 reduces to x = w_bak - local_lr * g")
    np.testing.assert_array_equal(u0, -(F32(0.07) * gr))
    # the velocity carries over: two steps from u = 0 on a constant gradient move by (1 + (1 + mu)) * step
    z = np.zeros(n, F32)
    x1, ua = impl.local_update_momentum(w, gr, z, 0.5, 0.5, 0.0)
    x2, ub = impl.local_update_momentum(x1, gr, ua, 0.5, 0.5, 0.0)
    np.testing.assert_allclose(x2, w - 0.5 * gr * 2.5, rtol=0, atol=2e-6)


# ----------------------------------------------------------------- DC-ASGD at the server

def pin_dcasgd_server(impl: Impl, seed: int = 77) -> None:
    """impl.dcasgd_step_c(g, w, bak, lr, lam) -> (w, bak);
    impl.dcasgd_step_a(g, w, bak, ms, lr, lam, m, eps) -> (w, bak, ms)"""
    g = read_golden("dc_local_update.txt")
    # same arithmetic as the worker-side rule with (w, backup) in the roles (w_bak, x_prev)
    w1, bak1 = impl.dcasgd_step_c(a32(g["c_g"]), a32(g["c_w_bak"]), a32(g["c_x_prev"]),
                                  float(g["c_eta"][0]), float(g["c_lambda"][0]))
    assert np.array_equal(w1, a32(g["c_x"])), ("Eq. 4 at the server", w1)
    assert np.array_equal(bak1, w1), "the worker pulls the new weights after its gradient is applied"
    w1, bak1, ms1 = impl.dcasgd_step_a(a32(g["a_g"]), a32(g["a_w_bak"]), a32(g["a_x_prev"]), a32(g["a_ms"]),
                                       float(g["a_eta"][0]), float(g["a_lambda"][0]), float(g["a_m"][0]),
                                       float(g["a_eps"][0]))
    assert np.array_equal(w1, a32(g["a_x"])) and np.array_equal(ms1, a32(g["a_ms_new"]))
    assert np.array_equal(bak1, w1)
    rng = np.random.default_rng(seed)
    n = 500
    w = a32(rng.normal(0, 1, n))
    bak = a32(w + rng.normal(0, 0.05, n))
    gr = a32(rng.normal(0, 0.5, n))
    # lambda = 0, or a worker that is not behind: plain SGD, i.e. the ASGD step without momentum and decay
    plain, _ = impl.asgd_step(gr, w.copy(), np.zeros(n, F32), 0.1, 0.0, 0.0)
    w1, _ = impl.dcasgd_step_c(gr, w.copy(), bak.copy(), 0.1, 0.0)
    assert_same_bits(w1, plain, "lambda = 0")
    w1, b1 = impl.dcasgd_step_c(gr, w.copy(), w.copy(), 0.1, 2.0)
    assert_same_bits(w1, plain, "no delay")
    # bit-identical to the (separately pinned) worker-side rule
    w1, b1 = impl.dcasgd_step_c(gr, w.copy(), bak.copy(), 0.1, 2.0)
    assert_same_bits(w1, impl.local_update_dc_c(w, gr, bak, 0.1, 2.0), "server rule vs worker rule, Eq. 4")
    ms = a32(rng.uniform(0.01, 1, n))
    w1, b1, ms1 = impl.dcasgd_step_a(gr, w.copy(), bak.copy(), ms.copy(), 0.1, 2.0, 0.95, 1e-7)
    xe, mse = impl.local_update_dc_a(w, gr, bak, ms.copy(), 0.1, 2.0, 0.95, 1e-7)
    assert_same_bits(w1, xe, "server rule vs worker rule, Eq. 5")
    assert_same_bits(ms1, mse, "Eq. 6 state")
    assert_same_bits(b1, w1, "backup after the step")
    # two workers taking turns: the one that pulled last is not behind
    wa, ba = impl.dcasgd_step_c(gr, w.copy(), w.copy(), 0.1, 2.0)       # worker 0, fresh
    g2 = a32(rng.normal(0, 0.5, n))
    wb, bb = impl.dcasgd_step_c(g2, wa.copy(), w.copy(), 0.1, 2.0)      # worker 1 still holds w
    diff = wa.astype(np.float64) - w
    expect = wa - 0.1 * (g2 + 2.0 * g2.astype(np.float64) ** 2 * diff)
    np.testing.assert_allclose(wb, expect, rtol=0, atol=1e-6)


CORE_PINS = (pin_worked_example, pin_rounding_order, pin_ssgd_quadratic_closed_form,
             pin_odsgd_quadratic_matrix_form, pin_odsgd_special_cases, pin_invariants,
             pin_special_values, pin_exact_rational)
DC_PINS = (pin_dc_worked_example, pin_dc_reductions)
EXT_PINS = (pin_multipliers, pin_dcasgd_server, pin_local_momentum)
