"""Pins the CPU oracle to facts fixed outside it, and shows the pins have teeth.

Nothing here needs a GPU.  The wrong variants further down are planted on the
CPU: each is a plausible slip (a dropped term, a wrong sign, the wrong weight
vector, a different summation order) and each must be rejected by a pin.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.filterwarnings("ignore::RuntimeWarning")

import oracle
import pins
from pins import F32, Impl, a32


class OracleImpl(Impl):
    def global_update(self, grads, w, v, lr, momentum, wd):
        w, v = w.copy(), v.copy()
        wp = np.empty_like(w)
        oracle.global_update(list(grads), w, v, lr=lr, momentum=momentum, wd=wd, w_prev=wp)
        return w, v, wp

    def ssgd_step(self, grads, w, v, lr, momentum, wd):
        w, v = w.copy(), v.copy()
        oracle.ssgd_step(list(grads), w, v, lr=lr, momentum=momentum, wd=wd)
        return w, v

    def local_update(self, w_bak, g, local_lr):
        return oracle.local_update(w_bak, g, local_lr=local_lr)

    def asgd_step(self, g, w, v, lr, momentum, wd):
        w, v = w.copy(), v.copy()
        oracle.asgd_step(g, w, v, lr=lr, momentum=momentum, wd=wd)
        return w, v

    def local_update_dc_c(self, w_bak, g, x_prev, local_lr, lam):
        return oracle.local_update_dc_c(w_bak, g, x_prev, local_lr=local_lr, lam=lam)

    def local_update_dc_a(self, w_bak, g, x_prev, ms, local_lr, lam, m, eps):
        ms = ms.copy()
        x = oracle.local_update_dc_a(w_bak, g, x_prev, ms, local_lr=local_lr, lam=lam, m=m, eps=eps)
        return x, ms


    def local_update_momentum(self, w_bak, g, u, local_lr, momentum, wd):
        u = u.copy()
        x = oracle.local_update_momentum(w_bak, g, u, local_lr=local_lr, momentum=momentum, wd=wd)
        return x, u

    def global_update_mult(self, grads, w, v, lr, momentum, wd, offsets, lr_mult, wd_mult):
        w, v = w.copy(), v.copy()
        wp = np.empty_like(w)
        oracle.global_update_mult(list(grads), w, v, lr=lr, momentum=momentum, wd=wd, offsets=offsets,
                                  lr_mult=lr_mult, wd_mult=wd_mult, w_prev=wp)
        return w, v, wp

    def dcasgd_step_c(self, g, w, bak, lr, lam):
        w, bak = w.copy(), bak.copy()
        oracle.dcasgd_step_c(g, w, bak, lr=lr, lam=lam)
        return w, bak

    def dcasgd_step_a(self, g, w, bak, ms, lr, lam, m, eps):
        w, bak, ms = w.copy(), bak.copy(), ms.copy()
        oracle.dcasgd_step_a(g, w, bak, ms, lr=lr, lam=lam, m=m, eps=eps)
        return w, bak, ms


class NumpyImpl(Impl):
    """The rules restated with numpy fp32 array ops; the base the wrong variants are cut from."""

    def _server(self, gbar, w, v, lr, mu, wd):
        lr, mu, wd = F32(lr), F32(mu), F32(wd)
        d = gbar + wd * w
        vn = mu * v - lr * d
        return w + vn, vn

    def _sum(self, grads):
        s = grads[0].copy()
        for g in grads[1:]:
            s = s + g
        return s

    def global_update(self, grads, w, v, lr, momentum, wd):
        gbar = self._sum(grads) * (F32(1.0) / F32(len(grads)))
        wn, vn = self._server(gbar, w, v, lr, momentum, wd)
        return wn, vn, w.copy()

    def ssgd_step(self, grads, w, v, lr, momentum, wd):
        return self.global_update(grads, w, v, lr, momentum, wd)[:2]

    def local_update(self, w_bak, g, local_lr):
        return w_bak - F32(local_lr) * g

    def asgd_step(self, g, w, v, lr, momentum, wd):
        return self._server(g, w, v, lr, momentum, wd)

    def local_update_dc_c(self, w_bak, g, x_prev, local_lr, lam):
        return w_bak - F32(local_lr) * (g + (F32(lam) * (g * g)) * (w_bak - x_prev))

    def local_update_dc_a(self, w_bak, g, x_prev, ms, local_lr, lam, m, eps):
        ms = F32(m) * ms + (F32(1.0) - F32(m)) * (g * g)
        lam_t = F32(lam) / np.sqrt(ms + F32(eps))
        return w_bak - F32(local_lr) * (g + (lam_t * (g * g)) * (w_bak - x_prev)), ms


    def local_update_momentum(self, w_bak, g, u, local_lr, momentum, wd):
        x, un = self._server(g, w_bak, u, local_lr, momentum, wd)
        return x, un

    def global_update_mult(self, grads, w, v, lr, momentum, wd, offsets, lr_mult, wd_mult):
        gbar = self._sum(grads) * (F32(1.0) / F32(len(grads)))
        lr_e, wd_e = np.empty_like(w), np.empty_like(w)
        for t, (a, b) in enumerate(zip(offsets[:-1], offsets[1:])):
            lr_e[a:b] = F32(lr) * lr_mult[t]
            wd_e[a:b] = F32(wd) * wd_mult[t]
        d = gbar + wd_e * w
        vn = F32(momentum) * v - lr_e * d
        return w + vn, vn, w.copy()

    def dcasgd_step_c(self, g, w, bak, lr, lam):
        wn = self.local_update_dc_c(w, g, bak, lr, lam)
        return wn, wn.copy()

    def dcasgd_step_a(self, g, w, bak, ms, lr, lam, m, eps):
        wn, msn = self.local_update_dc_a(w, g, bak, ms, lr, lam, m, eps)
        return wn, wn.copy(), msn


ORACLE = OracleImpl()


@pytest.mark.parametrize("pin", pins.CORE_PINS + pins.DC_PINS + pins.EXT_PINS, ids=lambda f: f.__name__)
def test_oracle_pin(pin):
    pin(ORACLE)


def test_oracle_close_to_fp64_rules():
    def g64(grads, w, v, lr, mu, wd):
        oracle.global_update_f64(grads, w, v, lr=lr, momentum=mu, wd=wd)

    def l64(w, g, llr):
        return oracle.local_update_f64(w, g, local_lr=llr)

    pins.pin_fp64_agreement(ORACLE, g64, l64)


def test_fp64_asgd_twin_matches_one_worker_server_step():
    rng = np.random.default_rng(3)
    w, v, g = (rng.normal(size=100) for _ in range(3))
    w1, v1 = w.copy(), v.copy()
    oracle.asgd_step_f64(g, w1, v1, lr=0.1, momentum=0.9, wd=1e-3)
    w2, v2 = w.copy(), v.copy()
    oracle.global_update_f64([g], w2, v2, lr=0.1, momentum=0.9, wd=1e-3)
    np.testing.assert_allclose(w1, w2, rtol=1e-15)
    np.testing.assert_allclose(v1, v2, rtol=1e-15)


@pytest.mark.parametrize("pin", pins.CORE_PINS + pins.DC_PINS + pins.EXT_PINS, ids=lambda f: f.__name__)
def test_numpy_restatement_passes_too(pin):
    pin(NumpyImpl())


def test_oracle_equals_numpy_restatement_bitwise():
    rng = np.random.default_rng(9)
    n = 10_001
    w, v = a32(rng.normal(size=n)), a32(rng.normal(size=n) * 0.1)
    grads = [a32(rng.normal(size=n) * 0.01) for _ in range(6)]
    a, b = ORACLE.global_update(grads, w, v, 0.1, 0.9, 1e-4), NumpyImpl().global_update(grads, w, v, 0.1, 0.9, 1e-4)
    for x, y, nm in zip(a, b, ("w", "v", "w_prev")):
        pins.assert_same_bits(x, y, nm)
    pins.assert_same_bits(ORACLE.local_update(w, grads[2], 0.03), NumpyImpl().local_update(w, grads[2], 0.03), "x")


# ------------------------------------------------------------------ planted mistakes

class SumNotMean(NumpyImpl):
    def global_update(self, grads, w, v, lr, momentum, wd):
        wn, vn = self._server(self._sum(grads), w, v, lr, momentum, wd)
        return wn, vn, w.copy()


class DecaySignFlipped(NumpyImpl):
    def _server(self, gbar, w, v, lr, mu, wd):
        return super()._server(gbar, w, v, lr, mu, -wd)


class DecayDropped(NumpyImpl):
    def _server(self, gbar, w, v, lr, mu, wd):
        return super()._server(gbar, w, v, lr, mu, 0.0)


class DecayOnNewWeights(NumpyImpl):
    # decoupled-style decay: applied to the weights, outside the momentum buffer
    def _server(self, gbar, w, v, lr, mu, wd):
        lr, mu, wd = F32(lr), F32(mu), F32(wd)
        vn = mu * v - lr * gbar
        return w + vn - lr * wd * w, vn


class MomentumOnWholeStep(NumpyImpl):
    def _server(self, gbar, w, v, lr, mu, wd):
        lr, mu, wd = F32(lr), F32(mu), F32(wd)
        vn = mu * (v - lr * (gbar + wd * w))
        return w + vn, vn


class WeightStepSignFlipped(NumpyImpl):
    def _server(self, gbar, w, v, lr, mu, wd):
        wn, vn = super()._server(gbar, w, v, lr, mu, wd)
        return w - vn, vn


class LrOutsideVelocity(NumpyImpl):
    # v accumulates raw gradients, lr applied at the weight step
    def _server(self, gbar, w, v, lr, mu, wd):
        lr, mu, wd = F32(lr), F32(mu), F32(wd)
        vn = mu * v + (gbar + wd * w)
        return w - lr * vn, vn


class DampenedMomentum(NumpyImpl):
    def _server(self, gbar, w, v, lr, mu, wd):
        lr, mu, wd = F32(lr), F32(mu), F32(wd)
        vn = mu * v - (F32(1) - mu) * lr * (gbar + wd * w)
        return w + vn, vn


class ReverseWorkerOrder(NumpyImpl):
    def _sum(self, grads):
        return super()._sum(grads[::-1])


class PairwiseTreeSum(NumpyImpl):
    def _sum(self, grads):
        g = [x.copy() for x in grads]
        while len(g) > 1:
            g = [g[i] + g[i + 1] if i + 1 < len(g) else g[i] for i in range(0, len(g), 2)]
        return g[0]


class DivideEachThenSum(NumpyImpl):
    def global_update(self, grads, w, v, lr, momentum, wd):
        inv = F32(1.0) / F32(len(grads))
        s = grads[0] * inv
        for g in grads[1:]:
            s = s + g * inv
        wn, vn = self._server(s, w, v, lr, momentum, wd)
        return wn, vn, w.copy()


class FusedDecay(NumpyImpl):
    # wd*w + gbar with a single rounding, as a fused multiply-add would do
    def _server(self, gbar, w, v, lr, mu, wd):
        d = (np.float64(F32(wd)) * w.astype(np.float64) + gbar.astype(np.float64)).astype(F32)
        vn = F32(mu) * v - F32(lr) * d
        return w + vn, vn


class BackupIsNewWeights(NumpyImpl):
    # hands the workers the weights AFTER the server step
    def global_update(self, grads, w, v, lr, momentum, wd):
        wn, vn, _ = super().global_update(grads, w, v, lr, momentum, wd)
        return wn, vn, wn.copy()


class LocalSignFlipped(NumpyImpl):
    def local_update(self, w_bak, g, local_lr):
        return w_bak + F32(local_lr) * g


class LocalFused(NumpyImpl):
    def local_update(self, w_bak, g, local_lr):
        return (w_bak.astype(np.float64) - np.float64(F32(local_lr)) * g.astype(np.float64)).astype(F32)


class LocalWithDecay(NumpyImpl):
    def local_update(self, w_bak, g, local_lr):
        return w_bak - F32(local_lr) * (g + F32(1e-2) * w_bak)


class AsgdAveraged(NumpyImpl):
    def asgd_step(self, g, w, v, lr, momentum, wd):
        return self._server(g * F32(0.5), w, v, lr, momentum, wd)


class FlushDenormals(NumpyImpl):
    @staticmethod
    def _ftz(x):
        x = x.copy()
        x[np.abs(x) < F32(1.1754944e-38)] = 0.0
        return x

    def global_update(self, grads, w, v, lr, momentum, wd):
        wn, vn, wp = super().global_update(grads, w, v, lr, momentum, wd)
        return self._ftz(wn), self._ftz(vn), wp

    def local_update(self, w_bak, g, local_lr):
        return self._ftz(super().local_update(w_bak, g, local_lr))


CORE_MUTANTS = [SumNotMean, DecaySignFlipped, DecayDropped, DecayOnNewWeights, MomentumOnWholeStep,
                WeightStepSignFlipped, LrOutsideVelocity, DampenedMomentum, ReverseWorkerOrder,
                PairwiseTreeSum, DivideEachThenSum, FusedDecay, BackupIsNewWeights,
                LocalSignFlipped, LocalFused, LocalWithDecay, AsgdAveraged, FlushDenormals]


def _rejected_by(impl, pin_list):
    caught = []
    for pin in pin_list:
        try:
            pin(impl)
        except AssertionError:
            caught.append(pin.__name__)
    return caught


@pytest.mark.parametrize("mutant", CORE_MUTANTS, ids=lambda c: c.__name__)
def test_planted_mistake_is_caught(mutant):
    caught = _rejected_by(mutant(), pins.CORE_PINS)
    assert caught, f"{mutant.__name__} slipped through every pin"


def test_closed_forms_alone_catch_the_arithmetic_mistakes():
    """The hand-worked example is not the only line of defence: closed forms and invariants,
    which are independent of it, reject the non-rounding mistakes on their own."""
    independent = (pins.pin_ssgd_quadratic_closed_form, pins.pin_odsgd_quadratic_matrix_form,
                   pins.pin_odsgd_special_cases, pins.pin_invariants)
    for mutant in (SumNotMean, DecaySignFlipped, DecayDropped, MomentumOnWholeStep,
                   WeightStepSignFlipped, DampenedMomentum, BackupIsNewWeights, LocalSignFlipped,
                   LocalWithDecay, AsgdAveraged):
        assert _rejected_by(mutant(), independent), mutant.__name__


class DcDiffSignFlipped(NumpyImpl):
    def local_update_dc_c(self, w_bak, g, x_prev, local_lr, lam):
        return super().local_update_dc_c(w_bak, g, 2 * w_bak - x_prev, local_lr, lam)

    def local_update_dc_a(self, w_bak, g, x_prev, ms, local_lr, lam, m, eps):
        return super().local_update_dc_a(w_bak, g, 2 * w_bak - x_prev, ms, local_lr, lam, m, eps)


class DcGradNotSquared(NumpyImpl):
    def local_update_dc_c(self, w_bak, g, x_prev, local_lr, lam):
        return w_bak - F32(local_lr) * (g + (F32(lam) * g) * (w_bak - x_prev))


class DcMeanSquareUsedBeforeUpdate(NumpyImpl):
    def local_update_dc_a(self, w_bak, g, x_prev, ms, local_lr, lam, m, eps):
        ms_new = F32(m) * ms + (F32(1.0) - F32(m)) * (g * g)
        lam_t = F32(lam) / np.sqrt(ms + F32(eps))
        return w_bak - F32(local_lr) * (g + (lam_t * (g * g)) * (w_bak - x_prev)), ms_new


class DcMeanSquareNoComplement(NumpyImpl):
    def local_update_dc_a(self, w_bak, g, x_prev, ms, local_lr, lam, m, eps):
        ms = F32(m) * ms + (g * g)
        lam_t = F32(lam) / np.sqrt(ms + F32(eps))
        return w_bak - F32(local_lr) * (g + (lam_t * (g * g)) * (w_bak - x_prev)), ms


class DcEpsOutsideRoot(NumpyImpl):
    def local_update_dc_a(self, w_bak, g, x_prev, ms, local_lr, lam, m, eps):
        ms = F32(m) * ms + (F32(1.0) - F32(m)) * (g * g)
        lam_t = F32(lam) / (np.sqrt(ms) + F32(eps))
        return w_bak - F32(local_lr) * (g + (lam_t * (g * g)) * (w_bak - x_prev)), ms


@pytest.mark.parametrize("mutant", [DcDiffSignFlipped, DcGradNotSquared, DcMeanSquareUsedBeforeUpdate,
                                    DcMeanSquareNoComplement, DcEpsOutsideRoot],
                         ids=lambda c: c.__name__)
def test_planted_dc_mistake_is_caught(mutant):
    assert _rejected_by(mutant(), pins.DC_PINS), f"{mutant.__name__} slipped through"


class MultSwapped(NumpyImpl):
    def global_update_mult(self, grads, w, v, lr, momentum, wd, offsets, lr_mult, wd_mult):
        return super().global_update_mult(grads, w, v, lr, momentum, wd, offsets, wd_mult, lr_mult)


class MultOffByOneTensor(NumpyImpl):
    def global_update_mult(self, grads, w, v, lr, momentum, wd, offsets, lr_mult, wd_mult):
        return super().global_update_mult(grads, w, v, lr, momentum, wd, offsets, np.roll(lr_mult, 1), np.roll(wd_mult, 1))


class MultOnVelocityToo(NumpyImpl):
    def global_update_mult(self, grads, w, v, lr, momentum, wd, offsets, lr_mult, wd_mult):
        wn, vn, wp = super().global_update_mult(grads, w, v, lr, momentum, wd, offsets, lr_mult, wd_mult)
        scale = np.empty_like(w)
        for t, (a, b) in enumerate(zip(offsets[:-1], offsets[1:])):
            scale[a:b] = lr_mult[t]
        return w + scale * vn, vn, wp


class LocalMomentumFromNewVelocityOnly(NumpyImpl):
    def local_update_momentum(self, w_bak, g, u, local_lr, momentum, wd):
        x, un = super().local_update_momentum(w_bak, g, u, local_lr, momentum, wd)
        return w_bak - F32(local_lr) * g, un  # forgets the velocity in the weights


class LocalMomentumDecayOnX(NumpyImpl):
    def local_update_momentum(self, w_bak, g, u, local_lr, momentum, wd):
        x, un = super().local_update_momentum(w_bak, g, u, local_lr, momentum, 0.0)
        return x - F32(local_lr) * F32(wd) * w_bak, un


class DcasgdBackupNotRefreshed(NumpyImpl):
    def dcasgd_step_c(self, g, w, bak, lr, lam):
        return self.local_update_dc_c(w, g, bak, lr, lam), bak.copy()

    def dcasgd_step_a(self, g, w, bak, ms, lr, lam, m, eps):
        wn, msn = self.local_update_dc_a(w, g, bak, ms, lr, lam, m, eps)
        return wn, bak.copy(), msn


class DcasgdRolesSwapped(NumpyImpl):
    def dcasgd_step_c(self, g, w, bak, lr, lam):
        wn = w - F32(lr) * (g + (F32(lam) * (g * g)) * (bak - w))
        return wn, wn.copy()


@pytest.mark.parametrize("mutant", [MultSwapped, MultOffByOneTensor, MultOnVelocityToo, DcasgdBackupNotRefreshed,
                                    DcasgdRolesSwapped, LocalMomentumFromNewVelocityOnly, LocalMomentumDecayOnX],
                         ids=lambda c: c.__name__)
def test_planted_ext_mistake_is_caught(mutant):
    assert _rejected_by(mutant(), pins.EXT_PINS), f"{mutant.__name__} slipped through"


def test_round_to_f32_is_correctly_rounded():
    from fractions import Fraction

    one = Fraction(1)
    ulp = Fraction(1, 2 ** 23)
    assert pins.round_to_f32(one + ulp / 2) == F32(1.0)                   # tie -> even
    assert pins.round_to_f32(one + ulp + ulp / 2) == F32(1.0) + F32(2.0 ** -22)  # tie -> even (up)
    assert pins.round_to_f32(one + ulp / 2 + Fraction(1, 2 ** 80)) == np.nextafter(F32(1), F32(2))
    assert pins.round_to_f32(Fraction(1, 3)) == F32(1.0) / F32(3.0)
    assert pins.round_to_f32(Fraction(1, 10)) == F32(0.1)
