"""Randomised checks of the CPU oracle against the exact-rational evaluation (every operator
rounded once, correctly, to binary32) over wide ranges of sizes, worker counts, magnitudes and
hyper-parameters.  No GPU."""
import numpy as np
from hypothesis import given, settings
from hypothesis import strategies as st

import oracle
import pins
from pins import F32, a32


def _values(rng, n, spread):
    mant = rng.normal(0, 1, n)
    expo = rng.integers(-spread, spread + 1, n)
    return a32(mant * np.power(2.0, expo))


@settings(max_examples=40, deadline=None)
@given(seed=st.integers(0, 2**31 - 1), n=st.integers(1, 24), m=st.integers(1, 9), spread=st.integers(0, 30),
       lr=st.floats(1e-4, 2.0), mu=st.floats(0.0, 0.99), wd=st.floats(0.0, 0.1))
def test_server_rule_matches_exact_rationals(seed, n, m, spread, lr, mu, wd):
    rng = np.random.default_rng(seed)
    w, v = _values(rng, n, spread), _values(rng, n, spread)
    grads = [_values(rng, n, spread) for _ in range(m)]
    wn, vn = pins.exact_global_update(grads, w, v, lr, mu, wd)
    w1, v1 = w.copy(), v.copy()
    wp = np.empty_like(w)
    oracle.global_update(grads, w1, v1, lr=lr, momentum=mu, wd=wd, w_prev=wp)
    pins.assert_same_bits(w1, wn, "w")
    pins.assert_same_bits(v1, vn, "v")
    pins.assert_same_bits(wp, w, "backup")
    # one worker: the ASGD step is the same arithmetic
    if m == 1:
        w2, v2 = w.copy(), v.copy()
        oracle.asgd_step(grads[0], w2, v2, lr=lr, momentum=mu, wd=wd)
        pins.assert_same_bits(w2, wn, "asgd w")
        pins.assert_same_bits(v2, vn, "asgd v")


@settings(max_examples=40, deadline=None)
@given(seed=st.integers(0, 2**31 - 1), n=st.integers(1, 64), spread=st.integers(0, 40), llr=st.floats(0.0, 4.0))
def test_local_rule_matches_exact_rationals(seed, n, spread, llr):
    rng = np.random.default_rng(seed)
    w, g = _values(rng, n, spread), _values(rng, n, spread)
    fr, rnd = pins._fr, pins.round_to_f32
    want = np.array([rnd(fr(w[i]) - fr(rnd(fr(F32(llr)) * fr(g[i])))) for i in range(n)], F32)
    pins.assert_same_bits(oracle.local_update(w, g, local_lr=llr), want, "x")


@settings(max_examples=25, deadline=None)
@given(seed=st.integers(0, 2**31 - 1), n=st.integers(1, 32), lam=st.floats(0.0, 4.0), llr=st.floats(1e-3, 1.0),
       m=st.floats(0.0, 0.999), eps=st.floats(1e-8, 1e-2))
def test_delay_compensated_rules_match_exact_rationals(seed, n, lam, llr, m, eps):
    rng = np.random.default_rng(seed)
    w = a32(rng.normal(0, 1, n))
    xp = a32(w + rng.normal(0, 0.1, n))
    g = a32(rng.normal(0, 0.5, n))
    ms = a32(rng.uniform(0, 1, n))
    fr, rnd = pins._fr, pins.round_to_f32
    lam32, llr32, m32, eps32 = F32(lam), F32(llr), F32(m), F32(eps)
    omm = rnd(fr(F32(1.0)) - fr(m32))

    def eq4(i, lam_i):
        diff = rnd(fr(w[i]) - fr(xp[i]))
        gg = rnd(fr(g[i]) * fr(g[i]))
        comp = rnd(fr(rnd(fr(lam_i) * fr(gg))) * fr(diff))
        d = rnd(fr(g[i]) + fr(comp))
        return rnd(fr(w[i]) - fr(rnd(fr(llr32) * fr(d))))

    want_c = np.array([eq4(i, lam32) for i in range(n)], F32)
    pins.assert_same_bits(oracle.local_update_dc_c(w, g, xp, local_lr=llr, lam=lam), want_c, "Eq. 4")
    # Eq. 6 exactly; Eq. 5's sqrt and division are correctly rounded IEEE operations, taken from numpy
    ms_new = np.empty(n, F32)
    want_a = np.empty(n, F32)
    for i in range(n):
        gg = rnd(fr(g[i]) * fr(g[i]))
        ms_new[i] = rnd(fr(rnd(fr(m32) * fr(ms[i]))) + fr(rnd(fr(omm) * fr(gg))))
        den = np.sqrt(F32(rnd(fr(ms_new[i]) + fr(eps32))))
        want_a[i] = eq4(i, F32(lam32 / den))
    ms1 = ms.copy()
    got = oracle.local_update_dc_a(w, g, xp, ms1, local_lr=llr, lam=lam, m=m, eps=eps)
    pins.assert_same_bits(ms1, ms_new, "Eq. 6")
    pins.assert_same_bits(got, want_a, "Eq. 5")
