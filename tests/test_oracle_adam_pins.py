"""Pins of the oracle's ADAM variant (Section 4: ADAM with the lazy update, 16-bit moments).
Nothing here re-types the oracle: each check compares it with something defined another
way -- exact rationals with explicit binary32 rounding, the separately pinned momentum and
plain updates, closed forms (sign descent), and a textbook fp64 ADAM.  CPU only."""
from fractions import Fraction
from math import isqrt

import numpy as np
import pytest

from oracle import (EXP_AMAX, OracleState, OracleTensor, oracle_adam_element, oracle_adam_step,
                    oracle_adam_step_tensor, oracle_element, oracle_momentum_element)


def qmax(b):
    return 2 ** (b - 1) - 1


def sat(x, bits):
    return max(-qmax(bits), min(qmax(bits), x))


def round_to_binary32(x: Fraction) -> Fraction:
    """Nearest binary32 value of an exact rational, ties to even (normal range only)."""
    if x == 0:
        return Fraction(0)
    sign = -1 if x < 0 else 1
    a = abs(x)
    e = 0
    while a >= 2 ** 24:
        a /= 2
        e += 1
    while a < 2 ** 23:
        a *= 2
        e -= 1
    assert -149 + 23 < e < 127 - 22          # stay inside the normal range in these tests
    return sign * Fraction(round(a)) * Fraction(2) ** e


def sqrt_to_binary32(x: Fraction) -> Fraction:
    """Correctly rounded binary32 square root of an exact non-negative rational: an integer
    square root with 40+ significant bits, plus half a unit when it is inexact so that the
    final rounding sees on which side of every 24-bit tie the true root lies."""
    if x == 0:
        return Fraction(0)
    k = 0
    while x * 4 ** k < 2 ** 80:
        k += 1
    scaled = x * 4 ** k
    n = scaled.numerator // scaled.denominator
    r = isqrt(n)
    exact = (r * r == n) and scaled.denominator == 1
    root = Fraction(r) if exact else Fraction(2 * r + 1, 2)
    return round_to_binary32(root / 2 ** k)


def exact_adam(qt, qc, qm, qv, g, lr, b1, b2, eps, m, n, s, e_in, e_out, em_in, em_out, ev_in, ev_out):
    two = Fraction(2)
    F = lambda x: Fraction(float(np.float32(x)))
    g, lr, b1, b2, eps = F(g), F(lr), F(b1), F(b2), F(eps)
    fl = round_to_binary32
    c1, c2 = fl(1 - b1), fl(1 - b2)
    ym = fl(fl(b1 * two ** (em_in - em_out)) * qm + fl(g * fl(c1 * two ** (-em_out))))
    yv = fl(fl(b2 * two ** (ev_in - ev_out)) * qv + fl(fl(g * g) * fl(c2 * two ** (-ev_out))))
    M = max(-2 ** 30, min(2 ** 30, round(ym)))
    V = max(-2 ** 30, min(2 ** 30, round(yv)))
    qm2, qv2 = sat(M, 16), sat(V, 16)
    mr, vr = qm2 * two ** em_out, max(1, qv2) * two ** ev_out
    den = fl(sqrt_to_binary32(vr) + eps)
    ec_in, ec_out = e_in - s, e_out - s
    q = fl(mr / den)
    d = max(-2 ** 30, min(2 ** 30, round(fl(q * fl(lr * two ** (-ec_out))))))
    val = qt * two ** e_in + (qc * two ** ec_in if n else 0) - d * two ** ec_out
    P = round(val / two ** e_out)
    qt2 = sat(P, m)
    if n == 0:
        return M, V, qm2, qv2, d, P, qt2, 0, 0
    Rq = round((val - qt2 * two ** e_out) / two ** ec_out)
    return M, V, qm2, qv2, d, P, qt2, Rq, sat(Rq, n)


def test_the_rounding_helpers_agree_with_numpy_binary32():
    rng = np.random.default_rng(0)
    for _ in range(3000):
        a = np.float32(abs(rng.standard_normal()) * 10.0 ** rng.integers(-12, 12))
        assert sqrt_to_binary32(Fraction(float(a))) == Fraction(float(np.sqrt(a)))
        b = np.float32(rng.standard_normal() + 3.0)
        assert round_to_binary32(Fraction(float(a)) / Fraction(float(b))) == Fraction(float(a / b))
    assert sqrt_to_binary32(Fraction(9, 4)) == Fraction(3, 2)
    assert sqrt_to_binary32(Fraction(2)) == Fraction(float(np.sqrt(np.float32(2))))


@pytest.mark.parametrize("m,n,k", [(8, 8, 0), (8, 16, 0), (16, 8, 0), (16, 16, 0), (16, 0, 0), (8, 8, 3),
                                   (5, 4, 1)])
def test_element_against_exact_rationals_with_binary32_rounding(m, n, k):
    rng = np.random.default_rng(m * 100 + n * 10 + k)
    s = n - 1 - k if n else 0
    for _ in range(1200):
        e_in = int(rng.integers(-20, -4))
        e_out = e_in + int(rng.integers(-8, 9))
        em_in = int(rng.integers(-30, -8))
        em_out = em_in + int(rng.integers(-8, 9))
        ev_in = int(rng.integers(-50, -20))
        ev_out = ev_in + int(rng.integers(-8, 9))
        qt = int(rng.integers(-2 ** (m - 1), 2 ** (m - 1)))
        qc = int(rng.integers(-2 ** (n - 1), 2 ** (n - 1))) if n else 0
        qm = int(rng.integers(-32768, 32768))
        qv = int(rng.integers(0, 32768)) if rng.random() < 0.9 else int(rng.integers(-50, 1))
        b1 = float(rng.choice([0.0, 0.5, 0.9]))
        b2 = float(rng.choice([0.0, 0.9, 0.999]))
        eps = float(rng.choice([1e-8, 1e-3, 0.0]))
        lr = float(rng.choice([1e-4, 1e-3, 0.01])) * 2.0 ** (e_out - s + 12)
        g = float(rng.standard_normal() * 2.0 ** em_out * rng.choice([3, 500, 40000, 1e6]))
        got = oracle_adam_element(qt, qc, qm, qv, g, lr, b1, b2, eps, m, n, s, e_in, e_out,
                                  em_in, em_out, ev_in, ev_out)
        want = exact_adam(qt, qc, qm, qv, g, lr, b1, b2, eps, m, n, s, e_in, e_out,
                          em_in, em_out, ev_in, ev_out)
        assert (got.M, got.V, got.q_m, got.q_v, got.upd.d, got.upd.P, got.upd.q_theta, got.upd.Rq,
                got.upd.q_comp) == want, (qt, qc, qm, qv, g, lr, b1, b2, eps, e_in, e_out, em_in,
                                          em_out, ev_in, ev_out)


def test_both_moments_are_the_pinned_momentum_recurrence():
    """m <- beta1 m + (1-beta1) g is the momentum oracle's velocity with mu = beta1 and step
    size fl(1-beta1); v is the same recurrence on fl(g*g) with beta2."""
    rng = np.random.default_rng(11)
    for _ in range(3000):
        em_in = int(rng.integers(-30, -8)); em_out = em_in + int(rng.integers(-8, 9))
        ev_in = int(rng.integers(-50, -20)); ev_out = ev_in + int(rng.integers(-8, 9))
        qm, qv = int(rng.integers(-32767, 32768)), int(rng.integers(0, 32768))
        b1, b2 = np.float32(rng.choice([0.5, 0.9])), np.float32(rng.choice([0.9, 0.999]))
        g = np.float32(rng.standard_normal() * 2.0 ** em_out * rng.choice([3, 500, 40000]))
        a = oracle_adam_element(0, 0, qm, qv, float(g), 1e-3, float(b1), float(b2), 1e-8, 16, 16, 15, -12,
                                -12, em_in, em_out, ev_in, ev_out)
        one = np.float32(1.0)
        vm = oracle_momentum_element(0, 0, qm, float(g), float(one - b1), float(b1), 16, 16, 15, 16, -12,
                                     -12, em_in, em_out)
        vv = oracle_momentum_element(0, 0, qv, float(g * g), float(one - b2), float(b2), 16, 16, 15, 16,
                                     -12, -12, ev_in, ev_out)
        assert (a.M, a.q_m) == (vm.V, vm.q_mom)
        assert (a.V, a.q_v) == (vv.V, vv.q_mom)


def test_statements_1_to_4_are_the_pinned_plain_update_with_the_same_increment():
    """Feeding the plain update a gradient equal to ADAM's integer increment and a step size
    of one compensation unit must give the same theta and c."""
    rng = np.random.default_rng(12)
    for (m, n, k) in ((8, 8, 0), (16, 8, 0), (16, 16, 0), (8, 8, 3), (16, 0, 0)):
        s = n - 1 - k if n else 0
        hits = 0
        for _ in range(1500):
            e_in = int(rng.integers(-20, -4)); e_out = e_in + int(rng.integers(-8, 9))
            qt = int(rng.integers(-qmax(m), qmax(m) + 1))
            qc = int(rng.integers(-qmax(n), qmax(n) + 1)) if n else 0
            qm, qv = int(rng.integers(-32767, 32768)), int(rng.integers(1, 32768))
            lr = 1e-3 * 2.0 ** (e_out - s + int(rng.integers(6, 14)))
            a = oracle_adam_element(qt, qc, qm, qv, 0.0, lr, 0.9, 0.999, 1e-8, m, n, s, e_in, e_out,
                                    -20, -20, -40, -40)
            if abs(a.upd.d) >= 2 ** 24:
                continue
            hits += 1
            p = oracle_element(qt, qc, float(a.upd.d), 2.0 ** (e_out - s), m, n, s, e_in, e_out)
            assert p.d == a.upd.d
            assert (p.T, p.P, p.q_theta, p.Rq, p.q_comp) == \
                (a.upd.T, a.upd.P, a.upd.q_theta, a.upd.Rq, a.upd.q_comp)
        assert hits > 1000


def test_beta_zero_eps_zero_is_sign_descent():
    """beta1 = beta2 = eps = 0 with a power-of-two gradient (exact on both moment grids):
    m / sqrt(v) = sign(g), so the increment is rne(lr * 2^-ec_out) with the sign of g, whatever
    the magnitude of g and whatever the moments held before."""
    rng = np.random.default_rng(13)
    e_t, s = -12, 15
    for _ in range(500):
        p = int(rng.integers(-9, -2))
        g = float(rng.choice([-1.0, 1.0])) * 2.0 ** p
        em = p - int(rng.integers(2, 14))
        ev = 2 * p - int(rng.integers(2, 14))
        lr = float(np.float32(rng.uniform(0.2, 3.0) * 2.0 ** (e_t - s + 9)))
        a = oracle_adam_element(123, -5, int(rng.integers(-30000, 30000)), int(rng.integers(0, 30000)), g,
                                lr, 0.0, 0.0, 0.0, 16, 16, s, e_t, e_t, em, em, ev, ev)
        want = round(Fraction(lr) * Fraction(2) ** (s - e_t))
        assert a.upd.d == (want if g > 0 else -want)
        assert a.q_m * Fraction(2) ** em == Fraction(g) and a.q_v * Fraction(2) ** ev == Fraction(g) ** 2


def test_non_finite_gradients_and_degenerate_denominators():
    base = dict(m=16, n=16, s=15, e_in=-12, e_out=-12, em_in=-20, em_out=-20, ev_in=-40, ev_out=-40)
    a = oracle_adam_element(100, 7, 500, 900, float("nan"), 1e-3, 0.9, 0.999, 1e-8, **base)
    assert (a.M, a.V, a.upd.d, a.upd.nonfinite) == (0, 0, 0, 1)
    assert (a.upd.q_theta, a.upd.q_comp) == (100, 7)
    a = oracle_adam_element(100, 7, 500, 900, float("inf"), 1e-3, 0.9, 0.999, 1e-8, **base)
    assert (a.M, a.V, a.q_m, a.q_v, a.upd.nonfinite) == (2 ** 30, 2 ** 30, 32767, 32767, 1)
    a = oracle_adam_element(100, 7, 500, 900, float("-inf"), 1e-3, 0.9, 0.999, 1e-8, **base)
    assert (a.M, a.V, a.q_m, a.q_v) == (-2 ** 30, 2 ** 30, -32767, 32767)
    # a second moment of zero (or a negative one, only reachable from a foreign state) enters
    # the denominator as one unit of its grid: with eps = 0 the step is m / sqrt(2^ev), not m/0
    for qv in (0, -9, 1):
        a = oracle_adam_element(100, 7, 512, qv, 0.0, 2.0 ** -20, 1.0, 1.0, 0.0, **base)
        # m = 512 * 2^-20, sqrt(v) = 2^-20: ratio 512, times lr = 2^-20 in units of 2^-27
        assert a.q_v == qv and a.upd.d == 512 * 2 ** 7
    a = oracle_adam_element(100, 7, 0, 0, 0.0, 1e-3, 1.0, 1.0, 0.0, **base)
    assert a.upd.d == 0 and (a.upd.q_theta, a.upd.q_comp) == (100, 7)


def test_step_tensor_is_the_element_rule_everywhere_and_its_statistics_are_brute_force():
    rng = np.random.default_rng(14)
    n_el = 5000
    theta = rng.integers(-127, 128, n_el).astype(np.int8)
    comp = rng.integers(-32767, 32768, n_el).astype(np.int16)
    m1 = rng.integers(-32767, 32768, n_el).astype(np.int16)
    m2 = rng.integers(0, 32768, n_el).astype(np.int16)
    g = (rng.standard_normal(n_el) * 2.0 ** -6).astype(np.float32)
    g[::97] *= 4000
    g[5], g[6] = np.nan, np.inf
    args = dict(e_in=-9, e_out=-10, em_in=-21, em_out=-20, ev_in=-27, ev_out=-28)
    t2, c2, a2, b2 = theta.copy(), comp.copy(), m1.copy(), m2.copy()
    st = oracle_adam_step_tensor(t2, c2, a2, b2, g, 8, 16, 0, lr=2e-3, beta1=0.9, beta2=0.999, eps=1e-8,
                                 n_threads=3, **args)
    am = dict(amax_theta=0, amax_comp=0, amax_m=0, amax_v=0, n_sat_theta=0, n_sat_comp=0, n_sat_m=0,
              n_sat_v=0, n_nonfinite=0)
    for i in range(n_el):
        e = oracle_adam_element(int(theta[i]), int(comp[i]), int(m1[i]), int(m2[i]), float(g[i]), 2e-3, 0.9,
                                0.999, 1e-8, 8, 16, 15, -9, -10, -21, -20, -27, -28)
        assert (t2[i], c2[i], a2[i], b2[i]) == (e.upd.q_theta, e.upd.q_comp, e.q_m, e.q_v)
        am["amax_theta"] = max(am["amax_theta"], abs(e.upd.P))
        am["amax_comp"] = max(am["amax_comp"], min(abs(e.upd.Rq), 2 ** 31 - 1))
        am["amax_m"] = max(am["amax_m"], abs(e.M)); am["amax_v"] = max(am["amax_v"], abs(e.V))
        am["n_sat_theta"] += e.upd.P != e.upd.q_theta; am["n_sat_comp"] += e.upd.Rq != e.upd.q_comp
        am["n_sat_m"] += e.M != e.q_m; am["n_sat_v"] += e.V != e.q_v
        am["n_nonfinite"] += e.upd.nonfinite
    assert st == am
    assert am["n_sat_m"] > 0 and am["n_sat_v"] > 0 and am["n_nonfinite"] == 2


def _textbook_adam(theta, grads, eta, b1, b2, eps):
    """fp64 ADAM as published (bias correction folded into the step size)."""
    m = np.zeros_like(theta); v = np.zeros_like(theta); th = theta.copy()
    for t, g in enumerate(grads, 1):
        m = b1 * m + (1 - b1) * g
        v = b2 * v + (1 - b2) * g * g
        th = th - eta * np.sqrt(1 - b2 ** t) / (1 - b1 ** t) * m / (np.sqrt(v) + eps)
    return th


def test_many_steps_track_textbook_fp64_adam_and_the_exponents_settle():
    """A short run with the exponent policy on (the dead band for both moments): the
    fixed-point trajectory stays within a few quantisation steps of fp64 ADAM, and the moments
    fill their 16 bits.  While the moments grow from zero (nearly doubling per step at first)
    the one-step-delayed exponent can lag and clip a few of the largest entries (a handful of
    element-steps in a quarter of a million)."""
    rng = np.random.default_rng(15)
    n_el, steps = 4096, 60
    eta, b1, b2, eps = 2e-4, 0.9, 0.999, 1e-8
    e_t = -19          # 32767 * 2^-19 = 0.0625: theta starts within 0.045 and moves at most 0.012,
    theta_real = np.clip(rng.standard_normal(n_el) * 0.03, -0.045, 0.045)   # so its exponent stays
    q = np.rint(theta_real * 2.0 ** -e_t).astype(np.int16)
    mean = rng.standard_normal(n_el) * 0.01
    grads = [(mean + rng.standard_normal(n_el) * 0.003).astype(np.float32) for _ in range(steps)]
    gmax = max(float(np.abs(g).max()) for g in grads)
    em0 = int(np.ceil(np.log2((1 - b1) * gmax / 32767)))
    ev0 = int(np.ceil(np.log2((1 - b2) * gmax ** 2 / 32767)))
    t = OracleTensor(theta=q.copy(), comp=np.zeros(n_el, np.int16), theta_bits=16, comp_bits=16, overlap_k=0,
                     exp_theta=e_t, exp_theta_next=e_t, mom=np.zeros(n_el, np.int16), mom_bits=16,
                     exp_mom=em0, exp_mom_next=em0, mom2=np.zeros(n_el, np.int16), exp_mom2=ev0,
                     exp_mom2_next=ev0)
    state = OracleState(tensors=[t], mode=EXP_AMAX, n_threads=2)
    for step, g in enumerate(grads, 1):
        lr_t = eta * np.sqrt(1 - b2 ** step) / (1 - b1 ** step)
        oracle_adam_step(state, [g], [lr_t], b1, b2, eps)
    assert t.n_sat_mom < 50 and t.n_sat_mom2 < 50 and t.n_sat_theta == 0 and t.n_sat_comp == 0
    assert 8192 <= t.amax_mom <= 32767 and 8192 <= t.amax_mom2 <= 32767
    got = t.theta.astype(np.float64) * 2.0 ** t.exp_theta + t.comp.astype(np.float64) * 2.0 ** (t.exp_theta - 15)
    want = _textbook_adam(q.astype(np.float64) * 2.0 ** e_t, [g.astype(np.float64) for g in grads], eta, b1,
                          b2, eps)
    moved = np.abs(want - q * 2.0 ** e_t)
    assert moved.mean() > 0.005                     # ~ steps * eta * |E g| / sqrt(E g^2)
    err = np.abs(got - want)
    # elements whose second moment stays above the 16-bit grid's resolution follow closely
    big = np.abs(mean) > 0.004
    assert big.sum() > 1000
    assert np.median(err[big]) < 0.02 * np.median(moved[big])
    assert err[big].max() < 0.25 * np.median(moved[big])
