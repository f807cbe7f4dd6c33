"""Pins of the oracle's momentum variant (v <- mu v + eta g, then Algorithm 1 with v in the
place of eta g).  As for the plain update, nothing here re-types the oracle: each check
compares it with something defined another way.  CPU only."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import (EXP_AMAX, EXP_FIXED, oracle_momentum_element, oracle_momentum_step_tensor,
                    oracle_next_exponent_velocity, oracle_step_tensor)


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
    assert e > -149 + 23           # stay away from subnormals in these tests
    return sign * Fraction(round(a)) * Fraction(2) ** e


def exact_momentum(qt, qc, qv, g, lr, mu, m, n, s, b, e_in, e_out, ev_in, ev_out):
    """The element in exact rationals, with binary32 rounding applied where the definition
    says fl32 / fma32."""
    two = Fraction(2)
    mu_s = round_to_binary32(Fraction(mu) * two ** (ev_in - ev_out))
    scale_v = round_to_binary32(Fraction(lr) * two ** (-ev_out))
    bq = round_to_binary32(Fraction(g) * scale_v)
    y = round_to_binary32(mu_s * qv + bq)
    V = max(-2 ** 30, min(2 ** 30, round(y)))
    qv2 = sat(V, b)
    ec_in, ec_out = e_in - s, e_out - s
    k = ev_out - ec_out
    d = max(-2 ** 30, min(2 ** 30, round(Fraction(qv2) * two ** k)))
    val = qt * two ** e_in + (qc * two ** ec_in if n else 0) - d * two ** ec_out
    P = round(val / two ** e_out)
    qt2 = sat(P, m)
    if n == 0:
        return V, qv2, d, P, qt2, 0, 0
    Rq = round((val - qt2 * two ** e_out) / two ** ec_out)
    return V, qv2, d, P, qt2, Rq, sat(Rq, n)


@pytest.mark.parametrize("m,n,k,b", [(8, 8, 0, 8), (8, 8, 0, 16), (16, 8, 0, 16), (16, 16, 0, 16),
                                     (8, 16, 0, 8), (8, 0, 0, 8), (16, 0, 0, 16), (8, 8, 3, 8),
                                     (5, 4, 1, 6)])
def test_element_against_exact_rationals_with_binary32_rounding(m, n, k, b):
    rng = np.random.default_rng(m * 1000 + n * 100 + k * 10 + b)
    s = n - 1 - k if n else 0
    for _ in range(1500):
        e_in = int(rng.integers(-20, -4))
        e_out = e_in + int(rng.integers(-8, 9))
        ev_in = int(rng.integers(-30, 0))
        ev_out = ev_in + int(rng.integers(-8, 9))
        qt = int(rng.integers(-2 ** (m - 1), 2 ** (m - 1)))
        qc = int(rng.integers(-2 ** (n - 1), 2 ** (n - 1))) if n else 0
        qv = int(rng.integers(-2 ** (b - 1), 2 ** (b - 1)))
        lr = float(np.float32(rng.choice([0.1, 0.01, 0.5, 1.0])))
        mu = float(np.float32(rng.choice([0.0, 0.5, 0.9, 0.99])))
        g = float(np.float32(rng.standard_normal() * 2.0 ** ev_out * rng.choice([0.3, 5, 60, 3000]) / lr))
        e = oracle_momentum_element(qt, qc, qv, g, lr, mu, m, n, s, b, e_in, e_out, ev_in, ev_out)
        V, qv2, d, P, qt2, Rq, qc2 = exact_momentum(qt, qc, qv, g, lr, mu, m, n, s, b, e_in, e_out,
                                                    ev_in, ev_out)
        assert (e.V, e.q_mom, e.upd.d, e.upd.P, e.upd.q_theta, e.upd.Rq, e.upd.q_comp) == \
            (V, qv2, d, P, qt2, Rq, qc2), (qt, qc, qv, g, lr, mu, e_in, e_out, ev_in, ev_out)


def test_mu_zero_on_the_compensation_grid_is_the_plain_lazy_update():
    """mu = 0 with the velocity stored on the compensation grid (k = 0) and wide enough not
    to clamp: the velocity is exactly the quantized increment, so theta and c must come out
    as from the (separately pinned) plain lazy update."""
    rng = np.random.default_rng(3)
    n_el = 20000
    for (m, n) in ((8, 8), (16, 8)):
        s = n - 1
        e_t = -11
        dt = np.int8 if m == 8 else np.int16
        theta0 = rng.integers(-qmax(m), qmax(m) + 1, n_el).astype(dt)
        comp0 = rng.integers(-60, 61, n_el).astype(np.int8)
        g = (rng.standard_normal(n_el) * 2.0 ** (e_t - s) * 90 / 0.1).astype(np.float32)
        ta, ca = theta0.copy(), comp0.copy()
        sa = oracle_step_tensor(ta, ca, g, m, n, 0, e_t, e_t, 0.1)
        tb, cb, vb = theta0.copy(), comp0.copy(), rng.integers(-3000, 3000, n_el).astype(np.int16)
        sb = oracle_momentum_step_tensor(tb, cb, vb, g, m, n, 0, 16, e_t, e_t, e_t - s, e_t - s, 0.1, 0.0)
        assert np.array_equal(ta, tb) and np.array_equal(ca, cb)
        for key in ("amax_theta", "amax_comp", "n_sat_theta", "n_sat_comp"):
            assert sa[key] == sb[key]
        assert sb["n_sat_mom"] == 0


def test_velocity_reaches_the_geometric_fixed_point_and_nothing_is_lost():
    """Constant gradient: v tends to eta*g / (1 - mu) (within the rounding of its grid), and
    theta*2^s + c decreases by exactly the sum of the increments taken from the stored v."""
    e_t, s, ev = -8, 7, -14
    lr, mu = 0.1, 0.9
    g = np.float32(0.02)
    theta = np.array([5000, -7, 0, -20101], np.int16)
    comp = np.zeros(4, np.int8)
    mom = np.zeros(4, np.int16)
    wide0 = theta.astype(np.int64) * 2 ** s + comp
    total = np.zeros(4, np.int64)
    k = ev - (e_t - s)
    assert k == 1
    for step in range(200):
        oracle_momentum_step_tensor(theta, comp, mom, np.full(4, g, np.float32), 16, 8, 0, 16, e_t, e_t,
                                    ev, ev, lr, mu)
        total += mom.astype(np.int64) * 2 ** k
        assert np.array_equal(theta.astype(np.int64) * 2 ** s + comp, wide0 - total)
    fixed = Fraction(float(g)) * Fraction(float(np.float32(lr))) / (1 - Fraction(float(np.float32(mu)))) \
        / Fraction(2) ** ev
    # each step rounds by at most 1/2 (+ float rounding); the error is amplified by 1/(1-mu)
    assert abs(int(mom[0]) - fixed) <= Fraction(1, 2) / (1 - Fraction(9, 10)) + 1
    assert len(set(mom.tolist())) == 1


@pytest.mark.parametrize("k", [-20, -9, -3, -1, 0, 1, 4, 9, 14, 15, 16, 25, 70])
def test_velocity_to_compensation_grid_shift_both_directions(k):
    """d = Q_v' * 2^k for k >= 0 (clamped at 2^30), rne(Q_v' / 2^-k) for k < 0, ties to even."""
    s, e_t = 7, 0
    ec = e_t - s
    ev = ec + k
    if not -64 <= ev <= 64:
        pytest.skip("velocity exponent out of range")
    for qv in (-32767, -1025, -3, -2, -1, 0, 1, 2, 3, 5, 6, 1024, 1536, 32767):
        # mu = 1, g = 0: the velocity is kept as it is
        e = oracle_momentum_element(0, 0, qv, 0.0, 0.1, 1.0, 16, 8, s, 16, e_t, e_t, ev, ev)
        assert e.q_mom == qv
        want = max(-2 ** 30, min(2 ** 30, round(Fraction(qv) * Fraction(2) ** k)))
        assert e.upd.d == want, (k, qv)


def test_velocity_saturation_and_special_values():
    e = oracle_momentum_element(0, 0, 100, 1.0, 1.0, 0.9, 8, 8, 7, 8, 0, 0, -4, -4)
    assert (e.V, e.q_mom) == (106, 106)
    e = oracle_momentum_element(0, 0, 120, 1.0, 1.0, 0.9, 8, 8, 7, 8, 0, 0, -4, -4)
    assert (e.V, e.q_mom) == (124, 124)
    e = oracle_momentum_element(0, 0, 120, 2.0, 1.0, 0.9, 8, 8, 7, 8, 0, 0, -4, -4)
    assert (e.V, e.q_mom) == (140, 127)                       # clamped, pre-clamp value reported
    e = oracle_momentum_element(3, 4, 50, float("nan"), 1.0, 0.9, 8, 8, 7, 8, 0, 0, -4, -4)
    assert (e.V, e.q_mom, e.upd.nonfinite) == (0, 0, 1)
    e = oracle_momentum_element(3, 4, 50, float("inf"), 1.0, 0.9, 8, 8, 7, 8, 0, 0, -4, -4)
    assert (e.V, e.q_mom, e.upd.nonfinite) == (2 ** 30, 127, 1)
    st = oracle_momentum_step_tensor(np.array([3], np.int8), np.array([4], np.int8), np.array([120], np.int8),
                                     np.array([2.0], np.float32), 8, 8, 0, 8, 0, 0, -4, -4, 1.0, 0.9)
    assert (st["amax_mom"], st["n_sat_mom"]) == (140, 1)


def test_threads_do_not_change_momentum_results():
    rng = np.random.default_rng(9)
    n_el = 150001
    theta0 = rng.integers(-127, 128, n_el).astype(np.int8)
    g = (rng.standard_t(3, n_el) * 1e-3).astype(np.float32)
    outs = []
    for nt in (1, 5):
        theta, comp, mom = theta0.copy(), np.zeros(n_el, np.int8), np.zeros(n_el, np.int8)
        st = None
        for _ in range(3):
            st = oracle_momentum_step_tensor(theta, comp, mom, g, 8, 8, 0, 8, -11, -11, -18, -18, 0.01,
                                             0.9, n_threads=nt)
        outs.append((theta, comp, mom, st))
    assert all(np.array_equal(a, b) for a, b in zip(outs[0][:3], outs[1][:3])) and outs[0][3] == outs[1][3]


@pytest.mark.parametrize("bits", [8, 16])
def test_velocity_exponent_has_a_dead_band(bits):
    """The velocity keeps its exponent while its largest mantissa is in (QMAX/4, QMAX]; outside
    it moves to the tight fit, so afterwards the largest mantissa is in (QMAX/2, QMAX]."""
    Q = qmax(bits)
    for A in list(range(1, 5 * Q)) + [2 ** 20, 2 ** 24 + 1]:
        e = oracle_next_exponent_velocity(A, bits, 0, EXP_AMAX)
        if 4 * A > Q and A <= Q:
            assert e == 0, A
        elif -8 < e < 8:
            top = Fraction(A) / Fraction(2) ** e
            assert top <= Q and 2 * top > Q, (A, e)
            assert e != 0
        elif e == 8:
            assert Fraction(A, 2 ** 7) > Q
        else:
            assert A * 2 ** 8 <= Q or A * 2 ** 7 <= Q
    assert oracle_next_exponent_velocity(0, bits, 3, EXP_AMAX) == 3
    assert oracle_next_exponent_velocity(10 * Q, bits, 3, EXP_FIXED) == 3
    assert oracle_next_exponent_velocity(10 * Q, bits, 63, EXP_AMAX) == 64
    assert oracle_next_exponent_velocity(1, bits, -63, EXP_AMAX) == -64
    # a maximum that wanders by less than a factor of two settles after at most two moves
    # (one to the tight fit, one back if it landed just under QMAX)
    e, moves = 0, 0
    rng = np.random.default_rng(bits)
    base = 0.3 * Q
    for _ in range(400):
        A = int(base * rng.uniform(0.75, 1.45) / 2.0 ** e)
        e2 = oracle_next_exponent_velocity(A, bits, e, EXP_AMAX)
        moves += e2 != e
        e = e2
    assert moves <= 2
