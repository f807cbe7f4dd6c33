"""Pins of the oracle's strict Algorithm 1 (every statement rounded into the stored format,
the accumulator an n-bit dynamic fixed-point tensor with its own exponent).  Each check
compares the oracle with something written another way.  CPU only."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import (EXP_AMAX, EXP_FIXED, OracleState, OracleTensor, oracle_element, oracle_next_exponent,
                    oracle_next_exponent_acc, oracle_step, oracle_strict_element, oracle_strict_step,
                    oracle_strict_step_tensor)


def qmax(b):
    return 2 ** (b - 1) - 1


def sat(x, bits):
    return max(-qmax(bits), min(qmax(bits), x))


def round_to_binary32(x: Fraction) -> Fraction:
    if x == 0:
        return Fraction(0)
    sign, a, e = (-1 if x < 0 else 1), abs(x), 0
    while a >= 2 ** 24:
        a /= 2; e += 1
    while a < 2 ** 23:
        a *= 2; e -= 1
    assert -149 + 23 < e < 127 - 22
    return sign * Fraction(round(a)) * Fraction(2) ** e


def quantize(x: Fraction, exponent: int, bits: int):
    """The stored format: nearest multiple of 2^exponent (ties to even), saturated.  Returns
    (unsaturated mantissa, stored mantissa)."""
    q = round(x / Fraction(2) ** exponent)
    return q, sat(q, bits)


def literal_algorithm_1(qt, qc, g, lr, m, n, e_in, e_out, ec_in, ec_out):
    """Algorithm 1 statement by statement, in the paper's own variables (acc, not c = -acc),
    in exact rationals; only the increment uses binary32, as everywhere in this method."""
    two = Fraction(2)
    theta = qt * two ** e_in
    acc = -qc * two ** ec_in
    scale = round_to_binary32(Fraction(lr) * two ** (-ec_out))
    d = max(-2 ** 30, min(2 ** 30, round(round_to_binary32(Fraction(g) * scale))))
    eta_g = d * two ** ec_out                      # "only the effective value in the significant figure of acc"
    a1_raw, a1 = quantize(acc + eta_g, ec_out, n)  # acc <- acc + eta g
    acc = a1 * two ** ec_out
    p_raw, p = quantize(theta - acc, e_out, m)     # theta_update = theta - acc
    theta_u = p * two ** e_out
    a2_raw, a2 = quantize(acc + (theta_u - theta), ec_out, n)   # acc <- acc + (theta_update - theta)
    return d, -a1_raw, -a1, p_raw, p, -a2_raw, -a2          # back to c = -acc


@pytest.mark.parametrize("m,n", [(8, 8), (8, 16), (16, 8), (16, 16), (5, 4)])
def test_element_is_the_literal_algorithm_in_exact_rationals(m, n):
    rng = np.random.default_rng(m * 100 + n)
    for _ in range(3000):
        e_in = int(rng.integers(-20, -4))
        e_out = e_in + int(rng.integers(-8, 9))
        ec_in = e_in - int(rng.integers(-8, 37))
        ec_out = max(e_out - 36, min(e_out + 8, ec_in + int(rng.integers(-8, 9))))
        qt = int(rng.integers(-qmax(m), qmax(m) + 1))
        qc = int(rng.integers(-qmax(n), qmax(n) + 1))
        lr = float(np.float32(rng.choice([0.01, 0.1, 1.0])))
        g = float(np.float32(rng.standard_normal() * 2.0 ** ec_out * rng.choice([0.4, 6, 90, 5000, 1e6]) / lr))
        got = oracle_strict_element(qt, qc, g, lr, m, n, e_in, e_out, ec_in, ec_out)
        want = literal_algorithm_1(qt, qc, g, lr, m, n, e_in, e_out, ec_in, ec_out)
        assert (got.d, got.C1, got.q_comp_mid, got.P, got.q_theta, got.C2, got.q_comp) == want, \
            (qt, qc, g, lr, e_in, e_out, ec_in, ec_out)


def test_tied_grids_without_accumulator_overflow_are_the_wide_update():
    """With c's exponent tied to theta's (e - s), no exponent change in the step and |c - d|
    within n bits, no statement of the strict form loses anything the wide form keeps: same
    theta', same c'.  (With an exponent change the strict form rounds c onto the new grid
    before theta is formed, the wide form rounds once at the end.)"""
    rng = np.random.default_rng(3)
    checked = 0
    for _ in range(6000):
        m, n = [(8, 8), (16, 8), (16, 16), (8, 16)][int(rng.integers(0, 4))]
        s = n - 1 - int(rng.integers(0, 3))
        e_in = int(rng.integers(-20, -4)); e_out = e_in
        qt, qc = int(rng.integers(-qmax(m), qmax(m) + 1)), int(rng.integers(-qmax(n) // 2, qmax(n) // 2))
        g = float(np.float32(rng.standard_normal() * 2.0 ** (e_out - s) * 30))
        st = oracle_strict_element(qt, qc, g, 1.0, m, n, e_in, e_out, e_in - s, e_out - s)
        if st.C1 != st.q_comp_mid:
            continue
        checked += 1
        w = oracle_element(qt, qc, g, 1.0, m, n, s, e_in, e_out)
        assert (st.d, st.P, st.q_theta, st.C2, st.q_comp) == (w.d, w.P, w.q_theta, w.Rq, w.q_comp)
    assert checked > 4000


def test_an_increment_beyond_the_accumulator_is_clipped_in_statement_1_only_in_the_strict_form():
    """eta*g = 1000 units of c with an 8-bit accumulator: the strict form stores 127 of them
    before theta sees anything; the wide form passes all 1000 on."""
    m, n, s, e = 16, 8, 7, -10
    g = float(np.float32(-1000 * 2.0 ** (e - s)))
    st = oracle_strict_element(0, 0, g, 1.0, m, n, e, e, e - s, e - s)
    w = oracle_element(0, 0, g, 1.0, m, n, s, e, e)
    assert st.d == w.d == -1000
    assert (st.C1, st.q_comp_mid) == (1000, 127) and (st.q_theta, st.q_comp) == (1, -1)     # 127/128 -> 1, -1 left
    assert (w.q_theta, w.q_comp) == (8, -24)                                               # 1000 = 8*128 - 24


def test_step_tensor_is_the_element_rule_with_brute_force_statistics():
    rng = np.random.default_rng(8)
    n_el = 6000
    theta = rng.integers(-127, 128, n_el).astype(np.int8)
    comp = rng.integers(-127, 128, n_el).astype(np.int8)
    g = (rng.standard_normal(n_el) * 2.0 ** -19 * 40).astype(np.float32)
    g[::101] *= 300
    g[3], g[4] = np.nan, -np.inf
    t2, c2 = theta.copy(), comp.copy()
    st = oracle_strict_step_tensor(t2, c2, g, 8, 8, -9, -10, -19, -18, 0.5, n_threads=3)
    want = dict(amax_theta=0, amax_comp=0, n_sat_theta=0, n_sat_comp=0, n_nonfinite=0)
    for i in range(n_el):
        e = oracle_strict_element(int(theta[i]), int(comp[i]), float(g[i]), 0.5, 8, 8, -9, -10, -19, -18)
        assert (t2[i], c2[i]) == (e.q_theta, e.q_comp)
        want["amax_theta"] = max(want["amax_theta"], min(abs(e.P), 2 ** 31 - 1))
        want["amax_comp"] = max(want["amax_comp"], min(max(abs(e.C1), abs(e.C2)), 2 ** 31 - 1))
        want["n_sat_theta"] += e.P != e.q_theta
        want["n_sat_comp"] += (e.C1 != e.q_comp_mid) + (e.C2 != e.q_comp)
        want["n_nonfinite"] += e.nonfinite
    assert st == want and want["n_sat_comp"] > 0 and want["n_nonfinite"] == 2
    with pytest.raises(ValueError):
        oracle_strict_step_tensor(t2, c2, g, 8, 8, -9, -9, -46, -46, 0.5)      # e - ec = 37
    with pytest.raises(ValueError):
        oracle_strict_step_tensor(t2, c2, g, 8, 8, 0, 8, -20, -3, 0.5)         # c's exponent moves by 17


def test_accumulator_exponent_policy_is_the_tight_fit_inside_the_window():
    for amax, bits, ec, e_next in [(100, 8, -20, -10), (1000, 8, -20, -10), (3, 16, -20, -10), (0, 8, -20, -10),
                                   (5, 8, -44, -10), (2 ** 31 - 1, 8, -5, -10), (70, 8, 60, 58)]:
        tight = oracle_next_exponent(amax, bits, ec, EXP_AMAX) if amax else ec - 8    # empty: 8 binades finer
        want = max(-64, min(64, max(e_next - 36, min(e_next + 8, tight))))
        assert oracle_next_exponent_acc(amax, bits, ec, e_next, EXP_AMAX) == want
        assert oracle_next_exponent_acc(amax, bits, ec, e_next, EXP_FIXED) == \
            max(-64, min(64, max(e_next - 36, min(e_next + 8, ec))))


def _constant_gradient_run(n, steps, e=-8, shift=12):
    g = np.full(64, np.float32(2.0 ** (e - shift)))
    t = OracleTensor(theta=np.full(64, 100, np.int8), comp=np.zeros(64, storage(n)), theta_bits=8, comp_bits=n,
                     overlap_k=0, exp_theta=e, exp_theta_next=e, exp_comp=e - (n - 1), exp_comp_next=e - (n - 1))
    st = OracleState([t], EXP_AMAX, 1)
    trace = []
    for _ in range(steps):
        oracle_strict_step(st, [g], [1.0])
        trace.append((int(t.theta[0]), int(t.comp[0]), t.exp_theta, t.exp_comp))
    return t, trace


def storage(bits):
    return np.int8 if bits <= 8 else np.int16


def test_small_constant_gradient_a_16_bit_accumulator_finds_its_scale_and_loses_next_to_nothing():
    """eta*g = 2^-12 of a theta unit.  An empty 16-bit accumulator first refines its grid, then
    the tight fit follows the growing sum; theta moves when the sum reaches half a unit (2048
    steps).  The only losses are at binade crossings, where the one-step-delayed exponent lets
    the mantissa clip once: theta + c stays within 1/16 of one increment of
    start - steps * eta*g."""
    e = -8
    t, trace = _constant_gradient_run(16, 3000)
    assert t.n_sat_theta == 0 and t.n_sat_comp <= 64 * 16
    thetas = [q for q, _, _, _ in trace]
    assert thetas.index(99) in (2047, 2048)                       # half a unit after 2048 increments (tie -> even)
    for step, (qt, qc, et, ec) in enumerate(trace):
        total = Fraction(qt) * Fraction(2) ** et + Fraction(qc) * Fraction(2) ** ec
        want = 100 * Fraction(2) ** e - (step + 1) * Fraction(2) ** (e - 12)
        assert abs(total - want) <= Fraction(2) ** (e - 12) / 16, step
    assert min(ec for _, _, _, ec in trace) <= e - 20 and trace[-1][3] >= e - 17     # fine first, coarser as acc grows


def test_small_constant_gradient_an_8_bit_accumulator_swamps_itself():
    """The same run with 8 bits: once the accumulated sum needs a grid whose half unit is not
    smaller than the increment, every further increment rounds away (ties to even keep the even
    mantissa 64) and theta never moves: the accumulator stops at 64 units of 2^(e-12+1), i.e.
    2^-5 theta units, for good.  The closed form of where it stops: |acc| in [2^6, 2^7) units
    with 2^(ec-1) >= eta*g."""
    e = -8
    t, trace = _constant_gradient_run(8, 1500)
    qt, qc, et, ec = trace[-1]
    assert trace[-1] == trace[-500] == trace[200]
    assert (qt, et) == (100, e)
    assert ec == e - 12 + 1 and abs(qc) == 64
