"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these checks re-types the oracle's formulas: each one compares it with
something defined another way (exact rational arithmetic, a closed form, a
literal four-statement transcription of Algorithm 1, a library rounding
routine, an invariant).  CPU only.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import (EXP_AMAX, EXP_FIXED, OracleState, OracleTensor, oracle_element,
                    oracle_increment, oracle_next_exponent, oracle_rne_shift, oracle_step,
                    oracle_step_tensor)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def qmax(b):
    return 2 ** (b - 1) - 1


def nearest_even(x: Fraction) -> int:
    """Round-half-to-even of an exact rational (Python's round on a Fraction)."""
    return round(x)


def sat(x, bits):
    return max(-qmax(bits), min(qmax(bits), x))


def exact_update(qt, qc, d, m, n, s, e_in, e_out):
    """Definition in exact rationals: theta' = value nearest to theta + c - d*2^ec_out on
    theta's output grid (ties to even), clamped; c' = the rest, on c's output grid, clamped."""
    ec_in, ec_out = e_in - s, e_out - s
    two = Fraction(2)
    v = qt * two ** e_in + (qc * two ** ec_in if n else 0) - d * two ** ec_out
    P = nearest_even(v / two ** e_out)
    qt2 = sat(P, m)
    if n == 0:
        return P, qt2, 0, 0
    Rq = nearest_even((v - qt2 * two ** e_out) / two ** ec_out)
    return P, qt2, Rq, sat(Rq, n)


def run_element(qt, qc, d, m, n, s, e_in, e_out):
    """Feed the oracle an increment that is exactly d accumulator LSBs (lr = 1, g = d*2^ec_out)."""
    ec_out = e_out - s if n else e_out
    g = float(np.float32(d * 2.0 ** ec_out))
    assert Fraction(g) == Fraction(d) * Fraction(2) ** ec_out
    return oracle_element(qt, qc, g, 1.0, m, n, s, e_in, e_out)


# ----------------------------------------------------------------------------- rounding

def test_rne_shift_matches_exact_rational_rounding():
    for r in range(0, 9):
        for a in range(-600, 601):
            assert oracle_rne_shift(a, r) == nearest_even(Fraction(a, 2 ** r)), (a, r)
    rng = np.random.default_rng(1)
    for a in rng.integers(-2 ** 40, 2 ** 40, 2000):
        for r in (1, 7, 15, 23):
            assert oracle_rne_shift(int(a), r) == nearest_even(Fraction(int(a), 2 ** r))


def test_rne_shift_ties_go_to_even():
    assert [oracle_rne_shift(a, 1) for a in (1, 3, 5, -1, -3, -5)] == [0, 2, 2, 0, -2, -2]
    assert oracle_rne_shift(0b0100, 3) == 0 and oracle_rne_shift(0b1100, 3) == 2


# ----------------------------------------------------------------------------- increment (stmt 1)

def test_increment_exact_when_product_is_representable():
    # g*lr*2^-ec exactly representable in binary32 -> d is the exact rational rounding
    for ec in (-18, -7, 0, 3):
        for num in range(-40, 41):
            for lr in (1.0, 0.5, 0.25):
                g = num * 2.0 ** (ec - 2)          # quarter-LSB steps: hits every tie
                want = nearest_even(Fraction(g) * Fraction(lr) / Fraction(2) ** ec)
                assert oracle_increment(g, lr, ec) == want, (g, lr, ec)


def test_increment_within_half_lsb_plus_product_rounding():
    rng = np.random.default_rng(2)
    g = (rng.standard_normal(3000) * 1e-3).astype(np.float32)
    for lr in (0.01, 0.1, 3e-4):
        lr32 = float(np.float32(lr))
        for ec in (-18, -24, -10):
            for gi in g[:1000]:
                exact = Fraction(float(gi)) * Fraction(lr32) / Fraction(2) ** ec
                d = oracle_increment(float(gi), lr32, ec)
                # binary32 product: relative error <= 2^-24 (scale itself is exact)
                assert abs(d - exact) <= Fraction(1, 2) + abs(exact) * Fraction(1, 2 ** 24)


def test_increment_is_one_binary32_multiply_then_rint():
    # library routine: numpy float32 multiply and rint (both IEEE, ties to even)
    rng = np.random.default_rng(3)
    g = (rng.standard_t(3, 20000) * 1e-3).astype(np.float32)
    lr = np.float32(0.01)
    for ec in (-18, -26):
        scale = np.float32(np.ldexp(lr, -ec))
        want = np.clip(np.rint((g * scale).astype(np.float32)).astype(np.int64), -2 ** 30, 2 ** 30)
        got = np.array([oracle_increment(float(x), float(lr), ec) for x in g])
        assert np.array_equal(got, want)


def test_increment_special_values():
    inf, nan = float("inf"), float("nan")
    assert oracle_increment(nan, 0.01, -18) == 0
    assert oracle_increment(inf, 0.01, -18) == 2 ** 30
    assert oracle_increment(-inf, 0.01, -18) == -2 ** 30
    assert oracle_increment(1e30, 0.01, -18) == 2 ** 30      # clamp
    assert oracle_increment(-1e30, 0.01, -18) == -2 ** 30
    assert oracle_increment(1e-45, 0.01, -18) == 0           # subnormal gradient
    assert oracle_increment(0.0, 0.01, -18) == 0
    e = oracle_element(5, 3, nan, 0.01, 8, 8, 7, -11, -11)
    assert (e.q_theta, e.q_comp, e.nonfinite) == (5, 3, 1)
    e = oracle_element(5, 3, inf, 0.01, 8, 8, 7, -11, -11)
    assert (e.q_theta, e.q_comp, e.nonfinite, e.d) == (-127, -127, 1, 2 ** 30)
    assert oracle_element(5, 3, 1.0, 0.01, 8, 8, 7, -11, -11).nonfinite == 0


# ----------------------------------------------------------------------------- P3 brute force

@pytest.mark.parametrize("m", [3, 4, 5, 6])
@pytest.mark.parametrize("n", [3, 4, 5, 6])
def test_brute_force_small_widths_vs_exact_rationals(m, n):
    """Every (Q_theta, Q_c, d) at small widths, every legal overlap k, fixed exponents."""
    for k in range(0, n):
        s = n - 1 - k
        span = 3 * 2 ** s + 2
        for qt in range(-2 ** (m - 1), 2 ** (m - 1)):
            for qc in range(-2 ** (n - 1), 2 ** (n - 1), 1 if n <= 4 else 3):
                for d in list(range(-span, span + 1, 1 if s <= 3 else 5)) + [-2 ** 12, 2 ** 12]:
                    e = run_element(qt, qc, d, m, n, s, -4, -4)
                    P, qt2, Rq, qc2 = exact_update(qt, qc, d, m, n, s, -4, -4)
                    assert (e.P, e.q_theta, e.Rq, e.q_comp, e.d) == (P, qt2, Rq, qc2, d), \
                        (m, n, k, qt, qc, d)


def test_brute_force_int8_vectorised_vs_float64_rounding():
    """All 256 x 256 int8 pairs x a sweep of increments, through the array entry point,
    against numpy's float64 rint (exact here: every value is an integer below 2^53)."""
    s, m, n = 7, 8, 8
    qt, qc = np.meshgrid(np.arange(-128, 128), np.arange(-128, 128), indexing="ij")
    qt = qt.ravel().astype(np.int8)
    qc = qc.ravel().astype(np.int8)
    for d in (0, 1, -1, 63, 64, 65, -64, 127, 128, 129, 191, 192, 193, -192, 300, -16383, 40000):
        theta, comp = qt.copy(), qc.copy()
        g = np.full(theta.size, d * 2.0 ** (-11 - s), dtype=np.float32)
        st = oracle_step_tensor(theta, comp, g, m, n, 0, -11, -11, 1.0)
        T = qt.astype(np.int64) * 2 ** s + qc.astype(np.int64) - d
        P = np.rint(T.astype(np.float64) / 2 ** s).astype(np.int64)
        want_t = np.clip(P, -127, 127)
        R = T - want_t * 2 ** s
        want_c = np.clip(R, -127, 127)
        assert np.array_equal(theta, want_t.astype(np.int8)), d
        assert np.array_equal(comp, want_c.astype(np.int8)), d
        assert st["amax_theta"] == int(np.abs(P).max())
        assert st["amax_comp"] == int(np.abs(R).max())
        assert st["n_sat_theta"] == int((P != want_t).sum())
        assert st["n_sat_comp"] == int((R != want_c).sum())


# ----------------------------------------------------------------------------- P7 regrid

@pytest.mark.parametrize("delta", list(range(-8, 9)))
def test_regrid_every_delta_vs_exact_rationals(delta):
    rng = np.random.default_rng(100 + delta)
    for (m, n, k) in ((8, 8, 0), (16, 8, 0), (16, 16, 0), (8, 16, 0), (8, 8, 3), (5, 4, 1)):
        s = n - 1 - k
        e_in, e_out = -9, -9 + delta
        for _ in range(300):
            qt = int(rng.integers(-2 ** (m - 1), 2 ** (m - 1)))
            qc = int(rng.integers(-2 ** (n - 1), 2 ** (n - 1)))
            d = int(rng.integers(-2 ** (s + 2), 2 ** (s + 2) + 1))
            e = run_element(qt, qc, d, m, n, s, e_in, e_out)
            P, qt2, Rq, qc2 = exact_update(qt, qc, d, m, n, s, e_in, e_out)
            assert (e.P, e.q_theta, e.Rq, e.q_comp) == (P, qt2, Rq, qc2), (m, n, k, qt, qc, d)
            two = Fraction(2)
            before = qt * two ** e_in + qc * two ** (e_in - s) - d * two ** (e_out - s)
            after = e.q_theta * two ** e_out + e.q_comp * two ** (e_out - s)
            if e.P == e.q_theta and e.Rq == e.q_comp:
                if delta <= 0:
                    assert after == before          # moving to a finer grid loses nothing
                else:
                    assert abs(after - before) <= two ** (e_out - s) / 2


# ----------------------------------------------------------------------------- P4 literal Algorithm 1

def literal_algorithm_1(theta, acc, eta_g, e_theta, e_acc, m, n):
    """The four statements as printed, on exact values, with a quantizer (nearest-even onto
    the destination's grid, symmetric saturation) after each statement that stores a value."""
    two = Fraction(2)

    def q_theta(v):
        return sat(nearest_even(v / two ** e_theta), m) * two ** e_theta

    def q_acc(v):
        return sat(nearest_even(v / two ** e_acc), n) * two ** e_acc

    acc = q_acc(acc + eta_g)                 # acc <- acc + eta dL/dtheta
    theta_update = q_theta(theta - acc)      # theta_update = theta - acc
    acc = q_acc(acc + (theta_update - theta))  # acc <- acc + (theta_update - theta)
    theta = theta_update                     # theta <- theta_update
    return theta, acc


@pytest.mark.parametrize("m,n,k", [(8, 8, 0), (8, 8, 2), (6, 5, 0), (8, 16, 0), (16, 8, 0)])
def test_literal_algorithm_1_agrees_when_accumulator_does_not_overflow(m, n, k):
    s = n - 1 - k
    e_t, e_c = -6, -6 - s
    two = Fraction(2)
    rng = np.random.default_rng(7)
    checked = 0
    for _ in range(4000):
        qt = int(rng.integers(-qmax(m), qmax(m) + 1))
        qc = int(rng.integers(-qmax(n), qmax(n) + 1))
        d = int(rng.integers(-2 ** (s + 1), 2 ** (s + 1) + 1))
        if abs(qc - d) > qmax(n):
            continue
        theta, acc = literal_algorithm_1(qt * two ** e_t, -qc * two ** e_c, d * two ** e_c,
                                         e_t, e_c, m, n)
        e = run_element(qt, qc, d, m, n, s, e_t, e_t)
        assert e.q_theta * two ** e_t == theta
        assert -e.q_comp * two ** e_c == acc     # c = -acc
        checked += 1
    assert checked > 1000


# ----------------------------------------------------------------------------- P1 stall vs move

def test_plain_sgd_stalls_while_lazy_update_moves():
    """Section 2: an increment below the parameter's precision never changes theta under
    Eq. 1, while the accumulator delivers it once enough has been gathered."""
    e_theta, s = -11, 7
    lr = 1.0
    g = np.float32(0.3 * 2.0 ** e_theta)
    q0 = np.array([-7, -3, 0, 1, 2, 77, 126], dtype=np.int8)
    N = 400

    plain = q0.copy()
    for _ in range(N):
        oracle_step_tensor(plain, None, np.full(q0.size, g, np.float32), 8, 0, 0, e_theta,
                           e_theta, lr)
    assert np.array_equal(plain, q0)

    theta, comp = q0.copy(), np.zeros(q0.size, np.int8)
    d = nearest_even(Fraction(float(g)) / Fraction(2) ** (e_theta - s))
    assert d == 38
    for step in range(1, N + 1):
        oracle_step_tensor(theta, comp, np.full(q0.size, g, np.float32), 8, 8, 0, e_theta,
                           e_theta, lr)
        for i, q in enumerate(q0):
            total = int(q) * 2 ** s - step * d
            assert int(theta[i]) * 2 ** s + int(comp[i]) == total
            assert abs(int(comp[i])) <= 2 ** (s - 1)
            # theta is a nearest grid point to the exact wide value at every step
            assert abs(Fraction(total, 2 ** s) - int(theta[i])) <= Fraction(1, 2)
    # ~0.3 LSB per step for 400 steps: theta moved by ~119 LSB
    assert np.all(q0.astype(int) - theta.astype(int) >= 118)


# ----------------------------------------------------------------------------- P2 invariant

@pytest.mark.parametrize("m,n", [(8, 8), (16, 8), (16, 16), (8, 16)])
def test_parameter_plus_compensation_tracks_exact_accumulation(m, n):
    s = n - 1
    e_t = -11 if m == 8 else -17
    e_c = e_t - s
    rng = np.random.default_rng(11)
    N = 4096
    dt_t = np.int8 if m == 8 else np.int16
    dt_c = np.int8 if n == 8 else np.int16
    theta = rng.integers(-qmax(m) // 2, qmax(m) // 2, N).astype(dt_t)
    comp = rng.integers(-2 ** (s - 1), 2 ** (s - 1), N).astype(dt_c)
    wide0 = theta.astype(object) * 2 ** s + comp.astype(object)
    lr = float(np.float32(0.01))
    sigma = 30 * 2.0 ** e_c / lr          # ~30 compensation LSBs per step
    int_sum = np.zeros(N, dtype=object)
    real_sum = [Fraction(0)] * N
    steps = 60
    for t in range(1, steps + 1):
        g = (rng.standard_normal(N) * sigma).astype(np.float32)
        st = oracle_step_tensor(theta, comp, g, m, n, 0, e_t, e_t, lr)
        assert st["n_sat_theta"] == 0 and st["n_sat_comp"] == 0
        d = np.array([oracle_increment(float(x), lr, e_c) for x in g], dtype=object)
        int_sum += d
        # exact integer invariant: nothing is ever lost
        assert np.all(theta.astype(object) * 2 ** s + comp.astype(object) == wide0 - int_sum)
        assert np.abs(comp.astype(np.int64)).max() <= 2 ** (s - 1)
        for i in range(0, N, 64):
            real_sum[i] += Fraction(float(g[i])) * Fraction(lr)
    two = Fraction(2)
    for i in range(0, N, 64):
        got = (int(theta[i]) * 2 ** s + int(comp[i])) * two ** e_c
        want = int(wide0[i]) * two ** e_c - real_sum[i]
        bound = steps * (two ** e_c / 2 + abs(real_sum[i]) * Fraction(1, 2 ** 20))
        assert abs(got - want) <= bound


# ----------------------------------------------------------------------------- P5 bit-width

def test_bitwidth_closed_form_and_tie_step_counts():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "bitwidth_extension.txt"))
            if ln.strip() and not ln.startswith("#")]
    for m, n, k, bits in (map(int, r) for r in rows):
        assert m + n - 2 - k == bits
        s = n - 1 - k
        assert (m - 1) + s == bits        # magnitude bits of theta plus the grid distance
    # dynamic check: increments of exactly one compensation LSB per step first move an even
    # mantissa after 2^(s-1)+1 steps and an odd one after 2^(s-1) steps (ties to even), so the
    # compensation really resolves 2^-s of a parameter LSB.
    for (m, n, k) in ((8, 8, 0), (8, 16, 0), (8, 8, 3), (16, 8, 0)):
        s = n - 1 - k
        e_t = -5
        g = np.float32(2.0 ** (e_t - s))
        for q0, want_steps in ((10, 2 ** (s - 1) + 1), (11, 2 ** (s - 1))):
            dt_t = np.int8 if m == 8 else np.int16
            dt_c = np.int8 if n == 8 else np.int16
            theta, comp = np.array([q0], dt_t), np.zeros(1, dt_c)
            steps = 0
            while int(theta[0]) == q0:
                oracle_step_tensor(theta, comp, np.array([g], np.float32), m, n, k, e_t, e_t, 1.0)
                steps += 1
                assert steps <= 2 ** s
                if int(theta[0]) == q0:      # one LSB of a grid s bits below theta's per step
                    assert int(comp[0]) == -steps
            assert steps == want_steps and int(theta[0]) == q0 - 1


# ----------------------------------------------------------------------------- P6 reductions

def test_plain_mode_is_eq_1_in_one_numpy_line():
    rng = np.random.default_rng(5)
    e_t, lr = -7, np.float32(0.1)
    theta0 = rng.integers(-127, 128, 50000).astype(np.int8)
    g = (rng.standard_normal(50000) * 0.3).astype(np.float32)
    theta = theta0.copy()
    st = oracle_step_tensor(theta, None, g, 8, 0, 0, e_t, e_t, float(lr))
    want = np.clip(theta0.astype(np.int64)
                   - np.rint(g * np.float32(np.ldexp(lr, -e_t))).astype(np.int64), -127, 127)
    assert np.array_equal(theta, want.astype(np.int8))
    assert st["amax_comp"] == 0 and st["n_sat_comp"] == 0


def test_zero_increment_is_identity():
    rng = np.random.default_rng(6)
    for (m, n, s) in ((8, 8, 7), (16, 8, 7), (16, 16, 15)):
        dt_t = np.int8 if m == 8 else np.int16
        dt_c = np.int8 if n == 8 else np.int16
        theta0 = rng.integers(-qmax(m), qmax(m) + 1, 10000).astype(dt_t)
        comp0 = rng.integers(-2 ** (s - 1) + 1, 2 ** (s - 1), 10000).astype(dt_c)
        theta, comp = theta0.copy(), comp0.copy()
        oracle_step_tensor(theta, comp, np.zeros(10000, np.float32), m, n, 0, -9, -9, 0.5)
        assert np.array_equal(theta, theta0) and np.array_equal(comp, comp0)


# ----------------------------------------------------------------------------- saturation (R3)

def test_saturation_mass_flows_into_compensation_and_is_counted():
    # theta at +QMAX pushed further up: theta stays, the excess lands in c until c clamps too
    theta, comp = np.array([127], np.int8), np.zeros(1, np.int8)
    g = np.array([-60 * 2.0 ** (-11 - 7)], np.float32)   # d = -60 -> T grows by 60 per step
    st = oracle_step_tensor(theta, comp, g, 8, 8, 0, -11, -11, 1.0)
    assert (int(theta[0]), int(comp[0]), st["n_sat_theta"]) == (127, 60, 0)
    st = oracle_step_tensor(theta, comp, g, 8, 8, 0, -11, -11, 1.0)   # T = 127*128+120 -> P = 128
    assert (int(theta[0]), int(comp[0])) == (127, 120)
    assert (st["amax_theta"], st["n_sat_theta"], st["n_sat_comp"]) == (128, 1, 0)
    st = oracle_step_tensor(theta, comp, g, 8, 8, 0, -11, -11, 1.0)   # R = 180 -> clamps to 127
    assert (int(theta[0]), int(comp[0])) == (127, 127)
    assert (st["n_sat_theta"], st["n_sat_comp"], st["amax_comp"]) == (1, 1, 180)
    # the most negative two's-complement code is accepted on input, never produced
    theta, comp = np.array([-128], np.int8), np.array([-128], np.int8)
    oracle_step_tensor(theta, comp, np.zeros(1, np.float32), 8, 8, 0, 0, 0, 1.0)
    assert int(theta[0]) == -127 and int(comp[0]) == -127


# ----------------------------------------------------------------------------- P8 exponent policy

@pytest.mark.parametrize("bits", [8, 16])
def test_next_exponent_is_the_tight_fit(bits):
    Q = qmax(bits)
    for A in list(range(1, 70000)) + [2 ** 18 - 1, 2 ** 18, 2 ** 20, 2 ** 20 + 1]:
        e = oracle_next_exponent(A, bits, 0, EXP_AMAX)
        delta = e - 0
        if -8 < delta < 8:
            # after rescaling, the largest mantissa sits in (QMAX/2, QMAX]
            top = Fraction(A, 1) / Fraction(2) ** delta
            assert top <= Q and 2 * top > Q, (A, e)
        elif delta == 8:
            assert Fraction(A, 2 ** 7) > Q          # even 7 binades up would not hold it
        else:
            assert A * 2 ** 8 <= Q or Fraction(A * 2 ** 8) / 2 <= Q
    assert oracle_next_exponent(0, bits, 5, EXP_AMAX) == 5
    assert oracle_next_exponent(123456, bits, 5, EXP_FIXED) == 5
    # range clamp
    assert oracle_next_exponent(10 * Q, bits, 63, EXP_AMAX) == 64
    assert oracle_next_exponent(1, bits, -63, EXP_AMAX) == -64
    # step clamp
    assert oracle_next_exponent(2 ** 31 - 1, 8, 0, EXP_AMAX) == 8
    assert oracle_next_exponent(1, 16, 0, EXP_AMAX) == -8


# ----------------------------------------------------------------------------- multi-tensor step

def test_step_rotates_exponents_and_follows_the_tensor_maximum():
    """A tensor whose values shrink is re-gridded finer one step later, and the values
    theta*2^e + c*2^ec survive the move exactly."""
    theta = np.array([40, -20, 3, 0], np.int8)
    comp = np.array([5, -7, 0, 1], np.int8)
    t = OracleTensor(theta, comp, 8, 8, 0, exp_theta=-4, exp_theta_next=-4)
    st = OracleState([t], EXP_AMAX)
    two = Fraction(2)
    before = [int(a) * two ** -4 + int(b) * two ** -11 for a, b in zip(theta, comp)]
    oracle_step(st, [np.zeros(4, np.float32)], [0.1])
    assert (t.exp_theta, t.exp_theta_next, t.amax_theta) == (-4, -5, 40)
    oracle_step(st, [np.zeros(4, np.float32)], [0.1])
    assert (t.exp_theta, t.exp_theta_next, t.amax_theta) == (-5, -5, 80)
    after = [int(a) * two ** -5 + int(b) * two ** -12 for a, b in zip(theta, comp)]
    assert before == after
    assert list(theta) == [80, -40, 6, 0]


def test_threads_do_not_change_results():
    rng = np.random.default_rng(9)
    theta0 = rng.integers(-32767, 32768, 200001).astype(np.int16)
    g = (rng.standard_t(3, 200001) * 1e-3).astype(np.float32)
    outs = []
    for nt in (1, 3, 8):
        theta, comp = theta0.copy(), np.zeros(theta0.size, np.int8)
        st = oracle_step_tensor(theta, comp, g, 16, 8, 0, -17, -17, 0.1, n_threads=nt)
        outs.append((theta, comp, st))
    for theta, comp, st in outs[1:]:
        assert np.array_equal(theta, outs[0][0]) and np.array_equal(comp, outs[0][1])
        assert st == outs[0][2]
