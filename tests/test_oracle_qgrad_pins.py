"""Pins of the step with fixed-point gradients (the paper's hardware model, Section 1: the
gradients are INT8/INT16 tensors with a shared exponent).  The oracle defines it as the plain
step on the exactly dequantized gradients; these checks pin the two facts that definition
rests on and show what the pre-quantization costs.  CPU only."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import (EXP_FIXED, OracleState, OracleTensor, oracle_dequantize_gradient, oracle_fit_exponent,
                    oracle_increment, oracle_quantize, oracle_step, oracle_step_qgrad)


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


@pytest.mark.parametrize("dtype", [np.int8, np.int16])
def test_dequantized_gradients_are_exact(dtype):
    info = np.iinfo(dtype)
    q = np.arange(info.min, info.max + 1, dtype=np.int64).astype(dtype)
    for e in (-64, -33, -1, 0, 7, 64):
        g = oracle_dequantize_gradient(q, e)
        assert g.dtype == np.float32
        assert all(Fraction(float(x)) == int(m) * Fraction(2) ** e for x, m in zip(g[::37], q[::37]))
        assert np.array_equal(np.ldexp(g.astype(np.float64), -e), q.astype(np.float64))


def test_increment_from_a_fixed_point_gradient_against_exact_rationals():
    """d = rne(fl32(Q_g 2^eg * fl32(eta 2^-ec))): one rounding for the step-size scale, one for
    the product, then ties-to-even to an integer."""
    rng = np.random.default_rng(5)
    for _ in range(4000):
        bits = int(rng.choice([8, 16]))
        q = int(rng.integers(-2 ** (bits - 1), 2 ** (bits - 1)))
        eg = int(rng.integers(-40, 0))
        ec = eg + int(rng.integers(-18, 6))
        lr = float(np.float32(rng.choice([1e-3, 0.01, 0.1, 0.37, 1.0])))
        g = float(oracle_dequantize_gradient(np.array([q], np.int8 if bits == 8 else np.int16), eg)[0])
        scale = round_to_binary32(Fraction(lr) * Fraction(2) ** (-ec))
        want = round(round_to_binary32(Fraction(q) * Fraction(2) ** eg * scale))
        want = max(-2 ** 30, min(2 ** 30, want))
        assert oracle_increment(g, lr, ec) == want, (q, eg, ec, lr)


def test_gradients_on_the_grid_give_the_binary32_step_and_small_ones_are_lost_before_the_update():
    """What the pre-quantization costs: with an INT8 gradient tensor whose exponent is set by
    one large entry, every entry below half a gradient unit reaches the update as zero, so
    neither theta nor the compensation moves however many steps are taken; the same
    gradients in binary32 accumulate in the compensation and move theta."""
    n = 4096
    rng = np.random.default_rng(6)
    g = (rng.standard_normal(n) * 1e-5).astype(np.float32)
    g[0] = 0.01                                       # one outlier fixes the INT8 grid
    eg = oracle_fit_exponent(g, 8)
    gq, _ = oracle_quantize(g, 8, 0, 0, eg)
    assert gq[0] == 127 or gq[0] == 126 or abs(int(gq[0])) > 63
    assert np.count_nonzero(gq[1:]) == 0              # 1e-5 is far below half a unit of 0.01/127
    theta0 = rng.integers(-100, 100, n).astype(np.int8)

    def run(quantized):
        t = OracleTensor(theta0.copy(), np.zeros(n, np.int16), 8, 16, 0, -7, -7)
        st = OracleState([t], EXP_FIXED, 1)
        for _ in range(200):
            if quantized:
                oracle_step_qgrad(st, [gq], [eg], [1.0])
            else:
                oracle_step(st, [g], [1.0])
        return t

    tq, tf = run(True), run(False)
    assert np.array_equal(tq.theta[1:], theta0[1:]) and not tq.comp[1:].any()
    moved = tf.theta.astype(np.int64) * 2 ** 15 + tf.comp - theta0.astype(np.int64) * 2 ** 15
    want = -200.0 * g.astype(np.float64) * 2.0 ** 22          # in compensation units of 2^(-7-15)
    assert np.abs(moved[1:] - want[1:]).max() <= 100.5        # 200 roundings of at most half a unit
    assert np.abs(moved[1:]).mean() > 1000
    # entries that are on the gradient grid take the same step either way
    on_grid = oracle_dequantize_gradient(gq, eg)
    a = OracleTensor(theta0.copy(), np.zeros(n, np.int16), 8, 16, 0, -7, -7)
    b = OracleTensor(theta0.copy(), np.zeros(n, np.int16), 8, 16, 0, -7, -7)
    oracle_step(OracleState([a], EXP_FIXED, 1), [on_grid], [1.0])
    oracle_step_qgrad(OracleState([b], EXP_FIXED, 1), [gq], [eg], [1.0])
    assert np.array_equal(a.theta, b.theta) and np.array_equal(a.comp, b.comp)
