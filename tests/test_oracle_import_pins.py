"""Pins of the oracle's fp32 <-> dynamic fixed-point import / export against exact
rationals and the properties the definition implies.  CPU only."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle_dequantize, oracle_fit_exponent, oracle_quantize
from test_oracle_momentum_pins import round_to_binary32


def qmax(b):
    return 2 ** (b - 1) - 1


def sat(x, b):
    return max(-qmax(b), min(qmax(b), x))


@pytest.mark.parametrize("bits", [8, 16])
def test_exponent_is_the_smallest_grid_that_holds_the_maximum(bits):
    rng = np.random.default_rng(bits)
    for scale in (1e-12, 3e-5, 0.02, 1.0, 77.0, 3e9):
        x = (rng.standard_normal(1000) * scale).astype(np.float32)
        x[::50] = np.nan
        x[1::97] = np.inf
        e = oracle_fit_exponent(x, bits)
        amax = max(abs(Fraction(float(v))) for v in x if np.isfinite(v))
        assert amax <= qmax(bits) * Fraction(2) ** e
        assert e == -64 or amax > qmax(bits) * Fraction(2) ** (e - 1)
    # exact boundaries: QMAX*2^e fits at e, the next float above needs e+1
    top = np.float32(qmax(bits) * 2.0 ** -7)
    assert oracle_fit_exponent(np.array([top], np.float32), bits) == -7
    assert oracle_fit_exponent(np.array([np.nextafter(top, np.float32(np.inf))], np.float32), bits) == -6
    assert oracle_fit_exponent(np.zeros(5, np.float32), bits) == 0
    assert oracle_fit_exponent(np.array([1e38], np.float32), bits) == 64
    assert oracle_fit_exponent(np.array([1e-38], np.float32), bits) == -64


@pytest.mark.parametrize("m,n,k", [(8, 0, 0), (16, 0, 0), (8, 8, 0), (16, 8, 0), (8, 16, 0), (16, 16, 0), (8, 8, 5)])
def test_quantize_matches_exact_rational_rounding_and_roundtrip_bound(m, n, k):
    rng = np.random.default_rng(m * 100 + n + k)
    s = n - 1 - k if n else 0
    x = (rng.standard_normal(4000) * 0.05).astype(np.float32)
    x[:40] = (np.arange(-20, 20) * 2.0 ** -9).astype(np.float32)       # grid points and ties
    x[40:80] = ((np.arange(-20, 20) + 0.5) * 2.0 ** -11).astype(np.float32)
    e = oracle_fit_exponent(x, m) + 1                                  # some head room, some saturation below
    x[80] = np.float32(10.0)
    x[81] = np.float32(-10.0)
    theta, comp = oracle_quantize(x, m, n, k, e)
    two = Fraction(2)
    for i in range(0, 4000, 7):
        v = Fraction(float(x[i]))
        qt = sat(round(v / two ** e), m)
        assert int(theta[i]) == qt, i
        if n:
            qc = sat(round((v - qt * two ** e) / two ** (e - s)), n)
            assert int(comp[i]) == qc, i
    back = oracle_dequantize(theta, comp, m, n, k, e)
    lsb = 2.0 ** (e - s)
    inside = np.abs(x) <= qmax(m) * 2.0 ** e
    err = np.abs(back.astype(np.float64) - x.astype(np.float64))[inside]
    assert err.max() <= 0.5 * lsb + np.abs(x[inside]).max() * 2.0 ** -24
    # values on the finest grid come back exactly
    on_grid = (np.arange(-100, 101) * lsb).astype(np.float32)
    t2, c2 = oracle_quantize(on_grid, m, n, k, e)
    assert np.array_equal(oracle_dequantize(t2, c2, m, n, k, e), on_grid)


def test_dequantize_is_the_exact_sum_rounded_once():
    rng = np.random.default_rng(4)
    theta = rng.integers(-32768, 32768, 3000).astype(np.int16)
    comp = rng.integers(-32768, 32768, 3000).astype(np.int16)
    for e, k in ((-15, 0), (3, 0), (-40, 7)):
        s = 15 - k
        got = oracle_dequantize(theta, comp, 16, 16, k, e)
        for i in range(0, 3000, 11):
            want = round_to_binary32(int(theta[i]) * Fraction(2) ** e + int(comp[i]) * Fraction(2) ** (e - s))
            assert Fraction(float(got[i])) == want, (i, e)


def test_special_values_on_import():
    x = np.array([np.nan, np.inf, -np.inf, 0.0, -0.0, 1e30, -1e30], np.float32)
    theta, comp = oracle_quantize(x, 8, 8, 0, -7)
    assert list(theta) == [0, 127, -127, 0, 0, 127, -127]
    assert list(comp[:5]) == [0, 0, 0, 0, 0] and list(comp[5:]) == [127, -127]
