"""Bit-exact parity of strict Algorithm 1 (kahan_sgd_strict_*: every statement rounded into
the stored format, the compensation with its own exponent) between the CUDA library and the
CPU oracle, with binary32 and with fixed-point gradients."""
import numpy as np
import pytest

from harness import LibraryRun, assert_same_state, make_oracle_state, storage_dtype
from oracle import (EXP_AMAX, EXP_FIXED, oracle_dequantize_gradient, oracle_max_threads, oracle_strict_step)
from paper_1810_05486_b200 import workloads as W

pytestmark = pytest.mark.gpu

FORMATS = [(8, 8), (8, 16), (16, 8), (16, 16)]


def qmax(b):
    return 2 ** (b - 1) - 1


def random_state(rng, n, tb, cb, full=False):
    lo_t, hi_t = (-2 ** (tb - 1), 2 ** (tb - 1)) if full else (-qmax(tb) // 2, qmax(tb) // 2)
    lo_c, hi_c = (-2 ** (cb - 1), 2 ** (cb - 1)) if full else (-qmax(cb) // 2, qmax(cb) // 2)
    return (rng.integers(lo_t, hi_t, n).astype(storage_dtype(tb)),
            rng.integers(lo_c, hi_c, n).astype(storage_dtype(cb)))


def run_both(specs, thetas, comps, grads_per_step, lrs, mode=EXP_AMAX, qgrad_exps=None):
    gpu = LibraryRun(specs, thetas, comps, mode, strict=True)
    ost = make_oracle_state(specs, thetas, comps, mode, oracle_max_threads())
    try:
        for step, grads in enumerate(grads_per_step):
            if qgrad_exps is None:
                gpu.step(grads, lrs)
                oracle_strict_step(ost, [g.copy() for g in grads], lrs)
            else:
                gpu.step_qgrad(grads, qgrad_exps[step], lrs)
                oracle_strict_step(ost, [oracle_dequantize_gradient(q, e) for q, e in zip(grads, qgrad_exps[step])],
                                   lrs)
            assert_same_state(gpu, ost, f"step {step}")
        assert gpu.guards_intact()
    finally:
        gpu.close()
    return ost


@pytest.mark.parametrize("tb,cb", FORMATS)
def test_every_format_ragged_sizes_many_steps_exponents_free(tb, cb):
    rng = np.random.default_rng(tb * 100 + cb)
    sizes = [1, 15, 16, 17, 4097, 8191, 8192, 8193, 3 * 8192 + 4095, 100003]
    e_t = -9 if tb == 8 else -15
    specs, thetas, comps = [], [], []
    for i, n in enumerate(sizes):
        t, c = random_state(rng, n, tb, cb)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=e_t, exp_comp=e_t - (cb - 1) - (i % 3)))
        thetas.append(t); comps.append(c)
    # increments from far below to well above the accumulator's unit
    grads = [[(rng.standard_normal(n) * 2.0 ** (e_t - cb) * (0.01, 3.0, 40.0, 0.5, 900.0, 1.0, 1.0, 0.2)[k] / 0.1)
              .astype(np.float32) for n in sizes] for k in range(8)]
    ost = run_both(specs, thetas, comps, grads, [0.1] * len(sizes))
    assert any(t.exp_comp != s["exp_comp"] for t, s in zip(ost.tensors, specs))


@pytest.mark.parametrize("gap", [-8, -3, 0, 1, 7, 15, 22, 23, 30, 36])
def test_every_distance_between_the_two_grids(gap):
    """e - ec from the accumulator coarser than theta (negative) to 36 binades finer, fixed
    exponents: the exact-fp32 path where it applies, the integer path elsewhere."""
    rng = np.random.default_rng(500 + gap)
    n = 40009
    specs, thetas, comps, grads = [], [], [], []
    for (tb, cb) in FORMATS:
        t, c = random_state(rng, n, tb, cb, full=True)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=-10, exp_comp=-10 - gap))
        thetas.append(t); comps.append(c)
        grads.append((rng.standard_normal(n) * 2.0 ** (-10 - gap) * 20).astype(np.float32))
    run_both(specs, thetas, comps, [grads] * 3, [1.0] * 4, EXP_FIXED)


@pytest.mark.parametrize("d_theta,d_comp", [(0, 3), (0, -8), (2, 0), (-8, 8), (8, -8), (-1, -1), (5, 8)])
def test_exponent_changes_of_theta_and_of_the_accumulator(d_theta, d_comp):
    rng = np.random.default_rng(900 + 17 * d_theta + d_comp)
    n = 30011
    specs, thetas, comps, grads = [], [], [], []
    for (tb, cb) in FORMATS:
        t, c = random_state(rng, n, tb, cb, full=True)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=-10, exp_theta_next=-10 + d_theta,
                          exp_comp=-20, exp_comp_next=-20 + d_comp))
        thetas.append(t); comps.append(c)
        g = (rng.standard_normal(n) * 2.0 ** -20 * 50).astype(np.float32)
        g[rng.choice(n, 40, replace=False)] = np.array([np.inf, -np.inf, np.nan, 3e38, 1e-45], np.float32)[
            np.arange(40) % 5]
        grads.append(g)
    run_both(specs, thetas, comps, [grads] * 2, [1.0] * 4, EXP_AMAX)


@pytest.mark.parametrize("gb", [8, 16])
def test_fixed_point_gradients_and_a_long_list(gb):
    """Both hardware-faithful modes together: INT8/INT16 gradients into the strict update."""
    rng = np.random.default_rng(300 + gb)
    n_t = 280
    sizes = [int(x) for x in rng.integers(1, 3000, n_t)]
    sizes[9], sizes[270] = 8192 * 2 + 77, 60000
    specs, thetas, comps = [], [], []
    for i, n in enumerate(sizes):
        tb, cb = FORMATS[i % 4]
        t, c = random_state(rng, n, tb, cb)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=-10, exp_comp=-10 - int(rng.integers(0, 20))))
        thetas.append(t); comps.append(c)
    grads = [[rng.integers(-2 ** (gb - 1), 2 ** (gb - 1), n).astype(storage_dtype(gb)) for n in sizes]
             for _ in range(4)]
    exps = [[s["exp_comp"] - gb + 3 + int(rng.integers(-3, 4)) for s in specs] for _ in range(4)]
    run_both(specs, thetas, comps, grads, [float(x) for x in rng.choice([0.1, 0.5, 1.0], n_t)], EXP_AMAX, exps)


def test_resnet20_shapes_forty_steps():
    wl = W.workload("c2_resnet20")
    thetas, comps = W.initial_state(wl)
    specs = [dict(numel=t.numel, theta_bits=t.theta_bits, comp_bits=t.comp_bits, exp_theta=t.exp_theta,
                  exp_comp=t.exp_theta - (t.comp_bits - 1)) for t in wl.tensors]
    grads = [W.gradients(wl, s) for s in range(40)]
    run_both(specs, thetas, comps, grads, [wl.lr] * len(specs))


def test_entry_points_of_the_other_kind_are_refused():
    from paper_1810_05486_b200 import binding as B
    rng = np.random.default_rng(1)
    t, c = random_state(rng, 1000, 8, 8)
    spec = dict(numel=1000, theta_bits=8, comp_bits=8, exp_theta=-9, exp_comp=-16)
    strict = LibraryRun([spec], [t], [c], EXP_AMAX, strict=True)
    plain = LibraryRun([spec], [t], [c], EXP_AMAX)
    try:
        with pytest.raises(B.KahanSgdError) as ei:
            strict.set_exponents([-9])
        assert ei.value.code == B.KSGD_ERR_MODE
        with pytest.raises(B.KahanSgdError) as ei:
            B.kahan_sgd_strict_exponents(plain.handle, 1)
        assert ei.value.code == B.KSGD_ERR_MODE
    finally:
        strict.close()
        plain.close()
