"""Bit-exact parity of the step with fixed-point gradients (kahan_sgd_step_qgrad: INT8 or
INT16 gradient mantissas with one exponent per tensor, the paper's hardware model) between
the CUDA library and the CPU oracle."""
import numpy as np
import pytest

from harness import LibraryRun, assert_same_state, make_oracle_state, storage_dtype
from oracle import EXP_AMAX, EXP_FIXED, oracle_fit_exponent, oracle_max_threads, oracle_quantize, oracle_step_qgrad
from paper_1810_05486_b200 import workloads as W

pytestmark = pytest.mark.gpu

FORMATS = [(8, 0), (8, 8), (8, 16), (16, 0), (16, 8), (16, 16)]


def qmax(b):
    return 2 ** (b - 1) - 1


def random_state(rng, n, tb, cb, full=False):
    theta = rng.integers(-2 ** (tb - 1) if full else -qmax(tb) // 2, 2 ** (tb - 1) if full else qmax(tb) // 2,
                         n).astype(storage_dtype(tb))
    if not cb:
        return theta, None
    lim = 2 ** (cb - 1) if full else 2 ** (cb - 2)
    return theta, rng.integers(-lim, lim, n).astype(storage_dtype(cb))


def run_both(specs, thetas, comps, grads_per_step, exps_per_step, lrs, mode=EXP_AMAX):
    gpu = LibraryRun(specs, thetas, comps, mode)
    ost = make_oracle_state(specs, thetas, comps, mode, oracle_max_threads())
    try:
        for step, (gq, eg) in enumerate(zip(grads_per_step, exps_per_step)):
            gpu.step_qgrad(gq, eg, lrs)
            oracle_step_qgrad(ost, gq, eg, lrs)
            assert_same_state(gpu, ost, f"step {step}")
        assert gpu.guards_intact()
    finally:
        gpu.close()
    return ost


@pytest.mark.parametrize("gb", [8, 16])
@pytest.mark.parametrize("tb,cb", FORMATS)
def test_every_format_ragged_sizes_full_range_gradient_mantissas(tb, cb, gb):
    rng = np.random.default_rng(tb * 1000 + cb * 10 + gb)
    sizes = [1, 15, 16, 17, 4097, 8191, 8192, 8193, 3 * 8192 + 4095, 100003]
    e_t = -9 if tb == 8 else -15
    s = cb - 1 if cb else 0
    specs, thetas, comps = [], [], []
    for n in sizes:
        t, c = random_state(rng, n, tb, cb)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=e_t))
        thetas.append(t); comps.append(c)
    # gradient units worth 2^-4 .. 2^3 compensation units at lr = 0.1
    steps, grads, exps = 6, [], []
    for k in range(steps):
        grads.append([rng.integers(-2 ** (gb - 1), 2 ** (gb - 1), n).astype(storage_dtype(gb)) for n in sizes])
        exps.append([e_t - s - gb + 4 + int(rng.integers(-4, 4)) for _ in sizes])
    run_both(specs, thetas, comps, grads, exps, [0.1] * len(sizes))


@pytest.mark.parametrize("gb", [8, 16])
def test_gradient_exponents_at_the_ends_of_the_range_and_huge_and_tiny_step_sizes(gb):
    """Exponent sums that leave the binary32 range of the combined factor scale * 2^eg (the
    exact-fp32 path must hand such tiles to the integer path), increments that clamp, and
    increments that vanish."""
    rng = np.random.default_rng(40 + gb)
    n = 30011
    cases = [(-64, 1e-30), (-64, 3e38), (64, 1e-38), (64, 1e-20), (64, 1.0), (-40, 1e30), (0, 1e-45), (-20, 0.5)]
    specs, thetas, comps, exps, lrs = [], [], [], [], []
    for i, (eg, lr) in enumerate(cases):
        tb, cb = FORMATS[1 + i % 5]
        t, c = random_state(rng, n, tb, cb)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=-10))
        thetas.append(t); comps.append(c); exps.append(eg); lrs.append(float(np.float32(lr)))
    grads = [[rng.integers(-2 ** (gb - 1), 2 ** (gb - 1), n).astype(storage_dtype(gb)) for _ in cases]
             for _ in range(2)]
    run_both(specs, thetas, comps, grads, [exps, exps], lrs, EXP_FIXED)


@pytest.mark.parametrize("gb", [8, 16])
def test_exponent_changes_saturation_and_a_long_list(gb):
    rng = np.random.default_rng(77 + gb)
    n_t = 300
    sizes = [int(x) for x in rng.integers(1, 3000, n_t)]
    sizes[5], sizes[299] = 8192 * 3 + 11, 50000
    specs, thetas, comps = [], [], []
    for i, n in enumerate(sizes):
        tb, cb = FORMATS[i % 6]
        t, c = random_state(rng, n, tb, cb, full=(i % 7 == 0))
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=-10,
                          exp_theta_next=-10 + int(rng.integers(-8, 9))))
        thetas.append(t); comps.append(c)
    grads = [[rng.integers(-2 ** (gb - 1), 2 ** (gb - 1), n).astype(storage_dtype(gb)) for n in sizes]
             for _ in range(4)]
    exps = [[int(e) for e in rng.integers(-30, -14, n_t)] for _ in range(4)]
    lrs = [float(x) for x in rng.choice([0.01, 0.1, 1.0], n_t)]
    ost = run_both(specs, thetas, comps, grads, exps, lrs)
    assert sum(t.n_sat_theta for t in ost.tensors) > 0


def test_resnet20_shapes_with_gradients_quantized_by_the_import_rule():
    """The paper's pipeline: binary32 gradients -> INT8 tensors with the exponent from the
    maximum (the oracle's quantizer; the CUDA quantizer is checked against it elsewhere) ->
    lazy update."""
    wl = W.workload("c2_resnet20")
    thetas, comps = W.initial_state(wl)
    specs = [dict(numel=t.numel, theta_bits=t.theta_bits, comp_bits=t.comp_bits, exp_theta=t.exp_theta)
             for t in wl.tensors]
    grads, exps = [], []
    for step in range(30):
        gs = W.gradients(wl, step)
        e = [oracle_fit_exponent(g, 8) for g in gs]
        grads.append([oracle_quantize(g, 8, 0, 0, ei)[0] for g, ei in zip(gs, e)])
        exps.append(e)
    run_both(specs, thetas, comps, grads, exps, [wl.lr] * len(specs))


def test_int8_gradients_on_a_list_long_enough_for_the_second_tile_table_every_format():
    """Steps on 8-bit gradients of long lists walk their own tile table (32768 elements per
    tile for 8-bit theta with an 8-bit or no c, 16384 for everything else).  Six tensors, one
    per format, ragged sizes, 1300 such tiles in all; a step on 16-bit gradients and one on
    8-bit gradients again, on the same handle, follow (the first table and back)."""
    rng = np.random.default_rng(77)
    sizes = {(8, 0): 250 * 32768 + 5, (8, 8): 250 * 32768 + 32767, (8, 16): 200 * 16384 + 16383,
             (16, 0): 200 * 16384 + 1, (16, 8): 200 * 16384 + 8191, (16, 16): 200 * 16384 + 17}
    specs, thetas, comps = [], [], []
    for (tb, cb), n in sizes.items():
        t, c = random_state(rng, n, tb, cb)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=-9 if tb == 8 else -15))
        thetas.append(t); comps.append(c)

    def grads(gb):
        return [rng.integers(-2 ** (gb - 1), 2 ** (gb - 1), sp["numel"]).astype(storage_dtype(gb)) for sp in specs]

    def exps(gb):
        return [sp["exp_theta"] - (sp["comp_bits"] - 1 if sp["comp_bits"] else 0) - gb + 5 for sp in specs]
    lrs = [0.1] * len(specs)
    gpu = LibraryRun(specs, thetas, comps, EXP_AMAX)
    ost = make_oracle_state(specs, thetas, comps, EXP_AMAX, oracle_max_threads())
    try:
        for step, gb in enumerate((8, 8, 16, 8)):
            gq, eg = grads(gb), exps(gb)
            gpu.step_qgrad(gq, eg, lrs)
            oracle_step_qgrad(ost, gq, eg, lrs)
            assert_same_state(gpu, ost, f"step {step} ({gb}-bit gradients)")
        assert gpu.guards_intact()
    finally:
        gpu.close()
