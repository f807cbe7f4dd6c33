"""Bit-exact parity of the momentum variant (v <- mu v + eta g, Algorithm 1 with v) between
the CUDA library, through its C ABI, and the CPU oracle: parameter, compensation and
velocity mantissas, both pairs of exponents, the three max scans and the four counters,
after every step."""
import numpy as np
import pytest

from harness import DeviceArena, storage_dtype
from oracle import EXP_AMAX, EXP_FIXED, OracleState, OracleTensor, oracle_max_threads, oracle_momentum_step
from paper_1810_05486_b200 import workloads as W

pytestmark = pytest.mark.gpu

FORMATS = [(8, 8, 8), (16, 8, 8), (8, 16, 8), (16, 16, 8), (8, 8, 16), (16, 8, 16), (8, 16, 16), (16, 16, 16)]


def qmax(b):
    return 2 ** (b - 1) - 1


class MomentumRun:
    """Drives kahan_sgd_momentum_* on device copies of the given tensors."""

    def __init__(self, specs, thetas, comps, moms, mode):
        import torch
        from paper_1810_05486_b200 import binding as B
        self.B, self.torch, self.specs, self.n = B, torch, specs, len(specs)
        self.th = DeviceArena([s["numel"] * (s["theta_bits"] // 8) for s in specs])
        self.c = DeviceArena([s["numel"] * (s["comp_bits"] // 8) for s in specs])
        self.v = DeviceArena([s["numel"] * (s["mom_bits"] // 8) for s in specs])
        self.g = DeviceArena([s["numel"] * 4 for s in specs])
        for i in range(self.n):
            self.th.upload(i, thetas[i])
            self.c.upload(i, comps[i])
            self.v.upload(i, moms[i])
        self.descs = B.make_descs([
            dict(theta=self.th.ptr(i), comp=self.c.ptr(i), numel=s["numel"], theta_bits=s["theta_bits"],
                 comp_bits=s["comp_bits"], overlap_k=s.get("overlap_k", 0), exp_theta=s["exp_theta"],
                 exp_theta_next=s.get("exp_theta_next", s["exp_theta"])) for i, s in enumerate(specs)])
        self.mdescs = B.make_momentum_descs([
            dict(mom=self.v.ptr(i), mom_bits=s["mom_bits"], exp_mom=s["exp_mom"],
                 exp_mom_next=s.get("exp_mom_next", s["exp_mom"])) for i, s in enumerate(specs)])
        nb = B.kahan_sgd_momentum_workspace_bytes(self.descs, self.mdescs)
        assert nb > 0
        self.ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
        self.h = B.kahan_sgd_momentum_init(self.descs, self.mdescs, mode, self.ws.data_ptr(), nb,
                                           torch.cuda.current_stream().cuda_stream)

    def step(self, grads, lrs, mus):
        for i, g in enumerate(grads):
            self.g.upload(i, g)
        self.B.kahan_sgd_momentum_step(self.h, [self.g.ptr(i) for i in range(self.n)], list(lrs), list(mus))

    def check(self, ost, where):
        st = self.B.kahan_sgd_momentum_amax(self.h, self.n)
        for i, (s, t) in enumerate(zip(self.specs, ost.tensors)):
            tag = f"{where} tensor {i} {s}"
            for name, arena, bits, want in (("theta", self.th, s["theta_bits"], t.theta),
                                            ("comp", self.c, s["comp_bits"], t.comp),
                                            ("mom", self.v, s["mom_bits"], t.mom)):
                got = arena.download(i, storage_dtype(bits))
                assert np.array_equal(got, want), f"{tag}: {name} differs at {np.flatnonzero(got != want)[:8]}"
            assert (st["exp_theta_cur"][i], st["exp_theta_next"][i]) == (t.exp_theta, t.exp_theta_next), tag
            assert (st["exp_mom_cur"][i], st["exp_mom_next"][i]) == (t.exp_mom, t.exp_mom_next), tag
            assert (st["amax_theta"][i], st["amax_comp"][i], st["amax_mom"][i]) == \
                (t.amax_theta, t.amax_comp, t.amax_mom), tag
            assert (st["n_sat_theta"][i], st["n_sat_comp"][i], st["n_sat_mom"][i], st["n_nonfinite"][i]) == \
                (t.n_sat_theta, t.n_sat_comp, t.n_sat_mom, t.n_nonfinite), tag

    def guards_intact(self):
        self.torch.cuda.synchronize()
        return all(a.guards_intact() for a in (self.th, self.c, self.v, self.g))

    def close(self):
        self.B.kahan_sgd_momentum_destroy(self.h)


def oracle_state(specs, thetas, comps, moms, mode):
    return OracleState([OracleTensor(t.copy(), c.copy(), s["theta_bits"], s["comp_bits"], s.get("overlap_k", 0),
                                     s["exp_theta"], s.get("exp_theta_next", s["exp_theta"]), mom=v.copy(),
                                     mom_bits=s["mom_bits"], exp_mom=s["exp_mom"],
                                     exp_mom_next=s.get("exp_mom_next", s["exp_mom"]))
                        for s, t, c, v in zip(specs, thetas, comps, moms)], mode, oracle_max_threads())


def run_both(specs, thetas, comps, moms, grads_per_step, lrs, mus, mode=EXP_AMAX):
    gpu = MomentumRun(specs, thetas, comps, moms, mode)
    ost = oracle_state(specs, thetas, comps, moms, mode)
    try:
        for step, grads in enumerate(grads_per_step):
            gpu.step(grads, lrs, mus)
            oracle_momentum_step(ost, [g.copy() for g in grads], lrs, mus)
            gpu.check(ost, f"step {step}")
        assert gpu.guards_intact()
    finally:
        gpu.close()
    return ost


def random_state(rng, n, tb, cb, vb, k=0, full=False):
    s = cb - 1 - k
    theta = rng.integers(-2 ** (tb - 1) if full else -qmax(tb) // 2, 2 ** (tb - 1) if full else qmax(tb) // 2,
                         n).astype(storage_dtype(tb))
    lim = 2 ** (cb - 1) if full else max(1, 2 ** (s - 1))
    comp = rng.integers(-lim, lim, n).astype(storage_dtype(cb))
    mom = rng.integers(-2 ** (vb - 1) if full else -qmax(vb) // 3, 2 ** (vb - 1) if full else qmax(vb) // 3,
                       n).astype(storage_dtype(vb))
    return theta, comp, mom


@pytest.mark.parametrize("tb,cb,vb", FORMATS)
def test_every_format_ragged_sizes_many_steps(tb, cb, vb):
    rng = np.random.default_rng(tb * 100 + cb * 10 + vb)
    sizes = [1, 15, 16, 17, 4097, 8191, 8192, 8193, 3 * 8192 + 4095, 100003]
    e_t = -9 if tb == 8 else -15
    s = cb - 1
    e_v = e_t - 6                                    # velocity grid between theta's and c's
    specs, thetas, comps, moms = [], [], [], []
    for n in sizes:
        t, c, v = random_state(rng, n, tb, cb, vb)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, mom_bits=vb, exp_theta=e_t, exp_mom=e_v))
        thetas.append(t); comps.append(c); moms.append(v)
    sigma = 2.0 ** e_v * qmax(vb) * 0.02 / 0.1
    grads = [[(rng.standard_normal(n) * sigma).astype(np.float32) for n in sizes] for _ in range(8)]
    ost = run_both(specs, thetas, comps, moms, grads, [0.1] * len(sizes), [0.9] * len(sizes))
    assert any(t.exp_mom != e_v or t.exp_theta != e_t for t in ost.tensors)    # exponents did move


@pytest.mark.parametrize("tb,cb,vb", [(8, 8, 8), (16, 16, 16), (16, 8, 16)])
def test_full_range_inputs_saturation_and_non_finite_gradients(tb, cb, vb):
    rng = np.random.default_rng(5 + tb + vb)
    n = 60013
    t, c, v = random_state(rng, n, tb, cb, vb, full=True)
    specs = [dict(numel=n, theta_bits=tb, comp_bits=cb, mom_bits=vb, exp_theta=-9, exp_mom=-12)]
    grads = []
    for step in range(5):
        g = (rng.standard_t(3, n) * 2.0 ** -12 * qmax(vb) * (0.01, 0.3, 2.0, 1e-4, 50.0)[step]).astype(np.float32)
        idx = rng.choice(n, 300, replace=False)
        g[idx] = np.array([np.inf, -np.inf, np.nan, 3e38, -3e38, 1e-45, 0.0], np.float32)[np.arange(300) % 7]
        grads.append([g])
    ost = run_both(specs, [t], [c], [v], grads, [1.0], [0.9], EXP_FIXED)
    assert ost.tensors[0].n_sat_mom > 0 and ost.tensors[0].n_sat_theta > 0 and ost.tensors[0].n_nonfinite > 0


@pytest.mark.parametrize("k_shift", [-20, -6, -1, 0, 1, 5, 9, 16, 25])
def test_velocity_grid_above_and_below_the_compensation_grid(k_shift):
    """k = ev - ec from far below (the velocity never reaches theta) to far above (every
    non-zero velocity is clamped) the compensation grid."""
    rng = np.random.default_rng(300 + k_shift)
    n = 30011
    specs, thetas, comps, moms, grads = [], [], [], [], []
    for (tb, cb, vb) in ((8, 8, 8), (16, 8, 16), (16, 16, 8)):
        s = cb - 1
        e_t = -10
        e_v = e_t - s + k_shift
        t, c, v = random_state(rng, n, tb, cb, vb)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, mom_bits=vb, exp_theta=e_t, exp_mom=e_v))
        thetas.append(t); comps.append(c); moms.append(v)
        grads.append((rng.standard_normal(n) * 2.0 ** e_v * 9).astype(np.float32))
    run_both(specs, thetas, comps, moms, [grads, grads, grads], [1.0] * 3, [0.5, 0.9, 0.99], EXP_FIXED)


def test_momentum_zero_and_large_coefficients_and_overlap():
    rng = np.random.default_rng(77)
    n = 20000
    specs, thetas, comps, moms, grads = [], [], [], [], []
    for k in (0, 3, 7):
        t, c, v = random_state(rng, n, 8, 8, 16, k)
        specs.append(dict(numel=n, theta_bits=8, comp_bits=8, mom_bits=16, overlap_k=k, exp_theta=-8, exp_mom=-16))
        thetas.append(t); comps.append(c); moms.append(v)
        grads.append((rng.standard_normal(n) * 2.0 ** -16 * 300).astype(np.float32))
    run_both(specs, thetas, comps, moms, [grads] * 4, [0.5] * 3, [0.0, 1.0, 1.5], EXP_AMAX)


def test_resnet20_shapes_int8_momentum_and_alexnet_last_layers_int16_momentum():
    """The two momentum settings the paper reports: mu = 0.9 in INT8 for the small CNNs and
    in INT16 for AlexNet (only its two smallest weight layers here, to keep the test short)."""
    wl = W.workload("c2_resnet20")
    thetas, comps = W.initial_state(wl)
    specs = [dict(numel=t.numel, theta_bits=8, comp_bits=8, mom_bits=8, exp_theta=t.exp_theta,
                  exp_mom=t.exp_theta - 7) for t in wl.tensors]
    moms = [np.zeros(t.numel, np.int8) for t in wl.tensors]
    grads = [W.gradients(wl, s) for s in range(40)]
    run_both(specs, thetas, comps, moms, grads, [wl.lr] * len(specs), [0.9] * len(specs))

    a = W.workload("c4_alexnet")
    pick = [i for i, t in enumerate(a.tensors) if t.name in ("conv1.weight", "conv2.weight", "fc8.weight", "fc8.bias")]
    specs = [dict(numel=a.tensors[i].numel, theta_bits=a.tensors[i].theta_bits, comp_bits=a.tensors[i].comp_bits,
                  mom_bits=16, exp_theta=a.tensors[i].exp_theta, exp_mom=a.tensors[i].exp_theta - 8) for i in pick]
    thetas = [W.theta_slice(a, i, 0, a.tensors[i].numel) for i in pick]
    comps = [np.zeros(a.tensors[i].numel, storage_dtype(a.tensors[i].comp_bits)) for i in pick]
    moms = [np.zeros(a.tensors[i].numel, np.int16) for i in pick]
    grads = [[W.grad_slice(a, i, s, 0, a.tensors[i].numel) for i in pick] for s in range(10)]
    run_both(specs, thetas, comps, moms, grads, [a.lr] * len(pick), [0.9] * len(pick))


def test_a_list_longer_than_the_inline_argument_block():
    """More than 256 tensors: gradients, step sizes and momentum coefficients reach the
    kernel through the workspace instead of the kernel parameters."""
    rng = np.random.default_rng(901)
    n_t = 300
    sizes = [int(x) for x in rng.integers(1, 3000, n_t)]
    sizes[17], sizes[290] = 8192 * 2 + 5, 40000
    specs, thetas, comps, moms = [], [], [], []
    for i, n in enumerate(sizes):
        tb, cb, vb = FORMATS[i % len(FORMATS)]
        t, c, v = random_state(rng, n, tb, cb, vb)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, mom_bits=vb, exp_theta=-10, exp_mom=-17))
        thetas.append(t); comps.append(c); moms.append(v)
    grads = [[(rng.standard_normal(n) * 2.0 ** -17 * 400).astype(np.float32) for n in sizes] for _ in range(3)]
    lrs = [float(x) for x in rng.choice([0.05, 0.1, 0.2], n_t)]
    mus = [float(x) for x in rng.choice([0.0, 0.5, 0.9], n_t)]
    run_both(specs, thetas, comps, moms, grads, lrs, mus)
