"""Bit-exact parity of the ADAM variant (16-bit moment tensors, Algorithm 1 with
lr_t * m / (sqrt(v) + eps) as the increment) between the CUDA library, through its C ABI, and
the CPU oracle: parameter, compensation and both moment mantissas, the three pairs of
exponents, the four max scans and the five counters, after every step."""
import numpy as np
import pytest

from harness import DeviceArena, storage_dtype
from oracle import EXP_AMAX, EXP_FIXED, OracleState, OracleTensor, oracle_adam_step, oracle_max_threads
from paper_1810_05486_b200 import workloads as W

pytestmark = pytest.mark.gpu

FORMATS = [(8, 8), (16, 8), (8, 16), (16, 16)]


def qmax(b):
    return 2 ** (b - 1) - 1


def bias_corrected(eta, b1, b2, t):
    c1 = 1.0 - b1 ** t if b1 < 1.0 else 1.0
    c2 = 1.0 - b2 ** t if b2 < 1.0 else 1.0
    return float(np.float32(eta * np.sqrt(c2) / c1))


class AdamRun:
    """Drives kahan_sgd_adam_* on device copies of the given tensors."""

    def __init__(self, specs, thetas, comps, m1s, m2s, mode):
        import torch
        from paper_1810_05486_b200 import binding as B
        self.B, self.torch, self.specs, self.n = B, torch, specs, len(specs)
        self.th = DeviceArena([s["numel"] * (s["theta_bits"] // 8) for s in specs])
        self.c = DeviceArena([s["numel"] * (s["comp_bits"] // 8) for s in specs])
        self.m1 = DeviceArena([s["numel"] * 2 for s in specs])
        self.m2 = DeviceArena([s["numel"] * 2 for s in specs])
        self.g = DeviceArena([s["numel"] * 4 for s in specs])
        for i in range(self.n):
            self.th.upload(i, thetas[i])
            self.c.upload(i, comps[i])
            self.m1.upload(i, m1s[i])
            self.m2.upload(i, m2s[i])
        self.descs = B.make_descs([
            dict(theta=self.th.ptr(i), comp=self.c.ptr(i), numel=s["numel"], theta_bits=s["theta_bits"],
                 comp_bits=s["comp_bits"], overlap_k=s.get("overlap_k", 0), exp_theta=s["exp_theta"],
                 exp_theta_next=s.get("exp_theta_next", s["exp_theta"])) for i, s in enumerate(specs)])
        self.adescs = B.make_adam_descs([
            dict(mom1=self.m1.ptr(i), mom2=self.m2.ptr(i), exp_m=s["exp_m"],
                 exp_m_next=s.get("exp_m_next", s["exp_m"]), exp_v=s["exp_v"],
                 exp_v_next=s.get("exp_v_next", s["exp_v"])) for i, s in enumerate(specs)])
        nb = B.kahan_sgd_adam_workspace_bytes(self.descs, self.adescs)
        assert nb > 0
        self.ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
        self.h = B.kahan_sgd_adam_init(self.descs, self.adescs, mode, self.ws.data_ptr(), nb,
                                       torch.cuda.current_stream().cuda_stream)

    def step(self, grads, lrs, b1, b2, eps):
        for i, g in enumerate(grads):
            self.g.upload(i, g)
        self.B.kahan_sgd_adam_step(self.h, [self.g.ptr(i) for i in range(self.n)], list(lrs), b1, b2, eps)

    def check(self, ost, where):
        st = self.B.kahan_sgd_adam_amax(self.h, self.n)
        for i, (s, t) in enumerate(zip(self.specs, ost.tensors)):
            tag = f"{where} tensor {i} {s}"
            for name, arena, bits, want in (("theta", self.th, s["theta_bits"], t.theta),
                                            ("comp", self.c, s["comp_bits"], t.comp),
                                            ("m", self.m1, 16, t.mom), ("v", self.m2, 16, t.mom2)):
                got = arena.download(i, storage_dtype(bits))
                assert np.array_equal(got, want), f"{tag}: {name} differs at {np.flatnonzero(got != want)[:8]}"
            assert (st["exp_theta_cur"][i], st["exp_theta_next"][i]) == (t.exp_theta, t.exp_theta_next), tag
            assert (st["exp_m_cur"][i], st["exp_m_next"][i]) == (t.exp_mom, t.exp_mom_next), tag
            assert (st["exp_v_cur"][i], st["exp_v_next"][i]) == (t.exp_mom2, t.exp_mom2_next), tag
            assert (st["amax_theta"][i], st["amax_comp"][i], st["amax_m"][i], st["amax_v"][i]) == \
                (t.amax_theta, t.amax_comp, t.amax_mom, t.amax_mom2), tag
            assert (st["n_sat_theta"][i], st["n_sat_comp"][i], st["n_sat_m"][i], st["n_sat_v"][i],
                    st["n_nonfinite"][i]) == \
                (t.n_sat_theta, t.n_sat_comp, t.n_sat_mom, t.n_sat_mom2, t.n_nonfinite), tag

    def guards_intact(self):
        self.torch.cuda.synchronize()
        return all(a.guards_intact() for a in (self.th, self.c, self.m1, self.m2, self.g))

    def close(self):
        self.B.kahan_sgd_adam_destroy(self.h)


def oracle_state(specs, thetas, comps, m1s, m2s, mode):
    return OracleState([OracleTensor(t.copy(), c.copy(), s["theta_bits"], s["comp_bits"], s.get("overlap_k", 0),
                                     s["exp_theta"], s.get("exp_theta_next", s["exp_theta"]), mom=a.copy(),
                                     mom_bits=16, exp_mom=s["exp_m"], exp_mom_next=s.get("exp_m_next", s["exp_m"]),
                                     mom2=b.copy(), exp_mom2=s["exp_v"],
                                     exp_mom2_next=s.get("exp_v_next", s["exp_v"]))
                        for s, t, c, a, b in zip(specs, thetas, comps, m1s, m2s)], mode, oracle_max_threads())


def run_both(specs, thetas, comps, m1s, m2s, grads_per_step, lrs_per_step, b1, b2, eps, mode=EXP_AMAX):
    gpu = AdamRun(specs, thetas, comps, m1s, m2s, mode)
    ost = oracle_state(specs, thetas, comps, m1s, m2s, mode)
    try:
        for step, (grads, lrs) in enumerate(zip(grads_per_step, lrs_per_step)):
            gpu.step(grads, lrs, b1, b2, eps)
            oracle_adam_step(ost, [g.copy() for g in grads], lrs, b1, b2, eps)
            gpu.check(ost, f"step {step}")
        assert gpu.guards_intact()
    finally:
        gpu.close()
    return ost


def random_state(rng, n, tb, cb, k=0, full=False, zero_moments=False):
    s = cb - 1 - k
    theta = rng.integers(-2 ** (tb - 1) if full else -qmax(tb) // 2, 2 ** (tb - 1) if full else qmax(tb) // 2,
                         n).astype(storage_dtype(tb))
    lim = 2 ** (cb - 1) if full else max(1, 2 ** (s - 1))
    comp = rng.integers(-lim, lim, n).astype(storage_dtype(cb))
    if zero_moments:
        return theta, comp, np.zeros(n, np.int16), np.zeros(n, np.int16)
    m1 = rng.integers(-32768 if full else -9000, 32768 if full else 9000, n).astype(np.int16)
    m2 = rng.integers(-32768 if full else 0, 32768 if full else 9000, n).astype(np.int16)
    return theta, comp, m1, m2


def moment_exponents(sigma, b1, b2):
    """Exponents that hold a first moment of about 4 sigma and a second of about 16 sigma^2."""
    return int(np.ceil(np.log2(4 * sigma / 32767))), int(np.ceil(np.log2(16 * sigma ** 2 / 32767)))


@pytest.mark.parametrize("tb,cb", FORMATS)
def test_every_format_ragged_sizes_many_steps_from_zero_moments(tb, cb):
    rng = np.random.default_rng(tb * 100 + cb)
    sizes = [1, 15, 16, 17, 4097, 8191, 8192, 8193, 3 * 8192 + 4095, 100003]
    e_t = -9 if tb == 8 else -15
    sigma, eta, b1, b2, eps = 0.01, 2.0 ** (e_t + 1), 0.9, 0.999, 1e-8
    e_m, e_v = moment_exponents(sigma, b1, b2)
    specs, thetas, comps, m1s, m2s = [], [], [], [], []
    for n in sizes:
        t, c, a, b = random_state(rng, n, tb, cb, zero_moments=True)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=e_t, exp_m=e_m - 3, exp_v=e_v - 9))
        thetas.append(t); comps.append(c); m1s.append(a); m2s.append(b)
    steps = 10
    grads = [[(rng.standard_normal(n) * sigma + 0.3 * sigma).astype(np.float32) for n in sizes]
             for _ in range(steps)]
    lrs = [[bias_corrected(eta, b1, b2, t + 1)] * len(sizes) for t in range(steps)]
    ost = run_both(specs, thetas, comps, m1s, m2s, grads, lrs, b1, b2, eps)
    assert any(t.exp_mom != e_m - 3 for t in ost.tensors) and any(t.exp_mom2 != e_v - 9 for t in ost.tensors)


@pytest.mark.parametrize("tb,cb", [(8, 8), (16, 16), (16, 8)])
def test_full_range_inputs_saturation_and_non_finite_gradients(tb, cb):
    rng = np.random.default_rng(5 + tb + cb)
    n = 60013
    t, c, a, b = random_state(rng, n, tb, cb, full=True)
    specs = [dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=-9, exp_m=-20, exp_v=-30)]
    grads = []
    for step in range(5):
        g = (rng.standard_t(3, n) * 2.0 ** -20 * 32767 * (0.01, 0.3, 2.0, 1e-4, 50.0)[step]).astype(np.float32)
        idx = rng.choice(n, 300, replace=False)
        g[idx] = np.array([np.inf, -np.inf, np.nan, 3e38, -3e38, 1e-45, 0.0], np.float32)[np.arange(300) % 7]
        grads.append([g])
    ost = run_both(specs, [t], [c], [a], [b], grads, [[0.02]] * 5, 0.9, 0.999, 1e-8, EXP_FIXED)
    o = ost.tensors[0]
    assert o.n_sat_mom > 0 and o.n_sat_mom2 > 0 and o.n_sat_theta > 0 and o.n_nonfinite > 0


@pytest.mark.parametrize("b1,b2,eps", [(0.0, 0.0, 0.0), (0.5, 0.9, 1e-3), (1.0, 1.0, 0.0), (0.9, 0.999, 0.0),
                                       (0.9, 0.999, 1.0)])
def test_coefficient_corners_and_zero_denominators(b1, b2, eps):
    """eps = 0 with second moments that are or round to zero (taken as one unit of the grid);
    beta = 1 freezes a moment; beta = 0 makes it the quantized gradient."""
    rng = np.random.default_rng(int(b1 * 10) + int(b2 * 1000))
    n = 50021
    specs, thetas, comps, m1s, m2s, grads = [], [], [], [], [], []
    for (tb, cb) in FORMATS:
        t, c, a, b = random_state(rng, n, tb, cb)
        a[::3] = 0
        b[::2] = 0
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=-10, exp_m=-21, exp_v=-36))
        thetas.append(t); comps.append(c); m1s.append(a); m2s.append(b)
        g = (rng.standard_normal(n) * 0.004).astype(np.float32)
        g[::5] = 0.0
        grads.append(g)
    run_both(specs, thetas, comps, m1s, m2s, [grads] * 3, [[2.0 ** -12] * 4] * 3, b1, b2, eps, EXP_FIXED)


@pytest.mark.parametrize("d_theta,d_m,d_v", [(0, 0, 3), (0, -2, 0), (1, 0, 0), (-8, 8, -8), (8, -8, 8), (-1, 1, 2)])
def test_exponent_changes_of_theta_and_of_each_moment(d_theta, d_m, d_v):
    rng = np.random.default_rng(1000 + d_theta * 31 + d_m * 7 + d_v)
    n = 40009
    specs, thetas, comps, m1s, m2s, grads = [], [], [], [], [], []
    for (tb, cb) in FORMATS:
        t, c, a, b = random_state(rng, n, tb, cb)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=-10, exp_theta_next=-10 + d_theta,
                          exp_m=-21, exp_m_next=-21 + d_m, exp_v=-36, exp_v_next=-36 + d_v))
        thetas.append(t); comps.append(c); m1s.append(a); m2s.append(b)
        grads.append((rng.standard_normal(n) * 0.004).astype(np.float32))
    run_both(specs, thetas, comps, m1s, m2s, [grads] * 2, [[2.0 ** -11] * 4] * 2, 0.9, 0.999, 1e-8, EXP_FIXED)


def test_large_steps_that_clamp_the_increment_and_overlap_formats():
    rng = np.random.default_rng(88)
    n = 30000
    specs, thetas, comps, m1s, m2s, grads = [], [], [], [], [], []
    for k in (0, 3, 7):
        t, c, a, b = random_state(rng, n, 8, 8, k)
        specs.append(dict(numel=n, theta_bits=8, comp_bits=8, overlap_k=k, exp_theta=-8, exp_m=-21, exp_v=-36))
        thetas.append(t); comps.append(c); m1s.append(a); m2s.append(b)
        grads.append((rng.standard_normal(n) * 0.004).astype(np.float32))
    for lr in (1e-6, 0.3, 3e4, 3e30):
        run_both(specs, thetas, comps, m1s, m2s, [grads] * 2, [[lr] * 3] * 2, 0.9, 0.999, 1e-8, EXP_AMAX)


def test_resnet20_shapes_with_the_two_adam_settings_of_the_paper():
    """beta1 = 0.9, beta2 = 0.999 (Section 4) and beta1 = 0.5, beta2 = 0.9, eps = 1e-3 (the
    GAN experiment), on the tensor list of the small CNN with INT16 weights and moments."""
    wl = W.workload("c2_resnet20")
    thetas8, _ = W.initial_state(wl)
    for (b1, b2, eps, eta) in ((0.9, 0.999, 1e-8, 1e-3), (0.5, 0.9, 1e-3, 1e-4)):
        thetas = [t.astype(np.int16) * 256 for t in thetas8]
        specs = [dict(numel=t.numel, theta_bits=16, comp_bits=16, exp_theta=t.exp_theta - 8,
                      exp_m=-30, exp_v=-45) for t in wl.tensors]
        comps = [np.zeros(t.numel, np.int16) for t in wl.tensors]
        m1s = [np.zeros(t.numel, np.int16) for t in wl.tensors]
        m2s = [np.zeros(t.numel, np.int16) for t in wl.tensors]
        steps = 25
        grads = [W.gradients(wl, s) for s in range(steps)]
        lrs = [[bias_corrected(eta, b1, b2, s + 1)] * len(specs) for s in range(steps)]
        run_both(specs, thetas, comps, m1s, m2s, grads, lrs, b1, b2, eps)


def test_fast_path_division_and_square_root_equal_the_correctly_rounded_operations():
    """Exhaustive over the operands the fast path can meet (see the header)."""
    from paper_1810_05486_b200 import binding as B
    assert B.kahan_sgd_adam_selfcheck() == (0, 0)


def test_a_list_longer_than_the_inline_argument_block():
    """More than 256 tensors: gradients and step sizes reach the kernel through the workspace
    instead of the kernel parameters."""
    rng = np.random.default_rng(902)
    n_t = 300
    sizes = [int(x) for x in rng.integers(1, 3000, n_t)]
    sizes[17], sizes[290] = 8192 * 2 + 5, 40000
    specs, thetas, comps, m1s, m2s = [], [], [], [], []
    for i, n in enumerate(sizes):
        tb, cb = FORMATS[i % 4]
        t, c, a, b = random_state(rng, n, tb, cb)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, exp_theta=-10, exp_m=-21, exp_v=-36))
        thetas.append(t); comps.append(c); m1s.append(a); m2s.append(b)
    grads = [[(rng.standard_normal(n) * 0.004).astype(np.float32) for n in sizes] for _ in range(3)]
    lrs = [[float(x) for x in rng.choice([2.0 ** -12, 2.0 ** -11, 3e-4], n_t)] for _ in range(3)]
    run_both(specs, thetas, comps, m1s, m2s, grads, lrs, 0.9, 0.999, 1e-8)
