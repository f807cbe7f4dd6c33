"""Bit-exact parity of the CUDA library (through its C ABI) with the CPU oracle.

Everything the step produces is compared: parameter mantissas, compensation mantissas,
current and next exponents, both max scans and the three counters, after every step.
"""
import numpy as np
import pytest

from harness import LibraryRun, assert_same_state, make_oracle_state, specs_of, storage_dtype
from oracle import EXP_AMAX, EXP_FIXED, oracle_step
from paper_1810_05486_b200 import workloads as W

pytestmark = pytest.mark.gpu

VARIANTS = [(8, 0), (8, 8), (8, 16), (16, 0), (16, 8), (16, 16)]


def qmax(b):
    return 2 ** (b - 1) - 1


def run_both(specs, thetas, comps, grads_per_step, lrs_per_step, mode=EXP_AMAX, exps_per_step=None):
    gpu = LibraryRun(specs, thetas, comps, mode)
    ost = make_oracle_state(specs, thetas, comps, mode)
    try:
        for step, (grads, lrs) in enumerate(zip(grads_per_step, lrs_per_step)):
            if exps_per_step is not None and exps_per_step[step] is not None:
                gpu.set_exponents(exps_per_step[step])
                for t, e in zip(ost.tensors, exps_per_step[step]):
                    t.exp_theta_next = e
            gpu.step(grads, lrs)
            oracle_step(ost, [g.copy() for g in grads], lrs)
            assert_same_state(gpu, ost, f"step {step}")
        assert gpu.guards_intact()
    finally:
        gpu.close()
    return ost


def random_tensor(rng, numel, tb, cb, k=0, full_range=True):
    s = cb - 1 - k if cb else 0
    lo_t = -2 ** (tb - 1) if full_range else -qmax(tb)
    theta = rng.integers(lo_t, 2 ** (tb - 1), numel).astype(storage_dtype(tb))
    comp = None
    if cb:
        lim = 2 ** (cb - 1) if full_range else max(1, 2 ** (s - 1))
        comp = rng.integers(-lim, lim, numel).astype(storage_dtype(cb))
    return theta, comp


# ----------------------------------------------------------------------------- exhaustive grid

def test_all_int8_pairs_times_gradient_sweep():
    """Every (Q_theta, Q_c) int8 pair, including the -128 codes, against a sweep of
    increments from far below one compensation LSB to far beyond the parameter range."""
    qt, qc = np.meshgrid(np.arange(-128, 128), np.arange(-128, 128), indexing="ij")
    theta = qt.ravel().astype(np.int8)
    comp = qc.ravel().astype(np.int8)
    e_t, s = -11, 7
    lsb = 2.0 ** (e_t - s)
    mults = [0.0, 0.25, 0.5, 0.75, 1.0, 1.5, 2.5, 3.5, 63.5, 64.0, 64.5, 127.5, 128.0, 128.5, 191.5,
             192.5, 1000.25, 16383.5, 16384.5, 40000.0, 3e6, 2.0 ** 30, 2.0 ** 31, 1e30]
    mults = mults + [-m for m in mults[1:]]
    specs = [dict(numel=theta.size, theta_bits=8, comp_bits=8, overlap_k=0, exp_theta=e_t)]
    grads = [[np.full(theta.size, np.float32(m * lsb / 0.25), np.float32)] for m in mults]
    gpu = LibraryRun(specs, [theta], [comp], EXP_FIXED)
    try:
        for m, g in zip(mults, grads):
            # same starting state for every increment: re-upload
            gpu.theta_arena.upload(0, theta)
            gpu.comp_arena.upload(0, comp)
            ost = make_oracle_state(specs, [theta], [comp], EXP_FIXED)
            prev = gpu.stats()
            gpu.step(g, [0.25])
            oracle_step(ost, [g[0].copy()], [0.25])
            got_t, got_c = gpu.thetas()[0], gpu.comps()[0]
            assert np.array_equal(got_t, ost.tensors[0].theta), m
            assert np.array_equal(got_c, ost.tensors[0].comp), m
            st = gpu.stats()
            assert st["amax_theta"][0] == ost.tensors[0].amax_theta, m
            assert st["amax_comp"][0] == ost.tensors[0].amax_comp, m
            assert st["n_sat_theta"][0] - prev["n_sat_theta"][0] == ost.tensors[0].n_sat_theta, m
            assert st["n_sat_comp"][0] - prev["n_sat_comp"][0] == ost.tensors[0].n_sat_comp, m
        assert gpu.guards_intact()
    finally:
        gpu.close()


# ----------------------------------------------------------------------------- ragged sizes, all variants

@pytest.mark.parametrize("tb,cb", VARIANTS)
def test_ragged_sizes_every_variant(tb, cb):
    rng = np.random.default_rng(tb * 100 + cb)
    sizes = [1, 7, 8, 15, 16, 17, 31, 33, 4097, 8191, 8192, 8193, 16384 + 5, 3 * 8192 + 4095, 100003]
    e_t = -11 if tb == 8 else -17
    s = cb - 1 if cb else 0
    specs, thetas, comps = [], [], []
    for n in sizes:
        th, c = random_tensor(rng, n, tb, cb, full_range=False)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, overlap_k=0, exp_theta=e_t))
        thetas.append(th)
        comps.append(c)
    steps = 6
    sigma = 2.0 ** (e_t - s) * 40 / 0.1
    grads = [[(rng.standard_normal(n) * sigma).astype(np.float32) for n in sizes]
             for _ in range(steps)]
    lrs = [[0.1] * len(sizes)] * steps
    run_both(specs, thetas, comps, grads, lrs, EXP_AMAX)


@pytest.mark.parametrize("tb,cb", VARIANTS)
def test_full_range_inputs_and_heavy_saturation(tb, cb):
    """Inputs include the most negative codes; gradients are large enough to clamp both
    the parameter and the compensation in a good share of the elements."""
    rng = np.random.default_rng(7 + tb + cb)
    n = 50021
    e_t = -9
    s = cb - 1 if cb else 0
    th, c = random_tensor(rng, n, tb, cb, full_range=True)
    specs = [dict(numel=n, theta_bits=tb, comp_bits=cb, overlap_k=0, exp_theta=e_t)]
    grads, lrs = [], []
    for step in range(5):
        scale = 2.0 ** e_t * qmax(tb) * (0.02, 0.5, 3.0, 1e-4, 1e3)[step]
        grads.append([(rng.standard_t(3, n) * scale).astype(np.float32)])
        lrs.append([1.0])
    ost = run_both(specs, [th], [c], grads, lrs, EXP_FIXED)
    assert ost.tensors[0].n_sat_theta > 0
    if cb:
        assert ost.tensors[0].n_sat_comp > 0


# ----------------------------------------------------------------------------- exponent changes

@pytest.mark.parametrize("tb,cb,k", [(8, 8, 0), (16, 8, 0), (16, 16, 0), (8, 16, 0), (8, 0, 0),
                                     (16, 0, 0), (8, 8, 3), (16, 16, 15), (8, 8, 7)])
def test_every_exponent_change(tb, cb, k):
    """Each change of -8..8 binades, forced through kahan_sgd_set_exponents, on one list."""
    rng = np.random.default_rng(1000 + tb + cb + k)
    deltas = list(range(-8, 9))
    n = 20011
    s = cb - 1 - k if cb else 0
    specs, thetas, comps = [], [], []
    for _ in deltas:
        th, c = random_tensor(rng, n, tb, cb, k, full_range=True)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, overlap_k=k, exp_theta=-20))
        thetas.append(th)
        comps.append(c)
    sigma = 2.0 ** (-20 - s) * 50
    grads = [[(rng.standard_normal(n) * sigma).astype(np.float32) for _ in deltas] for _ in range(3)]
    lrs = [[1.0] * len(deltas)] * 3
    exps = [[-20 + d for d in deltas], None, [-20 for _ in deltas]]
    # step 1 follows the max scan after the forced change; step 2 is forced back
    # (the forced value must stay within 8 of the then-current exponent, which it does)
    gpu = LibraryRun(specs, thetas, comps, EXP_AMAX)
    ost = make_oracle_state(specs, thetas, comps, EXP_AMAX)
    try:
        for step in range(3):
            if exps[step] is not None:
                cur = [t.exp_theta for t in ost.tensors]
                want = [max(c - 8, min(c + 8, e)) for c, e in zip(cur, exps[step])]
                gpu.set_exponents(exps[step])
                for t, e in zip(ost.tensors, want):
                    t.exp_theta_next = e
            gpu.step(grads[step], lrs[step])
            oracle_step(ost, [g.copy() for g in grads[step]], lrs[step])
            assert_same_state(gpu, ost, f"step {step}")
        assert gpu.guards_intact()
    finally:
        gpu.close()


def test_exponents_follow_growing_and_shrinking_tensors():
    """Exponent policy end to end: a tensor driven upwards re-grids coarser, one that
    collapses towards zero re-grids finer, all decided on the device."""
    rng = np.random.default_rng(77)
    n = 30000
    specs = [dict(numel=n, theta_bits=8, comp_bits=8, overlap_k=0, exp_theta=-8),
             dict(numel=n, theta_bits=16, comp_bits=16, overlap_k=0, exp_theta=-12),
             dict(numel=n, theta_bits=16, comp_bits=8, overlap_k=0, exp_theta=-12)]
    thetas = [rng.integers(-127, 128, n).astype(np.int8), rng.integers(-3000, 3000, n).astype(np.int16),
              rng.integers(-32767, 32768, n).astype(np.int16)]
    comps = [np.zeros(n, np.int8), np.zeros(n, np.int16), np.zeros(n, np.int8)]
    grads, lrs = [], []
    for step in range(14):
        grads.append([np.full(n, -0.2, np.float32) * np.float32(1.7 ** step),      # grows
                      (rng.standard_normal(n) * 1e-7).astype(np.float32),           # small values
                      (thetas[2].astype(np.float32) * 2.0 ** -12 * 0.45)])          # shrinks
        lrs.append([1.0, 1.0, 1.0])
    ost = run_both(specs, thetas, comps, grads, lrs, EXP_AMAX)
    assert ost.tensors[0].exp_theta > -8
    assert ost.tensors[1].exp_theta < -12


# ----------------------------------------------------------------------------- special values

def test_non_finite_and_extreme_gradients():
    rng = np.random.default_rng(5)
    n = 40000
    for tb, cb in VARIANTS:
        th, c = random_tensor(rng, n, tb, cb, full_range=False)
        g = (rng.standard_normal(n) * 1e-4).astype(np.float32)
        idx = rng.choice(n, 600, replace=False)
        specials = np.array([np.inf, -np.inf, np.nan, 3.4e38, -3.4e38, 1e-45, -1e-45, 1e-38, 0.0,
                             -0.0, 1.17549435e-38, 2.0 ** 30, -2.0 ** 31], np.float32)
        g[idx] = specials[np.arange(600) % specials.size]
        specs = [dict(numel=n, theta_bits=tb, comp_bits=cb, overlap_k=0, exp_theta=-12)]
        ost = run_both(specs, [th], [c], [[g], [g[::-1].copy()]], [[0.05], [0.05]], EXP_AMAX)
        assert ost.tensors[0].n_nonfinite == 2 * int((~np.isfinite(g)).sum())


@pytest.mark.parametrize("lr", [1e-30, 1.1754944e-38, 6e-8, 1.0, 3.0e4, 1e20, 3e38])
def test_learning_rate_extremes(lr):
    rng = np.random.default_rng(8)
    n = 9000
    specs, thetas, comps, grads = [], [], [], []
    for e_t in (-64, -30, 0, 40, 64):
        th, c = random_tensor(rng, n, 8, 16, full_range=False)
        specs.append(dict(numel=n, theta_bits=8, comp_bits=16, overlap_k=0, exp_theta=e_t))
        thetas.append(th)
        comps.append(c)
        target = 2.0 ** (e_t - 15) * 200.0
        grads.append((rng.standard_normal(n) * min(target / lr, 1e37)).astype(np.float32))
    run_both(specs, thetas, comps, [grads, grads], [[lr] * 5, [lr] * 5], EXP_FIXED)


# ----------------------------------------------------------------------------- mixed lists

def test_mixed_formats_in_one_list_and_long_lists():
    """More tensors than fit in the kernel-parameter argument block (so the upload path
    runs), every format variant and several overlaps interleaved."""
    rng = np.random.default_rng(21)
    specs, thetas, comps = [], [], []
    for i in range(300):
        tb, cb = VARIANTS[i % len(VARIANTS)]
        k = 0 if cb == 0 else int(rng.integers(0, cb))
        n = int(rng.integers(1, 30000))
        th, c = random_tensor(rng, n, tb, cb, k, full_range=False)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, overlap_k=k,
                          exp_theta=int(rng.integers(-30, -5))))
        thetas.append(th)
        comps.append(c)
    grads, lrs = [], []
    for step in range(4):
        gs = []
        for sp in specs:
            s = sp["comp_bits"] - 1 - sp["overlap_k"] if sp["comp_bits"] else 0
            gs.append((rng.standard_normal(sp["numel"]) * 2.0 ** (sp["exp_theta"] - s) * 300)
                      .astype(np.float32))
        grads.append(gs)
        lrs.append([float(x) for x in rng.uniform(0.01, 1.0, len(specs)).astype(np.float32)])
    run_both(specs, thetas, comps, grads, lrs, EXP_AMAX)


def test_long_lists_with_8bit_theta_take_the_large_tiles():
    """A list long enough for the 16384-element tiles of 8-bit theta (the library picks the
    tile size per list): every 8-bit format, sizes around the large and the small tile
    boundary, 16-bit tensors (which keep the small tiles) in between, an exponent change and
    saturating steps included."""
    rng = np.random.default_rng(77)
    T = 16384
    sizes8 = [T * 300 + 5, T * 270 + T - 1, T * 260 + 8193, T * 250, T + 1, T - 1, 8192, 8193, 17, 1, 3 * T + 16]
    specs, thetas, comps = [], [], []
    for i, n in enumerate(sizes8):
        tb, cb = [(8, 8), (8, 0), (8, 16)][i % 3]
        th, c = random_tensor(rng, n, tb, cb, full_range=(i % 4 == 0))
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, overlap_k=0, exp_theta=-11))
        thetas.append(th)
        comps.append(c)
    for n, (tb, cb) in [(8192 * 5 + 9, (16, 16)), (100003, (16, 8)), (16384, (16, 0))]:
        th, c = random_tensor(rng, n, tb, cb, full_range=False)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, overlap_k=0, exp_theta=-17))
        thetas.append(th)
        comps.append(c)
    assert sum((sp["numel"] + T - 1) // T for sp in specs if sp["theta_bits"] == 8) >= 1024
    grads, lrs = [], []
    for step in range(4):
        gs = []
        for sp in specs:
            s = sp["comp_bits"] - 1 if sp["comp_bits"] else 0
            sigma = 2.0 ** (sp["exp_theta"] - s) * (4000 if step == 2 else 40) / 0.1
            gs.append((rng.standard_normal(sp["numel"]) * sigma).astype(np.float32))
        grads.append(gs)
        lrs.append([0.1] * len(specs))
    run_both(specs, thetas, comps, grads, lrs, EXP_AMAX)


@pytest.mark.parametrize("extra", [0, 1, 2, 19, 74, 75, 147])
def test_last_round_of_the_tile_table_cut_into_pieces(extra):
    """The tiles of a table's last, incomplete round over the blocks are cut into 2^k pieces
    each (k the largest with at most one piece per block): one leftover tile becomes 16 pieces
    of 512 elements, 19 become 133 of 1024, 75 and more stay whole, none is nothing to cut.
    Two tensors, so that the round spans a tensor border, ragged ends, an exponent change."""
    import torch
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rng = np.random.default_rng(4000 + extra)
    tiles = 2 * sms + extra
    n0 = 8192 * (tiles - max(extra // 2, 1)) - 7          # ends inside a tile
    n1 = 8192 * tiles - (n0 + 8191) // 8192 * 8192 - 3
    specs, thetas, comps = [], [], []
    for n in (n0, n1):
        th, c = random_tensor(rng, n, 16, 8, full_range=False)
        specs.append(dict(numel=n, theta_bits=16, comp_bits=8, overlap_k=0, exp_theta=-14))
        thetas.append(th); comps.append(c)
    grads = [[(rng.standard_normal(n) * 2.0 ** -19 * (1 + 40 * (k == 1))).astype(np.float32) for n in (n0, n1)]
             for k in range(3)]
    run_both(specs, thetas, comps, grads, [[1.0, 0.5]] * 3)


def test_checkpoint_resume_is_bit_identical():
    """N steps in one go == N/2 steps, read the state back, re-init from it, N/2 more."""
    rng = np.random.default_rng(31)
    wl = W.scaled_sweep(400_000, 12)
    specs = specs_of(wl)
    thetas, comps = W.initial_state(wl)
    grads = [W.gradients(wl, s) for s in range(6)]
    grads = [[g * np.float32(30.0) for g in gs] for gs in grads]
    lrs = [[wl.lr] * len(specs)] * 6
    a = LibraryRun(specs, thetas, comps, EXP_AMAX)
    for s in range(6):
        a.step(grads[s], lrs[s])
    ta, ca, sa = a.thetas(), a.comps(), a.stats()
    a.close()
    b = LibraryRun(specs, thetas, comps, EXP_AMAX)
    for s in range(3):
        b.step(grads[s], lrs[s])
    tb_, cb_, sb = b.thetas(), b.comps(), b.stats()
    b.close()
    specs2 = [dict(sp, exp_theta=sb["exp_theta_cur"][i], exp_theta_next=sb["exp_theta_next"][i])
              for i, sp in enumerate(specs)]
    c = LibraryRun(specs2, tb_, cb_, EXP_AMAX)
    for s in range(3, 6):
        c.step(grads[s], lrs[s])
    tc, cc, sc = c.thetas(), c.comps(), c.stats()
    c.close()
    for i in range(len(specs)):
        assert np.array_equal(ta[i], tc[i]) and np.array_equal(ca[i], cc[i])
    for key in ("amax_theta", "amax_comp", "exp_theta_cur", "exp_theta_next"):
        assert sa[key] == sc[key]


def test_step_on_a_side_stream_and_back_to_back_steps():
    """Many steps enqueued without any host synchronisation, on a non-default stream."""
    import torch
    rng = np.random.default_rng(41)
    n = 200_003
    th, c = random_tensor(rng, n, 16, 8, full_range=False)
    specs = [dict(numel=n, theta_bits=16, comp_bits=8, overlap_k=0, exp_theta=-17)]
    g = (rng.standard_normal(n) * 1e-4).astype(np.float32)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        gpu = LibraryRun(specs, [th], [c], EXP_AMAX, stream=side)
        gpu.grad_arena.upload(0, g)
        side.synchronize()
        for _ in range(25):
            gpu.B.kahan_sgd_step(gpu.handle, gpu.grad_ptrs, [0.1])
        side.synchronize()
    ost = make_oracle_state(specs, [th], [c], EXP_AMAX)
    for _ in range(25):
        oracle_step(ost, [g], [0.1])
    assert_same_state(gpu, ost, "after 25 steps")
    gpu.close()


def test_step_host_matches_device_step():
    """The host-buffer entry point gives the same bits as uploading by hand."""
    import torch
    rng = np.random.default_rng(51)
    wl = W.scaled_sweep(300_000, 9)
    specs = specs_of(wl)
    thetas, comps = W.initial_state(wl)
    grads = [g * np.float32(25.0) for g in W.gradients(wl, 0)]
    lrs = [wl.lr] * len(specs)
    gpu = LibraryRun(specs, [np.zeros_like(t) for t in thetas], [np.zeros_like(c) for c in comps],
                 EXP_AMAX)
    ost = make_oracle_state(specs, thetas, comps, EXP_AMAX)
    th_h = [t.copy() for t in thetas]
    c_h = [c.copy() for c in comps]
    need = sum((sp["numel"] + 3) // 4 * 16 for sp in specs)
    staging = torch.empty(need, dtype=torch.uint8, device="cuda")
    for _ in range(2):
        gpu.B.kahan_sgd_step_host(gpu.handle, [t.ctypes.data for t in th_h],
                                  [c.ctypes.data for c in c_h], [g.ctypes.data for g in grads],
                                  lrs, staging.data_ptr(), need)
        oracle_step(ost, grads, lrs)
        for i, t in enumerate(ost.tensors):
            assert np.array_equal(th_h[i], t.theta) and np.array_equal(c_h[i], t.comp)
    assert_same_state(gpu, ost, "host step")
    gpu.close()


def test_tensor_with_more_than_2_31_elements_in_full():
    """One int8/int8 tensor of 2^31 + 12345 elements (element and byte offsets beyond 32 bits),
    fixed exponent so that the oracle can take it slice by slice: every mantissa of theta and
    c is compared, and the two scans and the three counters of the whole tensor must equal the
    maximum / the sum over the oracle's slices.  A few planted gradients (NaN, both
    infinities, values far beyond theta's range) sit on both sides of the 2^31-element and
    2^32-byte marks; a guard band behind each array must stay untouched."""
    import torch
    from oracle import oracle_max_threads, oracle_step_tensor
    from paper_1810_05486_b200 import binding as B
    free, _ = torch.cuda.mem_get_info()
    if free < 20 << 30:
        pytest.skip("needs 20 GB of free device memory")
    n = 2 ** 31 + 12345
    guard = 4096
    gen = torch.Generator(device="cuda").manual_seed(1234)
    theta = torch.empty(n + guard, dtype=torch.int8, device="cuda")
    comp = torch.empty(n + guard, dtype=torch.int8, device="cuda")
    grad = torch.empty(n + guard, dtype=torch.float32, device="cuda")
    piece = 1 << 28
    for lo in range(0, n, piece):                     # inputs come from torch's generator, in pieces
        hi = min(n, lo + piece)
        theta[lo:hi] = torch.randint(-127, 128, (hi - lo,), generator=gen, device="cuda", dtype=torch.int8)
        comp[lo:hi] = torch.randint(-64, 65, (hi - lo,), generator=gen, device="cuda", dtype=torch.int8)
        grad[lo:hi] = torch.randn(hi - lo, generator=gen, device="cuda") * (2.0 ** -18 * 40)
    planted = {123: float("nan"), 2 ** 30 - 1: float("inf"), 2 ** 30 + 16: -float("inf"),
               2 ** 31 - 3: 1.0e3, 2 ** 31 + 5: float("inf"), 2 ** 31 + 8200: -2.0e-2, n - 2: float("nan"),
               n - 9000: 7.0e-3}
    for idx, val in planted.items():
        grad[idx] = val
    theta[n:] = 0x5A
    comp[n:] = 0x5A
    grad[n:] = 7.0
    # host copies of the inputs, taken before the step
    t_host = np.empty(n, np.int8)
    c_host = np.empty(n, np.int8)
    g_host = np.empty(n, np.float32)
    for lo in range(0, n, piece):
        hi = min(n, lo + piece)
        t_host[lo:hi] = theta[lo:hi].cpu().numpy()
        c_host[lo:hi] = comp[lo:hi].cpu().numpy()
        g_host[lo:hi] = grad[lo:hi].cpu().numpy()
    descs = B.make_descs([dict(theta=theta.data_ptr(), comp=comp.data_ptr(), numel=n, theta_bits=8,
                               comp_bits=8, exp_theta=-11)])
    nb = B.kahan_sgd_workspace_bytes(descs)
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    h = B.kahan_sgd_init(descs, B.KSGD_EXP_FIXED, ws.data_ptr(), nb, torch.cuda.current_stream().cuda_stream)
    B.kahan_sgd_step(h, [grad.data_ptr()], [1.0])
    st = B.kahan_sgd_amax(h, 1)
    B.kahan_sgd_destroy(h)
    want = dict(amax_theta=0, amax_comp=0, n_sat_theta=0, n_sat_comp=0, n_nonfinite=0)
    threads = oracle_max_threads()
    for lo in range(0, n, piece):
        hi = min(n, lo + piece)
        res = oracle_step_tensor(t_host[lo:hi], c_host[lo:hi], g_host[lo:hi], 8, 8, 0, -11, -11, 1.0, threads)
        assert np.array_equal(theta[lo:hi].cpu().numpy(), t_host[lo:hi]), (lo, hi)
        assert np.array_equal(comp[lo:hi].cpu().numpy(), c_host[lo:hi]), (lo, hi)
        for key in ("amax_theta", "amax_comp"):
            want[key] = max(want[key], res[key])
        for key in ("n_sat_theta", "n_sat_comp", "n_nonfinite"):
            want[key] += res[key]
    assert want["n_nonfinite"] == 5 and want["n_sat_theta"] >= 4
    for key, w in want.items():
        assert st[key][0] == w, (key, st[key][0], w)
    assert st["exp_theta_cur"][0] == -11 and st["exp_theta_next"][0] == -11
    assert bool((theta[n:] == 0x5A).all()) and bool((comp[n:] == 0x5A).all()) and bool((grad[n:] == 7.0).all())


def test_device_error_word_reaches_the_caller():
    """A kernel whose bounded wait runs out sets a sticky word in the workspace and
    kahan_sgd_amax then returns KSGD_ERR_DEVICE.  No wait is made to run out here: the host
    writes the word itself, between two healthy steps, and the read-out must report it
    (and keep reporting it) while the statistics still come back."""
    import torch
    from paper_1810_05486_b200 import binding as B
    wl = W.scaled_sweep(200_000, 5)
    specs = specs_of(wl)
    thetas, comps = W.initial_state(wl)
    gpu = LibraryRun(specs, thetas, comps, EXP_AMAX)
    lrs = [wl.lr] * len(specs)
    try:
        gpu.step(W.gradients(wl, 0), lrs)
        gpu.stats()                                           # healthy: no exception
        off = B.kahan_sgd_workspace_error_offset(gpu.descs)
        word = gpu.workspace[off:off + 4]
        assert bool((word == 0).all())
        torch.cuda.synchronize()
        word.copy_(torch.tensor([2, 0, 0, 0], dtype=torch.uint8))     # the code of a producer that gave up
        torch.cuda.synchronize()
        for _ in range(2):
            with pytest.raises(B.KahanSgdError) as ei:
                gpu.stats()
            assert ei.value.code == B.KSGD_ERR_DEVICE
        gpu.step(W.gradients(wl, 1), lrs)                     # the word is sticky: later steps do not clear it
        with pytest.raises(B.KahanSgdError) as ei:
            gpu.stats()
        assert ei.value.code == B.KSGD_ERR_DEVICE
    finally:
        gpu.close()


def test_steps_captured_in_a_cuda_graph_and_replayed():
    """kahan_sgd_step only enqueues work on the handle's stream, so a sequence of steps can
    be recorded into a CUDA graph and replayed: 4 steps per graph, 3 replays, against 12
    oracle steps (the captured gradient buffers are refilled between replays)."""
    import torch
    rng = np.random.default_rng(61)
    wl = W.workload("c2_resnet20")
    specs = specs_of(wl)
    thetas, comps = W.initial_state(wl)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        gpu = LibraryRun(specs, thetas, comps, EXP_AMAX, stream=side)
        lrs = [wl.lr] * len(specs)
        grads = [W.gradients(wl, s) for s in range(4)]
        # four resident gradient sets, one per captured step
        sets = []
        for gs in grads:
            bufs = [torch.from_numpy(g).cuda() for g in gs]
            sets.append(bufs)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for bufs in sets:
                gpu.B.kahan_sgd_step(gpu.handle, [b.data_ptr() for b in bufs], lrs)
        ost = make_oracle_state(specs, thetas, comps, EXP_AMAX)
        for replay in range(3):
            for k, bufs in enumerate(sets):          # new gradients into the captured buffers
                for b, g in zip(bufs, W.gradients(wl, 4 * replay + k)):
                    b.copy_(torch.from_numpy(g))
            torch.cuda.synchronize()
            graph.replay()
            torch.cuda.synchronize()
            for k in range(4):
                oracle_step(ost, W.gradients(wl, 4 * replay + k), lrs)
            assert_same_state(gpu, ost, f"replay {replay}")
        gpu.close()
