"""Randomised differential test of the CUDA library against the CPU oracle.

Every case draws, from one seed, a ragged list of tensors (formats, overlaps, sizes around
the tile borders, exponents), and then a sequence of steps in which the kind of gradient
(binary32, INT8, INT16), its magnitude (from far below the compensation's unit to far above
theta's range, so that exponents move both ways and both clamps fire), the learning rates
and an occasional forced exponent all vary.  The whole state is compared bit for bit after
every step (Algorithm 1 is defined per element, so every element is in scope)."""
import numpy as np
import pytest

from harness import LibraryRun, assert_same_state, make_oracle_state, storage_dtype
from oracle import (EXP_AMAX, EXP_FIXED, oracle_adam_step, oracle_dequantize, oracle_dequantize_gradient,
                    oracle_fit_exponent, oracle_max_threads, oracle_momentum_step, oracle_quantize, oracle_step,
                    oracle_step_qgrad, oracle_strict_step)

pytestmark = pytest.mark.gpu

FORMATS = [(8, 0), (8, 8), (8, 16), (16, 0), (16, 8), (16, 16)]
BORDER_SIZES = [1, 2, 15, 16, 17, 31, 33, 255, 4095, 4096, 8191, 8192, 8193, 16383, 16384, 16385, 24577,
                32767, 32768, 32769, 65537]
SPECIALS = np.array([np.inf, -np.inf, np.nan, 3.0e38, -3.0e38, 1.0e-45, -0.0], np.float32)


def draw_size(rng):
    kind = rng.integers(0, 3)
    if kind == 0:
        return int(BORDER_SIZES[rng.integers(0, len(BORDER_SIZES))])
    if kind == 1:
        return int(rng.integers(1, 3000))
    return int(rng.integers(3000, 150000))


def draw_list(rng, strict):
    n_tensors = int(rng.integers(1, 14))
    if rng.random() < 0.15:
        n_tensors = int(rng.integers(257, 300))      # beyond the inline argument block
    specs, thetas, comps = [], [], []
    for _ in range(n_tensors):
        tb, cb = FORMATS[rng.integers(0, len(FORMATS))]
        if strict and cb == 0:
            cb = 8 if rng.random() < 0.5 else 16
        numel = draw_size(rng) if n_tensors < 100 else int(rng.integers(1, 2000))
        k = int(rng.integers(0, cb)) if (cb and not strict and rng.random() < 0.3) else 0
        e = int(rng.integers(-30, 10))
        full = rng.random() < 0.3
        lim_t = 2 ** (tb - 1) if full else 2 ** (tb - 2)
        theta = rng.integers(-lim_t, lim_t, numel).astype(storage_dtype(tb))
        comp = None
        if cb:
            lim_c = 2 ** (cb - 1) if full else 2 ** (cb - 2)
            comp = rng.integers(-lim_c, lim_c, numel).astype(storage_dtype(cb))
        spec = dict(numel=numel, theta_bits=tb, comp_bits=cb, overlap_k=k, exp_theta=e)
        if strict:
            # anywhere in the window the library accepts: 8 above to 36 below theta's exponent
            spec["exp_comp"] = max(-64, e - int(rng.integers(-8, 37)))
        specs.append(spec)
        thetas.append(theta)
        comps.append(comp)
    return specs, thetas, comps


def comp_unit_exponent(t, strict):
    """Exponent of one compensation LSB of oracle tensor t as the coming step writes it."""
    if strict:
        return t.exp_comp_next
    s = t.comp_bits - 1 - t.overlap_k if t.comp_bits else 0
    return t.exp_theta_next - s


def draw_float_grads(rng, ost, strict, lrs):
    grads = []
    for t, lr in zip(ost.tensors, lrs):
        n = t.theta.size
        # increments of 2^-6 compensation units up to a few units of theta (the exact
        # steady path), in a third of the draws up to far beyond theta's range (clamps,
        # coarser grids)
        span = (t.comp_bits or 1) + 2
        if rng.random() < 0.33:
            span += t.theta_bits + 1
        mag = 2.0 ** (comp_unit_exponent(t, strict) + float(rng.uniform(-6, span))) / lr
        g = (rng.standard_normal(n) * mag).astype(np.float32)
        if rng.random() < 0.25:
            idx = rng.choice(n, min(n, 5), replace=False)
            g[idx] = SPECIALS[rng.integers(0, len(SPECIALS), idx.size)]
        if rng.random() < 0.1:
            g[:] = 0.0
        grads.append(g)
    return grads


def draw_fixed_grads(rng, ost, strict, lrs, gb):
    grads, exps = [], []
    for t, lr in zip(ost.tensors, lrs):
        n = t.theta.size
        g = rng.integers(-2 ** (gb - 1), 2 ** (gb - 1), n).astype(storage_dtype(gb))
        if rng.random() < 0.3:                      # a grid fixed by one outlier, the rest small
            g = (g // 2 ** (gb - 3)).astype(storage_dtype(gb))
            g[rng.integers(0, n)] = 2 ** (gb - 1) - 1
        # one gradient unit times lr worth 2^-5 .. 2^10 compensation units
        eg = comp_unit_exponent(t, strict) + int(rng.integers(-5, 11)) - int(np.round(np.log2(lr)))
        grads.append(g)
        exps.append(int(np.clip(eg, -64, 64)))
    return grads, exps


def draw_lrs(rng, n):
    if rng.random() < 0.5:
        return [float(np.float32(2.0 ** rng.integers(-6, 3)))] * n
    return [float(np.float32(rng.uniform(1e-3, 2.0))) for _ in range(n)]


def run_case(seed, strict, steps):
    rng = np.random.default_rng([seed, int(strict)])
    specs, thetas, comps = draw_list(rng, strict)
    mode = EXP_FIXED if rng.random() < 0.15 else EXP_AMAX
    gpu = LibraryRun(specs, thetas, comps, mode, strict=strict)
    ost = make_oracle_state(specs, thetas, comps, mode, oracle_max_threads())
    n = len(specs)
    kinds = []
    try:
        for step in range(steps):
            lrs = draw_lrs(rng, n)
            if not strict and rng.random() < 0.2:
                want = [int(np.clip(t.exp_theta + rng.integers(-10, 11), -64, 64)) for t in ost.tensors]
                gpu.set_exponents(want)
                for t, e in zip(ost.tensors, want):       # the device limits the change to 8 binades
                    t.exp_theta_next = max(t.exp_theta - 8, min(t.exp_theta + 8, e))
            if step > 0 and rng.random() < 0.15:
                # checkpoint and resume: a fresh handle (and a fresh oracle state) from the
                # mantissas and exponents as they stand, the next exponents as first-step targets
                kinds.append("resume")
                gpu.close()
                for sp, t in zip(specs, ost.tensors):
                    sp["exp_theta"], sp["exp_theta_next"] = t.exp_theta, t.exp_theta_next
                    if strict:
                        sp["exp_comp"], sp["exp_comp_next"] = t.exp_comp, t.exp_comp_next
                thetas = [t.theta.copy() for t in ost.tensors]
                comps = [None if t.comp is None else t.comp.copy() for t in ost.tensors]
                gpu = LibraryRun(specs, thetas, comps, mode, strict=strict)
                ost = make_oracle_state(specs, thetas, comps, mode, oracle_max_threads())
            kind = (32, 32, 8, 16, "host")[rng.integers(0, 4 if strict else 5)]
            kinds.append(kind)
            if kind == "host":
                # the host-buffer entry point: state and gradients travel from host arrays (the
                # oracle's copies, equal to the device's by the last comparison) and back
                import torch
                grads = draw_float_grads(rng, ost, strict, lrs)
                th_h = [t.theta.copy() for t in ost.tensors]
                c_h = [None if t.comp is None else t.comp.copy() for t in ost.tensors]
                need = sum((sp["numel"] + 3) // 4 * 16 for sp in specs)
                staging = torch.empty(need, dtype=torch.uint8, device="cuda")
                gpu.B.kahan_sgd_step_host(gpu.handle, [t.ctypes.data for t in th_h],
                                          [None if c is None else c.ctypes.data for c in c_h],
                                          [g.ctypes.data for g in grads], lrs, staging.data_ptr(), need)
                oracle_step(ost, [g.copy() for g in grads], lrs)
                for i, t in enumerate(ost.tensors):
                    assert np.array_equal(th_h[i], t.theta), f"seed {seed} step {step}: host theta of tensor {i}"
                    assert t.comp is None or np.array_equal(c_h[i], t.comp), \
                        f"seed {seed} step {step}: host comp of tensor {i}"
            elif kind == 32:
                grads = draw_float_grads(rng, ost, strict, lrs)
                gpu.step(grads, lrs)
                (oracle_strict_step if strict else oracle_step)(ost, [g.copy() for g in grads], lrs)
            else:
                gq, eg = draw_fixed_grads(rng, ost, strict, lrs, kind)
                gpu.step_qgrad(gq, eg, lrs, exponents_on_device=bool(rng.random() < 0.4))
                if strict:
                    oracle_strict_step(ost, [oracle_dequantize_gradient(q, e) for q, e in zip(gq, eg)], lrs)
                else:
                    oracle_step_qgrad(ost, gq, eg, lrs)
            assert_same_state(gpu, ost, f"seed {seed} strict {strict} step {step} kinds {kinds}")
        assert gpu.guards_intact()
    finally:
        gpu.close()


@pytest.mark.parametrize("seed", range(60))
def test_random_lists_and_step_sequences_plain_handle(seed):
    run_case(seed, strict=False, steps=7)


@pytest.mark.parametrize("seed", range(30))
def test_random_lists_and_step_sequences_strict_handle(seed):
    run_case(seed, strict=True, steps=6)


# ------------------------------------------------------------------ momentum and ADAM

def draw_optimizer_list(rng, with_velocity_bits):
    """A short ragged list for the optimizers (comp_bits != 0), with exponents for the extra
    state tensors placed around the size of the increments that will come."""
    n_tensors = int(rng.integers(1, 9))
    if rng.random() < 0.1:
        n_tensors = int(rng.integers(257, 280))      # beyond the inline argument block
    specs, thetas, comps = [], [], []
    for _ in range(n_tensors):
        tb = 8 if rng.random() < 0.5 else 16
        cb = 8 if rng.random() < 0.5 else 16
        numel = draw_size(rng) if n_tensors < 100 else int(rng.integers(1, 2000))
        k = int(rng.integers(0, cb)) if rng.random() < 0.25 else 0
        e = int(rng.integers(-24, 4))
        full = rng.random() < 0.25
        lim_t = 2 ** (tb - 1) if full else 2 ** (tb - 2)
        lim_c = 2 ** (cb - 1) if full else 2 ** (cb - 2)
        spec = dict(numel=numel, theta_bits=tb, comp_bits=cb, overlap_k=k, exp_theta=e)
        if with_velocity_bits:
            spec["mom_bits"] = 8 if rng.random() < 0.5 else 16
        specs.append(spec)
        thetas.append(rng.integers(-lim_t, lim_t, numel).astype(storage_dtype(tb)))
        comps.append(rng.integers(-lim_c, lim_c, numel).astype(storage_dtype(cb)))
    return specs, thetas, comps


def special_values(rng, g):
    if rng.random() < 0.2:
        idx = rng.choice(g.size, min(g.size, 5), replace=False)
        g[idx] = SPECIALS[rng.integers(0, len(SPECIALS), idx.size)]
    return g


def run_momentum_case(seed, steps):
    from test_gpu_momentum import MomentumRun, oracle_state
    rng = np.random.default_rng([seed, 2])
    specs, thetas, comps = draw_optimizer_list(rng, True)
    moms = []
    for s in specs:
        vb = s["mom_bits"]
        c_unit = s["exp_theta"] - (s["comp_bits"] - 1 - s["overlap_k"])
        # the velocity's unit from 20 binades below the compensation's to 12 above
        s["exp_mom"] = int(np.clip(c_unit + rng.integers(-20, 13), -64, 64))
        lim = 2 ** (vb - 1) if rng.random() < 0.25 else 2 ** (vb - 3)
        moms.append(rng.integers(-lim, lim, s["numel"]).astype(storage_dtype(vb)))
    mode = EXP_FIXED if rng.random() < 0.15 else EXP_AMAX
    gpu = MomentumRun(specs, thetas, comps, moms, mode)
    ost = oracle_state(specs, thetas, comps, moms, mode)
    try:
        for step in range(steps):
            if step > 0 and rng.random() < 0.15:      # checkpoint and resume from the state as it stands
                gpu.close()
                for sp, t in zip(specs, ost.tensors):
                    sp["exp_theta"], sp["exp_theta_next"] = t.exp_theta, t.exp_theta_next
                    sp["exp_mom"], sp["exp_mom_next"] = t.exp_mom, t.exp_mom_next
                thetas, comps = [t.theta.copy() for t in ost.tensors], [t.comp.copy() for t in ost.tensors]
                moms = [t.mom.copy() for t in ost.tensors]
                gpu = MomentumRun(specs, thetas, comps, moms, mode)
                ost = oracle_state(specs, thetas, comps, moms, mode)
            lrs = draw_lrs(rng, len(specs))
            mus = [float(np.float32(rng.choice([0.0, 0.5, 0.9, 0.99, 1.0])))] * len(specs)
            grads = []
            for t, lr in zip(ost.tensors, lrs):
                # lr * g worth 2^-4 .. 2^(bits + 2) units of the velocity grid the step writes
                mag = 2.0 ** (t.exp_mom_next + float(rng.uniform(-4, t.mom_bits + 2))) / lr
                grads.append(special_values(rng, (rng.standard_normal(t.theta.size) * mag).astype(np.float32)))
            gpu.step(grads, lrs, mus)
            oracle_momentum_step(ost, [g.copy() for g in grads], lrs, mus)
            gpu.check(ost, f"momentum seed {seed} step {step}")
        assert gpu.guards_intact()
    finally:
        gpu.close()


def run_adam_case(seed, steps):
    from test_gpu_adam import AdamRun, oracle_state
    rng = np.random.default_rng([seed, 3])
    specs, thetas, comps = draw_optimizer_list(rng, False)
    b1, b2, eps = [(0.9, 0.999, 1e-8), (0.5, 0.9, 1e-3), (0.9, 0.99, 0.0), (0.0, 0.999, 1e-6)][rng.integers(0, 4)]
    m1s, m2s, sigmas = [], [], []
    for s in specs:
        sigma = 2.0 ** float(rng.uniform(-20, 4))
        sigmas.append(sigma)
        # grids that hold a first moment of about 4 sigma and a second of about 16 sigma^2,
        # moved off by a few binades either way
        s["exp_m"] = int(np.clip(np.ceil(np.log2(4 * sigma / 32767)) + rng.integers(-3, 4), -64, 64))
        s["exp_v"] = int(np.clip(np.ceil(np.log2(16 * sigma ** 2 / 32767)) + rng.integers(-3, 4), -64, 64))
        zero = rng.random() < 0.3
        m1s.append(np.zeros(s["numel"], np.int16) if zero else rng.integers(-9000, 9000, s["numel"]).astype(np.int16))
        m2s.append(np.zeros(s["numel"], np.int16) if zero else rng.integers(0, 9000, s["numel"]).astype(np.int16))
    mode = EXP_FIXED if rng.random() < 0.15 else EXP_AMAX
    gpu = AdamRun(specs, thetas, comps, m1s, m2s, mode)
    ost = oracle_state(specs, thetas, comps, m1s, m2s, mode)
    try:
        for step in range(steps):
            if step > 0 and rng.random() < 0.15:      # checkpoint and resume from the state as it stands
                gpu.close()
                for sp, t in zip(specs, ost.tensors):
                    sp["exp_theta"], sp["exp_theta_next"] = t.exp_theta, t.exp_theta_next
                    sp["exp_m"], sp["exp_m_next"] = t.exp_mom, t.exp_mom_next
                    sp["exp_v"], sp["exp_v_next"] = t.exp_mom2, t.exp_mom2_next
                thetas, comps = [t.theta.copy() for t in ost.tensors], [t.comp.copy() for t in ost.tensors]
                m1s, m2s = [t.mom.copy() for t in ost.tensors], [t.mom2.copy() for t in ost.tensors]
                gpu = AdamRun(specs, thetas, comps, m1s, m2s, mode)
                ost = oracle_state(specs, thetas, comps, m1s, m2s, mode)
            lrs = []
            for t in ost.tensors:
                # a unit step (m / sqrt(v) ~ 1) worth 2^-3 .. 2^(bits of c + 4) compensation units
                c_unit = t.exp_theta_next - (t.comp_bits - 1 - t.overlap_k)
                lrs.append(float(np.float32(2.0 ** (c_unit + float(rng.uniform(-3, t.comp_bits + 4))))))
            grads = [special_values(rng, (rng.standard_normal(t.theta.size) * sg * 2.0 ** float(rng.uniform(-2, 2)))
                                    .astype(np.float32)) for t, sg in zip(ost.tensors, sigmas)]
            gpu.step(grads, lrs, b1, b2, eps)
            oracle_adam_step(ost, [g.copy() for g in grads], lrs, b1, b2, eps)
            gpu.check(ost, f"adam seed {seed} step {step}")
        assert gpu.guards_intact()
    finally:
        gpu.close()


@pytest.mark.parametrize("seed", range(30))
def test_random_lists_and_gradients_momentum(seed):
    run_momentum_case(seed, steps=6)


@pytest.mark.parametrize("seed", range(30))
def test_random_lists_and_gradients_adam(seed):
    run_adam_case(seed, steps=6)


# ------------------------------------------------------------------ fp32 <-> fixed point

def run_convert_case(seed):
    """Import and export of a random array at a random element offset (aligned and unaligned
    paths), magnitudes over the whole exponent range, specials sprinkled in, against the oracle;
    guard values before and after every output."""
    import torch
    from paper_1810_05486_b200 import binding as B
    rng = np.random.default_rng([seed, 4])
    st = torch.cuda.current_stream().cuda_stream
    tb = 8 if rng.random() < 0.5 else 16
    cb = int(rng.choice([0, 8, 16]))
    k = int(rng.integers(0, cb)) if (cb and rng.random() < 0.3) else 0
    n = draw_size(rng)
    off = int(rng.choice([0, 0, 1, 2, 3, 4, 8]))
    x = (rng.standard_t(3, n + off) * 2.0 ** float(rng.uniform(-70, 40))).astype(np.float32)
    if rng.random() < 0.4:
        idx = rng.choice(n + off, min(n + off, 6), replace=False)
        x[idx] = SPECIALS[rng.integers(0, len(SPECIALS), idx.size)]
    if rng.random() < 0.05:
        x[:] = 0.0
    src = np.ascontiguousarray(x[off:])
    dx = torch.from_numpy(x).cuda()
    tdt, cdt = (torch.int8 if tb == 8 else torch.int16), (torch.int8 if cb <= 8 else torch.int16)
    th = torch.full((n + off + 32,), 0x5A, dtype=tdt, device="cuda")
    c = torch.full((n + off + 32,), 0x5A, dtype=cdt, device="cuda")
    scratch = torch.zeros(4, dtype=torch.int32, device="cuda")
    e_req = B.KSGD_EXP_AUTO if rng.random() < 0.6 else int(rng.integers(-64, 65))
    cptr = (c.data_ptr() + off * (max(cb, 8) // 8)) if cb else None
    e = B.kahan_sgd_import(dx.data_ptr() + 4 * off, th.data_ptr() + off * (tb // 8), cptr, n, tb, cb, k, e_req,
                           scratch.data_ptr(), st)
    assert e == (oracle_fit_exponent(src, tb) if e_req == B.KSGD_EXP_AUTO else e_req), f"convert seed {seed}"
    wt, wc = oracle_quantize(src, tb, cb, k, e)
    assert np.array_equal(th[off:off + n].cpu().numpy(), wt), f"convert seed {seed}: theta"
    assert bool((th[:off] == 0x5A).all()) and bool((th[off + n:] == 0x5A).all())
    if cb:
        assert np.array_equal(c[off:off + n].cpu().numpy(), wc), f"convert seed {seed}: comp"
        assert bool((c[:off] == 0x5A).all()) and bool((c[off + n:] == 0x5A).all())
    out = torch.full((n + off + 8,), 7.0, dtype=torch.float32, device="cuda")
    B.kahan_sgd_export(th.data_ptr() + off * (tb // 8), cptr, out.data_ptr() + 4 * off, n, tb, cb, k, e, st)
    want = oracle_dequantize(wt, wc, tb, cb, k, e)
    assert np.array_equal(out[off:off + n].cpu().numpy().view(np.uint32), want.view(np.uint32)), \
        f"convert seed {seed}: export"
    assert bool((out[:off] == 7.0).all()) and bool((out[off + n:] == 7.0).all())


@pytest.mark.parametrize("seed", range(60))
def test_random_arrays_through_import_and_export(seed):
    run_convert_case(seed)
