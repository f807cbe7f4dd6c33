"""fp32 <-> dynamic fixed-point on the device against the oracle, bit for bit."""
import numpy as np
import pytest

from oracle import oracle_dequantize, oracle_fit_exponent, oracle_quantize

pytestmark = pytest.mark.gpu

FORMATS = [(8, 0, 0), (16, 0, 0), (8, 8, 0), (16, 8, 0), (8, 16, 0), (16, 16, 0), (8, 8, 5), (16, 16, 15)]


def storage(bits):
    return np.int8 if bits <= 8 else np.int16


@pytest.mark.parametrize("tb,cb,k", FORMATS)
def test_import_then_export_match_the_oracle(tb, cb, k):
    import torch
    from paper_1810_05486_b200 import binding as B
    rng = np.random.default_rng(tb * 100 + cb + k)
    for n, scale in ((1, 0.3), (1000003, 0.05), (65537, 3e-9), (4099, 2e7)):
        x = (rng.standard_t(3, n) * scale).astype(np.float32)
        if n > 100:
            x[rng.choice(n, 40, replace=False)] = np.array([np.nan, np.inf, -np.inf, 0.0, -0.0, 3e38, -3e38, 1e-45],
                                                           np.float32)[np.arange(40) % 8]
        dx = torch.from_numpy(x).cuda()
        th = torch.full((n + 64,), 0x5A, dtype=torch.int8 if tb == 8 else torch.int16, device="cuda")
        c = torch.full((n + 64,), 0x5A, dtype=torch.int8 if cb <= 8 else torch.int16, device="cuda")
        scratch = torch.zeros(4, dtype=torch.int32, device="cuda")
        st = torch.cuda.current_stream().cuda_stream
        for e_req in (B.KSGD_EXP_AUTO, -9):
            e = B.kahan_sgd_import(dx.data_ptr(), th.data_ptr(), c.data_ptr() if cb else None, n, tb, cb, k,
                                   e_req, scratch.data_ptr(), st)
            want_e = oracle_fit_exponent(x, tb) if e_req == B.KSGD_EXP_AUTO else e_req
            assert e == want_e
            wt, wc = oracle_quantize(x, tb, cb, k, e)
            assert np.array_equal(th[:n].cpu().numpy(), wt)
            if cb:
                assert np.array_equal(c[:n].cpu().numpy(), wc)
            assert bool((th[n:] == 0x5A).all()) and bool((c[n:] == 0x5A).all())     # nothing past the end
            out = torch.full((n + 16,), 7.0, dtype=torch.float32, device="cuda")
            B.kahan_sgd_export(th.data_ptr(), c.data_ptr() if cb else None, out.data_ptr(), n, tb, cb, k, e, st)
            got = out[:n].cpu().numpy()
            want = oracle_dequantize(wt, wc, tb, cb, k, e)
            assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
            assert bool((out[n:] == 7.0).all())


def test_imported_weights_can_be_stepped():
    """fp32 weights -> theta + c -> one lazy-update step -> fp32: the round trip stays within
    the resolution of the compensation grid of the exact update."""
    import torch
    from paper_1810_05486_b200 import binding as B
    rng = np.random.default_rng(5)
    n = 300000
    w = (rng.standard_normal(n) * 0.05).astype(np.float32)
    g = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    dw, dg = torch.from_numpy(w).cuda(), torch.from_numpy(g).cuda()
    th = torch.empty(n, dtype=torch.int8, device="cuda")
    c = torch.empty(n, dtype=torch.int16, device="cuda")
    scratch = torch.zeros(4, dtype=torch.int32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    e = B.kahan_sgd_import(dw.data_ptr(), th.data_ptr(), c.data_ptr(), n, 8, 16, 0, B.KSGD_EXP_AUTO,
                           scratch.data_ptr(), st) + 1          # one binade of head room
    B.kahan_sgd_import(dw.data_ptr(), th.data_ptr(), c.data_ptr(), n, 8, 16, 0, e, None, st)
    descs = B.make_descs([dict(theta=th.data_ptr(), comp=c.data_ptr(), numel=n, theta_bits=8, comp_bits=16,
                               exp_theta=e)])
    nb = B.kahan_sgd_workspace_bytes(descs)
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    h = B.kahan_sgd_init(descs, B.KSGD_EXP_FIXED, ws.data_ptr(), nb, st)
    B.kahan_sgd_step(h, [dg.data_ptr()], [0.1])
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    B.kahan_sgd_export(th.data_ptr(), c.data_ptr(), out.data_ptr(), n, 8, 16, 0, e, st)
    B.kahan_sgd_destroy(h)
    exact = w.astype(np.float64) - 0.1 * g.astype(np.float64)
    lsb_c = 2.0 ** (e - 15)
    assert np.abs(out.cpu().numpy().astype(np.float64) - exact).max() <= 1.01 * lsb_c + 1e-9


def test_import_on_the_device_feeds_the_fixed_point_gradient_step_without_the_host():
    """Gradients quantized on the device (max scan -> exponent in device memory -> int8
    mantissas, nothing copied to the host) and consumed by kahan_sgd_step_qgrad_dev, against
    the oracle: fit exponent, quantize, then the step on the fixed-point gradients."""
    import torch
    from harness import LibraryRun, assert_same_state, make_oracle_state, specs_of
    from oracle import EXP_AMAX, oracle_step_qgrad
    from paper_1810_05486_b200 import binding as B
    from paper_1810_05486_b200 import workloads as W
    wl = W.scaled_sweep(600_000, 7)
    specs = specs_of(wl)
    thetas, comps = W.initial_state(wl)
    gpu = LibraryRun(specs, thetas, comps, EXP_AMAX)
    ost = make_oracle_state(specs, thetas, comps, EXP_AMAX)
    n = len(specs)
    lrs = [wl.lr] * n
    st = torch.cuda.current_stream().cuda_stream
    exps_dev = torch.full((n,), 99, dtype=torch.int32, device="cuda")
    scratch = torch.zeros(2, dtype=torch.int32, device="cuda")
    try:
        for step, bits in enumerate((8, 16, 8)):
            grads = [g * np.float32(30.0) for g in W.gradients(wl, step)]
            grads[1][7] = np.float32(np.nan)
            grads[2][11] = np.float32(np.inf)
            dq = []
            for i, g in enumerate(grads):
                dg = torch.from_numpy(g).cuda()
                q = torch.zeros(g.size + 16, dtype=torch.int8 if bits == 8 else torch.int16, device="cuda")
                B.kahan_sgd_import_dev(dg.data_ptr(), q.data_ptr(), None, g.size, bits, 0, 0,
                                       exps_dev.data_ptr() + 4 * i, scratch.data_ptr(), st)
                dq.append(q)
            gpu.B.kahan_sgd_step_qgrad_dev(gpu.handle, [q.data_ptr() for q in dq], bits, exps_dev.data_ptr(), lrs)
            want_e = [oracle_fit_exponent(g, bits) for g in grads]
            want_q = [oracle_quantize(g, bits, 0, 0, e)[0] for g, e in zip(grads, want_e)]
            oracle_step_qgrad(ost, want_q, want_e, lrs)
            assert exps_dev.cpu().tolist() == want_e
            for q, w in zip(dq, want_q):
                assert np.array_equal(q[:w.size].cpu().numpy(), w)
            assert bool((scratch == 0).all())
            assert_same_state(gpu, ost, f"step {step}")
    finally:
        gpu.close()


def test_conversions_of_unaligned_and_ragged_arrays():
    """Source and outputs at odd element offsets (the scalar path), and lengths that are not a
    multiple of four (the tail of the vector path), with a guard value past the end."""
    import torch
    from paper_1810_05486_b200 import binding as B
    rng = np.random.default_rng(77)
    st = torch.cuda.current_stream().cuda_stream
    for tb, cb in ((8, 8), (16, 16), (8, 0), (16, 8)):
        for n, off in ((4097, 0), (4099, 1), (130, 3), (5, 2)):
            x = (rng.standard_normal(n + off) * 0.2).astype(np.float32)
            dx = torch.from_numpy(x).cuda()
            th = torch.full((n + off + 32,), 0x5A, dtype=torch.int8 if tb == 8 else torch.int16, device="cuda")
            c = torch.full((n + off + 32,), 0x5A, dtype=torch.int8 if cb <= 8 else torch.int16, device="cuda")
            scratch = torch.zeros(4, dtype=torch.int32, device="cuda")
            e = B.kahan_sgd_import(dx.data_ptr() + 4 * off, th.data_ptr() + off * (tb // 8),
                                   (c.data_ptr() + off * (max(cb, 8) // 8)) if cb else None, n, tb, cb, 0,
                                   B.KSGD_EXP_AUTO, scratch.data_ptr(), st)
            assert e == oracle_fit_exponent(np.ascontiguousarray(x[off:]), tb)
            wt, wc = oracle_quantize(np.ascontiguousarray(x[off:]), tb, cb, 0, e)
            assert np.array_equal(th[off:off + n].cpu().numpy(), wt)
            assert bool((th[:off] == 0x5A).all()) and bool((th[off + n:] == 0x5A).all())
            if cb:
                assert np.array_equal(c[off:off + n].cpu().numpy(), wc)
                assert bool((c[:off] == 0x5A).all()) and bool((c[off + n:] == 0x5A).all())
            out = torch.full((n + off + 8,), 7.0, dtype=torch.float32, device="cuda")
            B.kahan_sgd_export(th.data_ptr() + off * (tb // 8), (c.data_ptr() + off * (max(cb, 8) // 8)) if cb else None,
                               out.data_ptr() + 4 * off, n, tb, cb, 0, e, st)
            want = oracle_dequantize(wt, wc, tb, cb, 0, e)
            assert np.array_equal(out[off:off + n].cpu().numpy().view(np.uint32), want.view(np.uint32))
            assert bool((out[:off] == 7.0).all()) and bool((out[off + n:] == 7.0).all())
