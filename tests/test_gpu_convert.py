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
