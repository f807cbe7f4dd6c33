"""Bit-exact parity of the optimizer variants on the ResNet-50- and AlexNet-shaped workloads
at full size, driven through the same runner (buffers, descriptors, launch configuration)
that the benchmark times: momentum, ADAM, fixed-point gradients, strict Algorithm 1."""
import numpy as np
import pytest

from oracle import (EXP_AMAX, OracleState, OracleTensor, oracle_adam_step, oracle_fit_exponent, oracle_max_threads,
                    oracle_momentum_step, oracle_quantize, oracle_step_qgrad, oracle_strict_step)
from paper_1810_05486_b200 import workloads as W

pytestmark = pytest.mark.gpu

STEPS = 6


def _setup(name, **mode):
    from paper_1810_05486_b200.runner import DeviceRun, HostInputs
    wl = W.workload(name)
    host = HostInputs(wl, seed=0, n_sets=STEPS, pinned=False)
    tensors = [OracleTensor(host.thetas[i].copy(), host.comps[i].copy() if t.comp_bits else None, t.theta_bits,
                            t.comp_bits, t.overlap_k, t.exp_theta, t.exp_theta) for i, t in enumerate(wl.tensors)]
    return wl, host, DeviceRun(host, **mode), OracleState(tensors, EXP_AMAX, oracle_max_threads())


def _check_common(run, ost, st, where):
    for i, t in enumerate(ost.tensors):
        tag = f"{where} tensor {i}"
        assert np.array_equal(run.theta(i), t.theta), tag
        assert np.array_equal(run.comp(i), t.comp), tag
        assert (st["exp_theta_cur"][i], st["exp_theta_next"][i]) == (t.exp_theta, t.exp_theta_next), tag
        assert (st["amax_theta"][i], st["amax_comp"][i]) == (t.amax_theta, t.amax_comp), tag
        assert (st["n_sat_theta"][i], st["n_sat_comp"][i], st["n_nonfinite"][i]) == \
            (t.n_sat_theta, t.n_sat_comp, t.n_nonfinite), tag


@pytest.mark.parametrize("name,bits", [("c3_resnet50", 8), ("c4_alexnet", 16)])
def test_momentum_as_in_the_paper_int8_for_the_cnn_int16_for_alexnet(name, bits):
    wl, host, run, ost = _setup(name, mom_bits=bits)
    try:
        for t in ost.tensors:
            t.mom, t.mom_bits = np.zeros(t.theta.size, W.storage_dtype(bits)), bits
            t.exp_mom = t.exp_mom_next = t.exp_theta - 8
        for step in range(STEPS):
            run.step(step)
            oracle_momentum_step(ost, host.grads[step], [wl.lr] * run.n, [0.9] * run.n)
        st = run.stats()
        _check_common(run, ost, st, name)
        for i, t in enumerate(ost.tensors):
            assert np.array_equal(run.velocity(i), t.mom), i
            assert (st["exp_mom_cur"][i], st["exp_mom_next"][i], st["amax_mom"][i], st["n_sat_mom"][i]) == \
                (t.exp_mom, t.exp_mom_next, t.amax_mom, t.n_sat_mom), i
    finally:
        run.close()


def test_adam_on_resnet50_shapes():
    adam = dict(beta1=0.9, beta2=0.999, eps=1e-8, eta=2e-4)
    wl, host, run, ost = _setup("c3_resnet50", adam=adam)
    try:
        for i, t in enumerate(ost.tensors):
            t.mom, t.mom2, t.mom_bits = np.zeros(t.theta.size, np.int16), np.zeros(t.theta.size, np.int16), 16
            t.exp_mom = t.exp_mom_next = run.adescs[i].exp_m
            t.exp_mom2 = t.exp_mom2_next = run.adescs[i].exp_v
        for step in range(STEPS):
            run.step(step)
            lr_t = float(run.adam_lrs(step + 1)[0])
            oracle_adam_step(ost, host.grads[step], [lr_t] * run.n, adam["beta1"], adam["beta2"], adam["eps"])
        st = run.stats()
        _check_common(run, ost, st, "adam")
        for i, t in enumerate(ost.tensors):
            m1, m2 = run.moments(i)
            assert np.array_equal(m1, t.mom) and np.array_equal(m2, t.mom2), i
            assert (st["exp_m_next"][i], st["exp_v_next"][i], st["amax_m"][i], st["amax_v"][i]) == \
                (t.exp_mom_next, t.exp_mom2_next, t.amax_mom, t.amax_mom2), i
    finally:
        run.close()


def test_int8_gradients_on_alexnet_shapes_quantized_by_the_import_kernel():
    """The runner makes the fixed-point gradients on the device (kahan_sgd_import with the
    exponent from the maximum); the oracle quantizes the same binary32 gradients itself, so
    this also compares the two quantizers at full size."""
    wl, host, run, ost = _setup("c4_alexnet", grad_bits=8)
    try:
        for step in range(STEPS):
            run.step(step)
            exps = [oracle_fit_exponent(g, 8) for g in host.grads[step]]
            assert exps == list(run.gq_exp_sets[step])
            gq = [oracle_quantize(g, 8, 0, 0, e)[0] for g, e in zip(host.grads[step], exps)]
            oracle_step_qgrad(ost, gq, exps, [wl.lr] * run.n)
        _check_common(run, ost, run.stats(), "qgrad")
    finally:
        run.close()


def test_one_handle_alternating_int8_and_binary32_gradients_on_alexnet_shapes():
    """Steps on 8-bit gradients use their own tile table (larger tiles for the 8-bit layers)
    and leave their records where the next step, on binary32 gradients and the other table,
    finds them: the two kinds of step alternate on one handle and every tensor is compared
    after every step."""
    from oracle import oracle_step
    from paper_1810_05486_b200 import binding as B
    wl, host, run, ost = _setup("c4_alexnet", grad_bits=8)
    try:
        for step in range(4):
            if step % 2 == 0:
                run.step(step)
                exps = list(run.gq_exp_sets[step])
                gq = [oracle_quantize(g, 8, 0, 0, e)[0] for g, e in zip(host.grads[step], exps)]
                oracle_step_qgrad(ost, gq, exps, [wl.lr] * run.n)
            else:
                # the runner keeps only the first binary32 gradient set on the device in this mode
                assert len(run.dev_g) == 1
                B.kahan_sgd_step(run.handle, run.grad_ptr_sets[0], run.lrs)
                oracle_step(ost, host.grads[0], [wl.lr] * run.n)
            _check_common(run, ost, run.stats(), f"step {step}")
    finally:
        run.close()


def test_strict_algorithm_1_on_resnet50_shapes():
    from paper_1810_05486_b200 import binding as B
    wl, host, run, ost = _setup("c3_resnet50", strict=True)
    try:
        for t in ost.tensors:
            t.exp_comp = t.exp_comp_next = t.exp_theta - (t.comp_bits - 1 - t.overlap_k)
        for step in range(STEPS):
            run.step(step)
            oracle_strict_step(ost, host.grads[step], [wl.lr] * run.n)
        _check_common(run, ost, run.stats(), "strict")
        ec = B.kahan_sgd_strict_exponents(run.handle, run.n)
        assert ec["exp_comp_cur"] == [t.exp_comp for t in ost.tensors]
        assert ec["exp_comp_next"] == [t.exp_comp_next for t in ost.tensors]
    finally:
        run.close()


def test_strict_algorithm_1_on_int8_gradients_on_alexnet_shapes():
    """Both of the paper's hardware-faithful modes together (INT8 gradients, the accumulator
    rounded into n bits with its own exponent) at full size; these steps walk the tile table
    of large tiles."""
    from oracle import oracle_dequantize_gradient
    from paper_1810_05486_b200 import binding as B
    wl, host, run, ost = _setup("c4_alexnet", strict=True, grad_bits=8)
    try:
        for t in ost.tensors:
            t.exp_comp = t.exp_comp_next = t.exp_theta - (t.comp_bits - 1 - t.overlap_k)
        for step in range(4):
            run.step(step)
            exps = list(run.gq_exp_sets[step])
            gq = [oracle_quantize(g, 8, 0, 0, e)[0] for g, e in zip(host.grads[step], exps)]
            oracle_strict_step(ost, [oracle_dequantize_gradient(q, e) for q, e in zip(gq, exps)], [wl.lr] * run.n)
        _check_common(run, ost, run.stats(), "strict, int8 gradients")
        ec = B.kahan_sgd_strict_exponents(run.handle, run.n)
        assert ec["exp_comp_cur"] == [t.exp_comp for t in ost.tensors]
        assert ec["exp_comp_next"] == [t.exp_comp_next for t in ost.tensors]
    finally:
        run.close()
