"""The synthetic workloads: shapes, totals, determinism and slice-wise regeneration."""
import numpy as np
import pytest

from paper_1810_05486_b200 import workloads as W


def test_shapes_and_totals():
    want = {"c1_single": (1, 1_048_576), "c2_resnet20": (22, 269_712),
            "c3_resnet50": (161, 25_557_032), "c4_alexnet": (16, 61_100_840),
            "c5_sweep": (1024, 1_000_000_000)}
    for name, (nt, numel) in want.items():
        wl = W.workload(name)
        assert (len(wl.tensors), wl.numel) == (nt, numel)
    assert W.workload("c1_single").bytes_per_step == 8 * 1_048_576
    assert W.workload("c3_resnet50").bytes_per_step == 10 * 25_557_032
    assert W.workload("c5_sweep").bytes_per_step == 12 * 1_000_000_000
    c4 = W.workload("c4_alexnet")
    assert [t.theta_bits for t in c4.tensors][-2:] == [16, 16]
    assert sum(t.numel for t in c4.tensors if t.theta_bits == 16) == 4_097_000
    sizes = [t.numel for t in W.workload("c5_sweep").tensors]
    assert min(sizes) >= 1024 and any(s % 16 for s in sizes)


def test_resnet20_exponents_fit_their_ranges():
    wl = W.workload("c2_resnet20")
    by = {t.name: t for t in wl.tensors}
    assert by["bn.scale"].exp_theta == -6 and by["bn.bias"].exp_theta == -10
    for t in wl.tensors:
        assert 127 * 2.0 ** t.exp_theta > 0.09          # grid reaches the intended maximum
        assert t.grad_sigma == pytest.approx(1e-2 * 127 * 2.0 ** t.exp_theta)


def test_draws_are_deterministic_and_sliceable():
    wl = W.scaled_sweep(3_000_000, 5)
    a, _ = W.initial_state(wl, seed=0, threads=1)
    b, _ = W.initial_state(wl, seed=0, threads=4)
    c, _ = W.initial_state(wl, seed=1)
    for x, y, z in zip(a, b, c):
        assert np.array_equal(x, y) and not np.array_equal(x, z)
        assert x.min() >= -32767 and x.max() <= 32767
    g0 = W.gradients(wl, 0)
    g2 = W.gradients(wl, 2)      # period 2: step 2 repeats step 0
    g1 = W.gradients(wl, 1)
    tid = int(np.argmax([t.numel for t in wl.tensors]))
    assert np.array_equal(g0[tid], g2[tid]) and not np.array_equal(g0[tid], g1[tid])
    n = wl.tensors[tid].numel
    lo, hi = min(n - 2, W.SEGMENT - 5), min(n, W.SEGMENT + 11)
    assert np.array_equal(W.grad_slice(wl, tid, 0, lo, hi), g0[tid][lo:hi])
    assert np.array_equal(W.theta_slice(wl, tid, lo, hi), a[tid][lo:hi])


def test_gradient_distributions():
    wl = W.workload("c1_single")
    g = W.gradients(wl, 3)[0]
    assert g.dtype == np.float32 and abs(float(g.std()) - 1e-3) < 2e-5
    c4 = W.workload("c4_alexnet")
    g = W.grad_slice(c4, 10, 0, 0, 1_000_000)      # fc6.weight
    assert abs(float(np.median(np.abs(g))) - 0.7649e-3) < 2e-5   # median |t_3| = 0.7649
    assert float(np.abs(g).max()) > 2e-2                         # heavy tail
