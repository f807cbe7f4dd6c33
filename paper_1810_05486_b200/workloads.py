"""Seeded synthetic parameter sets and gradients shaped like the paper's networks.

This module only describes and draws INPUTS: tensor shapes, formats, initial
exponents, integer mantissas and fp32 gradients.  It contains none of the
update's arithmetic, so both the CUDA library's tests and the CPU oracle can
feed on the same bytes.

The five workloads stand in for the networks trained in Section 4 of
arXiv 1810.05486 (whose datasets and weights are not needed for an optimizer
update): only the tensor shapes of the public architectures are used.

  c1_single     one tensor of 2^20 parameters, int8 parameter / int8 compensation
  c2_resnet20   ResNet-20 (CIFAR-10) parameter list, 22 tensors, int8/int8
  c3_resnet50   ResNet-50 parameter list, 161 tensors, int16/int8
  c4_alexnet    AlexNet parameter list, 16 tensors, int8/int8 with the last FC
                layer at int16/int16 (Section 4.2 keeps that layer at 16 bits)
  c5_sweep      10^9 parameters in 1024 tensors of log-uniform size, int16/int16

Every array is drawn in independent segments of 2^20 elements, each from
numpy's PCG64 seeded by SeedSequence([seed, config, tensor, stream, step,
segment]), so any slice of any tensor can be regenerated alone (that is how the
full-size parity check samples a 10^9-parameter run) and segments can be drawn
by several threads.
"""
import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

SEGMENT = 1 << 20
_STREAM_THETA = 0
_STREAM_GRAD = 1


@dataclass(frozen=True)
class TensorSpec:
    name: str
    numel: int
    theta_bits: int      # 8 or 16
    comp_bits: int       # 0 (plain SGD), 8 or 16
    overlap_k: int       # bits of the compensation that overlap the parameter
    exp_theta: int       # initial shared exponent: value = mantissa * 2^exp_theta
    grad_sigma: float    # scale of this tensor's gradient distribution


@dataclass(frozen=True)
class Workload:
    name: str
    config_id: int
    tensors: Tuple[TensorSpec, ...]
    lr: float
    steps: int
    grad_dist: str               # "normal" or "student_t3"
    grad_period: Optional[int]   # gradients repeat with this period (None: fresh every step)

    @property
    def numel(self) -> int:
        return sum(t.numel for t in self.tensors)

    @property
    def bytes_per_step(self) -> int:
        """Algorithmic HBM bytes of one step: read+write both mantissa arrays, read fp32 g."""
        return sum(t.numel * (2 * (t.theta_bits // 8) + 2 * (t.comp_bits // 8) + 4)
                   for t in self.tensors)


def storage_dtype(bits: int):
    return np.int8 if bits <= 8 else np.int16


def qmax(bits: int) -> int:
    return (1 << (bits - 1)) - 1


def _fit_exponent(amax_real: float, bits: int) -> int:
    """Smallest exponent whose grid still holds amax_real: ceil(log2(amax / QMAX))."""
    return math.ceil(math.log2(amax_real / qmax(bits)))


# ----------------------------------------------------------------------------- shapes

def _c1() -> Workload:
    t = TensorSpec("theta", 1 << 20, 8, 8, 0, -11, 1e-3)
    return Workload("c1_single", 1, (t,), 0.01, 100, "normal", None)


def _c2() -> Workload:
    convs = [(3, 16)] + [(16, 16)] * 6 + [(16, 32)] + [(32, 32)] * 5 + [(32, 64)] + [(64, 64)] * 5
    tensors = []
    for i, (cin, cout) in enumerate(convs):
        e = _fit_exponent(3.0 * math.sqrt(2.0 / (9 * cin)), 8)
        tensors.append(TensorSpec(f"conv{i}.weight", 9 * cin * cout, 8, 8, 0, e,
                                  1e-2 * 127 * 2.0 ** e))
    n_bn = sum(cout for _, cout in convs)
    e = _fit_exponent(1.0, 8)
    tensors.append(TensorSpec("bn.scale", n_bn, 8, 8, 0, e, 1e-2 * 127 * 2.0 ** e))
    e = _fit_exponent(0.1, 8)
    tensors.append(TensorSpec("bn.bias", n_bn, 8, 8, 0, e, 1e-2 * 127 * 2.0 ** e))
    e = _fit_exponent(3.0 * math.sqrt(2.0 / 64), 8)
    tensors.append(TensorSpec("fc.weight", 64 * 10, 8, 8, 0, e, 1e-2 * 127 * 2.0 ** e))
    return Workload("c2_resnet20", 2, tuple(tensors), 0.1, 200, "normal", None)


def _c3() -> Workload:
    shapes = [("conv1", 7 * 7 * 3 * 64, 64)]
    cin = 64
    for stage, (blocks, width) in enumerate(zip([3, 4, 6, 3], [64, 128, 256, 512])):
        for b in range(blocks):
            p = f"layer{stage + 1}.{b}"
            shapes.append((p + ".conv1", cin * width, width))
            shapes.append((p + ".conv2", 9 * width * width, width))
            shapes.append((p + ".conv3", width * width * 4, width * 4))
            if b == 0:
                shapes.append((p + ".downsample", cin * width * 4, width * 4))
            cin = width * 4
    tensors = []
    for name, n, cout in shapes:
        tensors.append(TensorSpec(name + ".weight", n, 16, 8, 0, -17, 1e-4))
        tensors.append(TensorSpec(name + ".bn_scale", cout, 16, 8, 0, -17, 1e-4))
        tensors.append(TensorSpec(name + ".bn_bias", cout, 16, 8, 0, -17, 1e-4))
    tensors.append(TensorSpec("fc.weight", 2048 * 1000, 16, 8, 0, -17, 1e-4))
    tensors.append(TensorSpec("fc.bias", 1000, 16, 8, 0, -17, 1e-4))
    return Workload("c3_resnet50", 3, tuple(tensors), 0.1, 50, "normal", None)


def _c4() -> Workload:
    layers = [("conv1", 64 * 3 * 11 * 11, 64), ("conv2", 192 * 64 * 5 * 5, 192),
              ("conv3", 384 * 192 * 3 * 3, 384), ("conv4", 256 * 384 * 3 * 3, 256),
              ("conv5", 256 * 256 * 3 * 3, 256), ("fc6", 9216 * 4096, 4096),
              ("fc7", 4096 * 4096, 4096), ("fc8", 4096 * 1000, 1000)]
    tensors = []
    for name, n, cout in layers:
        bits, e = (16, -19) if name == "fc8" else (8, -11)
        tensors.append(TensorSpec(name + ".weight", n, bits, bits, 0, e, 1e-3))
        tensors.append(TensorSpec(name + ".bias", cout, bits, bits, 0, e, 1e-3))
    return Workload("c4_alexnet", 4, tuple(tensors), 0.01, 20, "student_t3", None)


def c5_sizes(total: int = 1_000_000_000, n_tensors: int = 1024, seed: int = 0,
             min_size: int = 1024) -> List[int]:
    """Log-uniform tensor sizes 2^10..2^24, rescaled so that they sum to `total` exactly.
    The rounding remainder goes to the last tensor (to the largest one if the last would
    drop below min_size, which only happens for scaled-down totals)."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 5, 0xC5])))
    raw = np.floor(2.0 ** (10.0 + 14.0 * rng.random(n_tensors)))
    rho = total / raw.sum()
    sizes = np.maximum(min_size, np.rint(rho * raw)).astype(np.int64)
    rest = total - int(sizes.sum())
    sink = n_tensors - 1 if sizes[-1] + rest >= min_size else int(np.argmax(sizes))
    sizes[sink] += rest
    assert sizes.min() >= min_size and int(sizes.sum()) == total
    return [int(x) for x in sizes]


def _c5(total: int = 1_000_000_000, n_tensors: int = 1024, min_size: int = 1024) -> Workload:
    tensors = tuple(TensorSpec(f"t{i}", n, 16, 16, 0, -15, 1e-3)
                    for i, n in enumerate(c5_sizes(total, n_tensors, 0, min_size)))
    return Workload("c5_sweep", 5, tensors, 0.01, 10, "normal", 2)


_BUILDERS = {"c1_single": _c1, "c2_resnet20": _c2, "c3_resnet50": _c3, "c4_alexnet": _c4,
             "c5_sweep": _c5}
WORKLOADS = tuple(_BUILDERS)


def workload(name: str) -> Workload:
    return _BUILDERS[name]()


def scaled_sweep(total: int, n_tensors: int) -> Workload:
    """The c5 recipe at a smaller size (same size law and formats); used by quick tests."""
    return _c5(total, n_tensors, min_size=max(1, min(1024, total // (64 * n_tensors))))


# ----------------------------------------------------------------------------- drawing

def _rng(seed: int, config_id: int, tensor_id: int, stream: int, step: int, seg: int):
    return np.random.Generator(np.random.PCG64(
        np.random.SeedSequence([seed, config_id, tensor_id, stream, step, seg])))


def _segments(lo: int, hi: int):
    """(segment index, start, stop) triples covering [lo, hi) along SEGMENT boundaries."""
    seg = lo // SEGMENT
    while seg * SEGMENT < hi:
        a, b = max(lo, seg * SEGMENT), min(hi, (seg + 1) * SEGMENT)
        yield seg, a, b
        seg += 1


def _draw_theta_segment(wl: Workload, tid: int, seed: int, seg: int, n: int) -> np.ndarray:
    t = wl.tensors[tid]
    q = qmax(t.theta_bits)
    return _rng(seed, wl.config_id, tid, _STREAM_THETA, 0, seg).integers(
        -q, q + 1, size=n, dtype=storage_dtype(t.theta_bits))


def _draw_grad_segment(wl: Workload, tid: int, seed: int, step: int, seg: int, n: int) -> np.ndarray:
    t = wl.tensors[tid]
    rng = _rng(seed, wl.config_id, tid, _STREAM_GRAD, step, seg)
    if wl.grad_dist == "normal":
        g = rng.standard_normal(n, dtype=np.float32)
        g *= np.float32(t.grad_sigma)
        return g
    if wl.grad_dist == "student_t3":
        return (rng.standard_t(3.0, n) * t.grad_sigma).astype(np.float32)
    raise ValueError(wl.grad_dist)


def _seg_len(numel: int, seg: int) -> int:
    return min(SEGMENT, numel - seg * SEGMENT)


def theta_slice(wl: Workload, tid: int, lo: int, hi: int, seed: int = 0) -> np.ndarray:
    """Initial parameter mantissas [lo, hi) of tensor tid, uniform over the symmetric range."""
    t = wl.tensors[tid]
    out = np.empty(hi - lo, dtype=storage_dtype(t.theta_bits))
    for seg, a, b in _segments(lo, hi):
        full = _draw_theta_segment(wl, tid, seed, seg, _seg_len(t.numel, seg))
        out[a - lo:b - lo] = full[a - seg * SEGMENT:b - seg * SEGMENT]
    return out


def grad_step_index(wl: Workload, step: int) -> int:
    return step if wl.grad_period is None else step % wl.grad_period


def grad_slice(wl: Workload, tid: int, step: int, lo: int, hi: int, seed: int = 0) -> np.ndarray:
    """fp32 gradient [lo, hi) of tensor tid at training step `step`."""
    t = wl.tensors[tid]
    k = grad_step_index(wl, step)
    out = np.empty(hi - lo, dtype=np.float32)
    for seg, a, b in _segments(lo, hi):
        full = _draw_grad_segment(wl, tid, seed, k, seg, _seg_len(t.numel, seg))
        out[a - lo:b - lo] = full[a - seg * SEGMENT:b - seg * SEGMENT]
    return out


def _default_threads() -> int:
    return max(1, min(32, len(os.sched_getaffinity(0))))


def _fill(jobs, threads: Optional[int]) -> None:
    threads = threads or _default_threads()
    if threads == 1 or len(jobs) == 1:
        for fn in jobs:
            fn()
        return
    with ThreadPoolExecutor(threads) as pool:
        for _ in pool.map(lambda fn: fn(), jobs):
            pass


def fill_theta(wl: Workload, out: Sequence[np.ndarray], seed: int = 0,
               threads: Optional[int] = None) -> None:
    """Draw every tensor's initial mantissas into the caller's arrays (one per tensor)."""
    jobs = []
    for tid, t in enumerate(wl.tensors):
        assert out[tid].size == t.numel and out[tid].dtype == storage_dtype(t.theta_bits)
        for seg, a, b in _segments(0, t.numel):
            def job(tid=tid, seg=seg, a=a, b=b):
                out[tid][a:b] = _draw_theta_segment(wl, tid, seed, seg, b - a)
            jobs.append(job)
    _fill(jobs, threads)


def fill_grads(wl: Workload, step: int, out: Sequence[np.ndarray], seed: int = 0,
               threads: Optional[int] = None) -> None:
    """Draw every tensor's gradient of training step `step` into the caller's fp32 arrays."""
    k = grad_step_index(wl, step)
    jobs = []
    for tid, t in enumerate(wl.tensors):
        assert out[tid].size == t.numel and out[tid].dtype == np.float32
        for seg, a, b in _segments(0, t.numel):
            def job(tid=tid, seg=seg, a=a, b=b):
                out[tid][a:b] = _draw_grad_segment(wl, tid, seed, k, seg, b - a)
            jobs.append(job)
    _fill(jobs, threads)


def initial_state(wl: Workload, seed: int = 0, threads: Optional[int] = None):
    """(theta arrays, compensation arrays) at step 0; compensation starts at zero."""
    thetas = [np.empty(t.numel, dtype=storage_dtype(t.theta_bits)) for t in wl.tensors]
    fill_theta(wl, thetas, seed, threads)
    comps = [np.zeros(t.numel, dtype=storage_dtype(t.comp_bits)) if t.comp_bits else None
             for t in wl.tensors]
    return thetas, comps


def gradients(wl: Workload, step: int, seed: int = 0, threads: Optional[int] = None):
    grads = [np.empty(t.numel, dtype=np.float32) for t in wl.tensors]
    fill_grads(wl, step, grads, seed, threads)
    return grads
