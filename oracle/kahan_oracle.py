"""ctypes binding of the C oracle plus the multi-tensor step built on it.

Test infrastructure only.  The per-element arithmetic lives in kahan_oracle.c;
this module adds what surrounds it in a training step (Algorithm 1 applied to
every parameter tensor, then the exponent choice for the next step) and keeps
the per-tensor state a caller would checkpoint.
"""
import ctypes
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

from . import build as _build

EXP_FIXED = 0
EXP_AMAX = 1


class OracleElem(ctypes.Structure):
    _fields_ = [("P", ctypes.c_int64), ("Rq", ctypes.c_int64), ("T", ctypes.c_int64),
                ("d", ctypes.c_int32), ("q_theta", ctypes.c_int32),
                ("q_comp", ctypes.c_int32), ("nonfinite", ctypes.c_int32)]


class OracleMomElem(ctypes.Structure):
    _fields_ = [("upd", OracleElem), ("V", ctypes.c_int64), ("q_mom", ctypes.c_int32)]


class _Stats(ctypes.Structure):
    _fields_ = [("amax_theta", ctypes.c_uint32), ("amax_comp", ctypes.c_uint32),
                ("n_sat_theta", ctypes.c_uint64), ("n_sat_comp", ctypes.c_uint64),
                ("n_nonfinite", ctypes.c_uint64)]


class _MomStats(ctypes.Structure):
    _fields_ = [("upd", _Stats), ("amax_mom", ctypes.c_uint32), ("n_sat_mom", ctypes.c_uint64)]


class OracleAdamElem(ctypes.Structure):
    _fields_ = [("upd", OracleElem), ("M", ctypes.c_int64), ("V", ctypes.c_int64),
                ("q_m", ctypes.c_int32), ("q_v", ctypes.c_int32)]


class _AdamStats(ctypes.Structure):
    _fields_ = [("upd", _Stats), ("amax_m", ctypes.c_uint32), ("amax_v", ctypes.c_uint32),
                ("n_sat_m", ctypes.c_uint64), ("n_sat_v", ctypes.c_uint64)]


class OracleStrictElem(ctypes.Structure):
    _fields_ = [("C1", ctypes.c_int64), ("T", ctypes.c_int64), ("P", ctypes.c_int64), ("C2", ctypes.c_int64),
                ("d", ctypes.c_int32), ("q_comp_mid", ctypes.c_int32), ("q_theta", ctypes.c_int32),
                ("q_comp", ctypes.c_int32), ("nonfinite", ctypes.c_int32)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        lib.ksgd_oracle_rne_shift.restype = ctypes.c_int64
        lib.ksgd_oracle_rne_shift.argtypes = [ctypes.c_int64, ctypes.c_int32]
        lib.ksgd_oracle_increment.restype = ctypes.c_int32
        lib.ksgd_oracle_increment.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_int32]
        lib.ksgd_oracle_element.restype = None
        lib.ksgd_oracle_element.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_float,
                                            ctypes.c_float] + [ctypes.c_int32] * 5 + [
                                                ctypes.POINTER(OracleElem)]
        lib.ksgd_oracle_step_tensor.restype = ctypes.c_int
        lib.ksgd_oracle_step_tensor.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
            ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
            ctypes.c_float, ctypes.POINTER(_Stats), ctypes.c_int32]
        lib.ksgd_oracle_next_exponent.restype = ctypes.c_int32
        lib.ksgd_oracle_next_exponent.argtypes = [ctypes.c_uint32, ctypes.c_int32,
                                                  ctypes.c_int32, ctypes.c_int32]
        lib.ksgd_oracle_momentum_element.restype = None
        lib.ksgd_oracle_momentum_element.argtypes = [ctypes.c_int32] * 3 + [ctypes.c_float] * 3 + \
            [ctypes.c_int32] * 8 + [ctypes.POINTER(OracleMomElem)]
        lib.ksgd_oracle_momentum_step_tensor.restype = ctypes.c_int
        lib.ksgd_oracle_momentum_step_tensor.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int64] + \
            [ctypes.c_int32] * 8 + [ctypes.c_float, ctypes.c_float, ctypes.POINTER(_MomStats),
                                    ctypes.c_int32]
        lib.ksgd_oracle_next_exponent_velocity.restype = ctypes.c_int32
        lib.ksgd_oracle_next_exponent_velocity.argtypes = [ctypes.c_uint32, ctypes.c_int32,
                                                           ctypes.c_int32, ctypes.c_int32]
        lib.ksgd_oracle_fit_exponent.restype = ctypes.c_int32
        lib.ksgd_oracle_fit_exponent.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32]
        lib.ksgd_oracle_quantize.restype = None
        lib.ksgd_oracle_quantize.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int64] + [ctypes.c_int32] * 4
        lib.ksgd_oracle_dequantize.restype = None
        lib.ksgd_oracle_dequantize.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int64] + [ctypes.c_int32] * 4
        lib.ksgd_oracle_adam_element.restype = None
        lib.ksgd_oracle_adam_element.argtypes = [ctypes.c_int32] * 4 + [ctypes.c_float] * 5 + \
            [ctypes.c_int32] * 9 + [ctypes.POINTER(OracleAdamElem)]
        lib.ksgd_oracle_adam_step_tensor.restype = ctypes.c_int
        lib.ksgd_oracle_adam_step_tensor.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_int64] + \
            [ctypes.c_int32] * 9 + [ctypes.c_float] * 4 + [ctypes.POINTER(_AdamStats), ctypes.c_int32]
        lib.ksgd_oracle_strict_element.restype = None
        lib.ksgd_oracle_strict_element.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_float,
                                                   ctypes.c_float] + [ctypes.c_int32] * 6 + \
            [ctypes.POINTER(OracleStrictElem)]
        lib.ksgd_oracle_strict_step_tensor.restype = ctypes.c_int
        lib.ksgd_oracle_strict_step_tensor.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int64] + \
            [ctypes.c_int32] * 6 + [ctypes.c_float, ctypes.POINTER(_Stats), ctypes.c_int32]
        lib.ksgd_oracle_next_exponent_acc.restype = ctypes.c_int32
        lib.ksgd_oracle_next_exponent_acc.argtypes = [ctypes.c_uint32] + [ctypes.c_int32] * 4
        lib.ksgd_oracle_max_threads.restype = ctypes.c_int32
        lib.ksgd_oracle_max_threads.argtypes = []
        _lib = lib
    return _lib


def oracle_max_threads() -> int:
    return int(_load().ksgd_oracle_max_threads())


def oracle_rne_shift(a: int, r: int) -> int:
    """a / 2^r rounded to nearest, ties to even."""
    return int(_load().ksgd_oracle_rne_shift(a, r))


def oracle_increment(g: float, lr: float, ec_out: int) -> int:
    """Algorithm 1 statement 1: eta*g rounded onto the accumulator grid 2^ec_out."""
    return int(_load().ksgd_oracle_increment(g, lr, ec_out))


def oracle_element(q_theta: int, q_comp: int, g: float, lr: float, m: int, n: int, s: int,
                   e_in: int, e_out: int) -> OracleElem:
    """Algorithm 1 for one element with m-bit parameter and n-bit compensation."""
    out = OracleElem()
    _load().ksgd_oracle_element(q_theta, q_comp, g, lr, m, n, s, e_in, e_out,
                                ctypes.byref(out))
    return out


def oracle_next_exponent(amax_theta: int, theta_bits: int, e_out: int, mode: int) -> int:
    """Exponent of the next step from this step's max |P| (max scan)."""
    return int(_load().ksgd_oracle_next_exponent(amax_theta, theta_bits, e_out, mode))


def oracle_next_exponent_velocity(amax_mom: int, mom_bits: int, ev_out: int, mode: int) -> int:
    """Velocity exponent of the next step: kept while the largest mantissa is in (QMAX/4, QMAX]."""
    return int(_load().ksgd_oracle_next_exponent_velocity(amax_mom, mom_bits, ev_out, mode))


def oracle_fit_exponent(x: np.ndarray, bits: int) -> int:
    """Smallest exponent whose b-bit grid holds max|x| (finite values only)."""
    assert x.dtype == np.float32 and x.flags.c_contiguous
    return int(_load().ksgd_oracle_fit_exponent(x.ctypes.data, x.size, bits))


def oracle_quantize(x: np.ndarray, theta_bits: int, comp_bits: int, overlap_k: int, e: int):
    """fp32 -> (theta mantissas, compensation mantissas or None) at exponent e."""
    assert x.dtype == np.float32 and x.flags.c_contiguous
    theta = np.empty(x.size, _storage_dtype(theta_bits))
    comp = np.empty(x.size, _storage_dtype(comp_bits)) if comp_bits else None
    _load().ksgd_oracle_quantize(x.ctypes.data, theta.ctypes.data, comp.ctypes.data if comp_bits else None,
                                 x.size, theta_bits, comp_bits, overlap_k, e)
    return theta, comp


def oracle_dequantize(theta: np.ndarray, comp, theta_bits: int, comp_bits: int, overlap_k: int,
                      e: int) -> np.ndarray:
    """(theta, compensation) at exponent e -> fp32, one rounding."""
    x = np.empty(theta.size, np.float32)
    _load().ksgd_oracle_dequantize(theta.ctypes.data, comp.ctypes.data if comp_bits else None,
                                   x.ctypes.data, theta.size, theta_bits, comp_bits, overlap_k, e)
    return x


def _storage_dtype(bits: int):
    return np.int8 if bits <= 8 else np.int16


def oracle_step_tensor(theta: np.ndarray, comp: Optional[np.ndarray], grad: np.ndarray,
                       theta_bits: int, comp_bits: int, overlap_k: int, e_in: int, e_out: int,
                       lr: float, n_threads: int = 1) -> dict:
    """Algorithm 1 over one tensor, in place on theta and comp; returns the step's stats."""
    assert theta.dtype == _storage_dtype(theta_bits) and theta.flags.c_contiguous
    assert grad.dtype == np.float32 and grad.flags.c_contiguous and grad.size == theta.size
    if comp_bits:
        assert comp is not None and comp.dtype == _storage_dtype(comp_bits)
        assert comp.flags.c_contiguous and comp.size == theta.size
    st = _Stats()
    rc = _load().ksgd_oracle_step_tensor(
        theta.ctypes.data, comp.ctypes.data if comp_bits else None, grad.ctypes.data,
        theta.size, theta_bits, comp_bits, overlap_k, e_in, e_out,
        ctypes.c_float(lr), ctypes.byref(st), n_threads)
    if rc != 0:
        raise ValueError("oracle rejected the tensor description")
    return {"amax_theta": st.amax_theta, "amax_comp": st.amax_comp,
            "n_sat_theta": st.n_sat_theta, "n_sat_comp": st.n_sat_comp,
            "n_nonfinite": st.n_nonfinite}


def oracle_momentum_element(q_theta: int, q_comp: int, q_mom: int, g: float, lr: float, mu: float,
                            m: int, n: int, s: int, b: int, e_in: int, e_out: int, ev_in: int,
                            ev_out: int) -> OracleMomElem:
    """Momentum with the lazy update for one element (v <- mu v + eta g, then Algorithm 1 with v)."""
    out = OracleMomElem()
    _load().ksgd_oracle_momentum_element(q_theta, q_comp, q_mom, g, lr, mu, m, n, s, b, e_in, e_out,
                                         ev_in, ev_out, ctypes.byref(out))
    return out


def oracle_momentum_step_tensor(theta, comp, mom, grad, theta_bits, comp_bits, overlap_k, mom_bits,
                                e_in, e_out, ev_in, ev_out, lr, mu, n_threads: int = 1) -> dict:
    """Momentum step over one tensor, in place on theta, comp and mom; returns the stats."""
    assert theta.dtype == _storage_dtype(theta_bits) and theta.flags.c_contiguous
    assert mom.dtype == _storage_dtype(mom_bits) and mom.flags.c_contiguous and mom.size == theta.size
    assert grad.dtype == np.float32 and grad.flags.c_contiguous and grad.size == theta.size
    if comp_bits:
        assert comp is not None and comp.dtype == _storage_dtype(comp_bits) and comp.size == theta.size
    st = _MomStats()
    rc = _load().ksgd_oracle_momentum_step_tensor(
        theta.ctypes.data, comp.ctypes.data if comp_bits else None, mom.ctypes.data, grad.ctypes.data,
        theta.size, theta_bits, comp_bits, overlap_k, mom_bits, e_in, e_out, ev_in, ev_out,
        ctypes.c_float(lr), ctypes.c_float(mu), ctypes.byref(st), n_threads)
    if rc != 0:
        raise ValueError("oracle rejected the tensor description")
    return {"amax_theta": st.upd.amax_theta, "amax_comp": st.upd.amax_comp,
            "n_sat_theta": st.upd.n_sat_theta, "n_sat_comp": st.upd.n_sat_comp,
            "n_nonfinite": st.upd.n_nonfinite, "amax_mom": st.amax_mom, "n_sat_mom": st.n_sat_mom}


def oracle_adam_element(q_theta, q_comp, q_m, q_v, g, lr, beta1, beta2, eps, m, n, s, e_in, e_out,
                        em_in, em_out, ev_in, ev_out) -> OracleAdamElem:
    """ADAM with the lazy update for one element (16-bit moments)."""
    out = OracleAdamElem()
    _load().ksgd_oracle_adam_element(q_theta, q_comp, q_m, q_v, g, lr, beta1, beta2, eps, m, n, s,
                                     e_in, e_out, em_in, em_out, ev_in, ev_out, ctypes.byref(out))
    return out


def oracle_adam_step_tensor(theta, comp, mom1, mom2, grad, theta_bits, comp_bits, overlap_k, e_in, e_out,
                            em_in, em_out, ev_in, ev_out, lr, beta1, beta2, eps, n_threads: int = 1) -> dict:
    """ADAM step over one tensor, in place on theta, comp and both moments; returns the stats."""
    assert theta.dtype == _storage_dtype(theta_bits) and theta.flags.c_contiguous
    for a in (mom1, mom2):
        assert a.dtype == np.int16 and a.flags.c_contiguous and a.size == theta.size
    assert grad.dtype == np.float32 and grad.flags.c_contiguous and grad.size == theta.size
    st = _AdamStats()
    rc = _load().ksgd_oracle_adam_step_tensor(
        theta.ctypes.data, comp.ctypes.data if comp_bits else None, mom1.ctypes.data, mom2.ctypes.data,
        grad.ctypes.data, theta.size, theta_bits, comp_bits, overlap_k, e_in, e_out, em_in, em_out,
        ev_in, ev_out, ctypes.c_float(lr), ctypes.c_float(beta1), ctypes.c_float(beta2),
        ctypes.c_float(eps), ctypes.byref(st), n_threads)
    if rc != 0:
        raise ValueError("oracle rejected the tensor description")
    return {"amax_theta": st.upd.amax_theta, "amax_comp": st.upd.amax_comp,
            "n_sat_theta": st.upd.n_sat_theta, "n_sat_comp": st.upd.n_sat_comp,
            "n_nonfinite": st.upd.n_nonfinite, "amax_m": st.amax_m, "amax_v": st.amax_v,
            "n_sat_m": st.n_sat_m, "n_sat_v": st.n_sat_v}


def oracle_strict_element(q_theta, q_comp, g, lr, m, n, e_in, e_out, ec_in, ec_out) -> OracleStrictElem:
    """Strict Algorithm 1 for one element (accumulator with its own exponent)."""
    out = OracleStrictElem()
    _load().ksgd_oracle_strict_element(q_theta, q_comp, g, lr, m, n, e_in, e_out, ec_in, ec_out,
                                       ctypes.byref(out))
    return out


def oracle_strict_step_tensor(theta, comp, grad, theta_bits, comp_bits, e_in, e_out, ec_in, ec_out, lr,
                              n_threads: int = 1) -> dict:
    assert theta.dtype == _storage_dtype(theta_bits) and comp.dtype == _storage_dtype(comp_bits)
    assert theta.flags.c_contiguous and comp.flags.c_contiguous and comp.size == theta.size
    assert grad.dtype == np.float32 and grad.flags.c_contiguous and grad.size == theta.size
    st = _Stats()
    rc = _load().ksgd_oracle_strict_step_tensor(theta.ctypes.data, comp.ctypes.data, grad.ctypes.data,
                                                theta.size, theta_bits, comp_bits, e_in, e_out, ec_in, ec_out,
                                                ctypes.c_float(lr), ctypes.byref(st), n_threads)
    if rc != 0:
        raise ValueError("oracle rejected the tensor description")
    return {"amax_theta": st.amax_theta, "amax_comp": st.amax_comp, "n_sat_theta": st.n_sat_theta,
            "n_sat_comp": st.n_sat_comp, "n_nonfinite": st.n_nonfinite}


def oracle_next_exponent_acc(amax_comp: int, comp_bits: int, ec_out: int, e_next: int, mode: int) -> int:
    return int(_load().ksgd_oracle_next_exponent_acc(amax_comp, comp_bits, ec_out, e_next, mode))


@dataclass
class OracleTensor:
    """One parameter tensor: mantissas, compensation, formats and exponents."""
    theta: np.ndarray
    comp: Optional[np.ndarray]
    theta_bits: int
    comp_bits: int
    overlap_k: int = 0
    exp_theta: int = 0          # exponent of the mantissas now stored
    exp_theta_next: int = 0     # exponent the next step writes
    amax_theta: int = 0         # of the most recent step
    amax_comp: int = 0
    n_sat_theta: int = 0        # cumulative
    n_sat_comp: int = 0
    n_nonfinite: int = 0
    # momentum variant only
    mom: Optional[np.ndarray] = None
    mom_bits: int = 0
    exp_mom: int = 0
    exp_mom_next: int = 0
    amax_mom: int = 0
    n_sat_mom: int = 0
    # strict Algorithm 1 only: the compensation's own exponent
    exp_comp: int = 0
    exp_comp_next: int = 0
    # ADAM only: `mom` is the first moment, `mom2` the second
    mom2: Optional[np.ndarray] = None
    exp_mom2: int = 0
    exp_mom2_next: int = 0
    amax_mom2: int = 0
    n_sat_mom2: int = 0

    @property
    def s(self) -> int:
        return 0 if self.comp_bits == 0 else self.comp_bits - 1 - self.overlap_k


@dataclass
class OracleState:
    tensors: List[OracleTensor] = field(default_factory=list)
    mode: int = EXP_AMAX
    n_threads: int = 1


def oracle_step(state: OracleState, grads: Sequence[np.ndarray], lrs: Sequence[float]) -> None:
    """One training-step update of every tensor, then the exponent choice.

    Each tensor is read at exp_theta and written at exp_theta_next (chosen from
    the previous step's max scan); afterwards exp_theta becomes the exponent
    just written and exp_theta_next the tight fit of this step's max |P|.
    """
    assert len(grads) == len(state.tensors) == len(lrs)
    for t, g, lr in zip(state.tensors, grads, lrs):
        e_in, e_out = t.exp_theta, t.exp_theta_next
        st = oracle_step_tensor(t.theta, t.comp, g, t.theta_bits, t.comp_bits, t.overlap_k,
                                e_in, e_out, float(lr), state.n_threads)
        t.amax_theta, t.amax_comp = st["amax_theta"], st["amax_comp"]
        t.n_sat_theta += st["n_sat_theta"]
        t.n_sat_comp += st["n_sat_comp"]
        t.n_nonfinite += st["n_nonfinite"]
        t.exp_theta = e_out
        t.exp_theta_next = oracle_next_exponent(t.amax_theta, t.theta_bits, e_out, state.mode)


def oracle_dequantize_gradient(q: np.ndarray, exp_grad: int) -> np.ndarray:
    """A fixed-point gradient tensor as binary32 values: Q * 2^exp_grad is exact for 8- and
    16-bit mantissas and exponents in [-64, 64]."""
    assert q.dtype in (np.int8, np.int16) and -64 <= exp_grad <= 64
    return np.ldexp(q.astype(np.float32), np.int32(exp_grad)).astype(np.float32)


def oracle_step_qgrad(state: OracleState, grads_q: Sequence[np.ndarray], exp_grads: Sequence[int],
                      lrs: Sequence[float]) -> None:
    """The step with gradients given in dynamic fixed point (the paper's hardware model,
    Section 1): by definition the plain step on the exactly dequantized gradients."""
    oracle_step(state, [oracle_dequantize_gradient(q, e) for q, e in zip(grads_q, exp_grads)], lrs)


def oracle_momentum_step(state: OracleState, grads: Sequence[np.ndarray], lrs: Sequence[float],
                         mus: Sequence[float]) -> None:
    """One momentum step of every tensor, then the exponent choices: theta's exponent
    follows max |P|, the velocity's exponent follows max |V|, each on its own (the velocity's with a dead band)."""
    assert len(grads) == len(state.tensors) == len(lrs) == len(mus)
    for t, g, lr, mu in zip(state.tensors, grads, lrs, mus):
        e_in, e_out, ev_in, ev_out = t.exp_theta, t.exp_theta_next, t.exp_mom, t.exp_mom_next
        st = oracle_momentum_step_tensor(t.theta, t.comp, t.mom, g, t.theta_bits, t.comp_bits,
                                         t.overlap_k, t.mom_bits, e_in, e_out, ev_in, ev_out,
                                         float(lr), float(mu), state.n_threads)
        t.amax_theta, t.amax_comp, t.amax_mom = st["amax_theta"], st["amax_comp"], st["amax_mom"]
        t.n_sat_theta += st["n_sat_theta"]
        t.n_sat_comp += st["n_sat_comp"]
        t.n_nonfinite += st["n_nonfinite"]
        t.n_sat_mom += st["n_sat_mom"]
        t.exp_theta = e_out
        t.exp_theta_next = oracle_next_exponent(t.amax_theta, t.theta_bits, e_out, state.mode)
        t.exp_mom = ev_out
        t.exp_mom_next = oracle_next_exponent_velocity(t.amax_mom, t.mom_bits, ev_out, state.mode)


def oracle_adam_step(state: OracleState, grads: Sequence[np.ndarray], lrs: Sequence[float], beta1: float,
                     beta2: float, eps: float) -> None:
    """One ADAM step of every tensor (lrs carry the bias correction), then the exponent
    choices: theta's by the tight fit, both moments' with the dead band."""
    assert len(grads) == len(state.tensors) == len(lrs)
    for t, g, lr in zip(state.tensors, grads, lrs):
        e_in, e_out = t.exp_theta, t.exp_theta_next
        em_in, em_out, ev_in, ev_out = t.exp_mom, t.exp_mom_next, t.exp_mom2, t.exp_mom2_next
        st = oracle_adam_step_tensor(t.theta, t.comp, t.mom, t.mom2, g, t.theta_bits, t.comp_bits,
                                     t.overlap_k, e_in, e_out, em_in, em_out, ev_in, ev_out, float(lr),
                                     float(beta1), float(beta2), float(eps), state.n_threads)
        t.amax_theta, t.amax_comp = st["amax_theta"], st["amax_comp"]
        t.amax_mom, t.amax_mom2 = st["amax_m"], st["amax_v"]
        t.n_sat_theta += st["n_sat_theta"]
        t.n_sat_comp += st["n_sat_comp"]
        t.n_nonfinite += st["n_nonfinite"]
        t.n_sat_mom += st["n_sat_m"]
        t.n_sat_mom2 += st["n_sat_v"]
        t.exp_theta = e_out
        t.exp_theta_next = oracle_next_exponent(t.amax_theta, t.theta_bits, e_out, state.mode)
        t.exp_mom = em_out
        t.exp_mom_next = oracle_next_exponent_velocity(t.amax_mom, 16, em_out, state.mode)
        t.exp_mom2 = ev_out
        t.exp_mom2_next = oracle_next_exponent_velocity(t.amax_mom2, 16, ev_out, state.mode)


def oracle_strict_step(state: OracleState, grads: Sequence[np.ndarray], lrs: Sequence[float]) -> None:
    """One strict step of every tensor, then both exponent choices (theta's first: the
    accumulator's window is placed around theta's next exponent)."""
    assert len(grads) == len(state.tensors) == len(lrs)
    for t, g, lr in zip(state.tensors, grads, lrs):
        e_in, e_out, ec_in, ec_out = t.exp_theta, t.exp_theta_next, t.exp_comp, t.exp_comp_next
        st = oracle_strict_step_tensor(t.theta, t.comp, g, t.theta_bits, t.comp_bits, e_in, e_out, ec_in,
                                       ec_out, float(lr), state.n_threads)
        t.amax_theta, t.amax_comp = st["amax_theta"], st["amax_comp"]
        t.n_sat_theta += st["n_sat_theta"]
        t.n_sat_comp += st["n_sat_comp"]
        t.n_nonfinite += st["n_nonfinite"]
        t.exp_theta = e_out
        t.exp_theta_next = oracle_next_exponent(t.amax_theta, t.theta_bits, e_out, state.mode)
        t.exp_comp = ec_out
        t.exp_comp_next = oracle_next_exponent_acc(t.amax_comp, t.comp_bits, ec_out, t.exp_theta_next,
                                                   state.mode)
