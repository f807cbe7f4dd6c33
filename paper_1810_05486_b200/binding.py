"""ctypes binding of the C ABI in include/kahan_sgd.h.

Argument marshalling only: every step of the update runs in the CUDA kernels of
libkahan_sgd.so.  There is no CPU fallback; if the library is missing the import
of this module fails with the build command to run.
"""
import ctypes
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIBRARY = os.path.join(_HERE, "libkahan_sgd.so")

KSGD_EXP_FIXED = 0
KSGD_EXP_AMAX = 1

KSGD_OK = 0
KSGD_ERR_NULL = -1
KSGD_ERR_BITS = -2
KSGD_ERR_OVERLAP = -3
KSGD_ERR_EXP_RANGE = -4
KSGD_ERR_NUMEL = -5
KSGD_ERR_ALIGN = -6
KSGD_ERR_WORKSPACE = -7
KSGD_ERR_LR = -8
KSGD_ERR_CUDA = -9
KSGD_ERR_MODE = -10
KSGD_ERR_DEVICE = -11

EXPORTS = (
    "kahan_sgd_workspace_bytes", "kahan_sgd_workspace_error_offset", "kahan_sgd_tile_table", "kahan_sgd_init", "kahan_sgd_step", "kahan_sgd_step_qgrad",
    "kahan_sgd_step_qgrad_dev", "kahan_sgd_import_dev",
    "kahan_sgd_step_host", "kahan_sgd_strict_workspace_bytes", "kahan_sgd_strict_init",
    "kahan_sgd_strict_exponents",
    "kahan_sgd_amax", "kahan_sgd_set_exponents", "kahan_sgd_step_static", "kahan_sgd_destroy",
    "kahan_sgd_strerror", "kahan_sgd_momentum_workspace_bytes", "kahan_sgd_momentum_init",
    "kahan_sgd_momentum_step", "kahan_sgd_momentum_amax", "kahan_sgd_momentum_destroy",
    "kahan_sgd_adam_workspace_bytes", "kahan_sgd_adam_init", "kahan_sgd_adam_step",
    "kahan_sgd_adam_amax", "kahan_sgd_adam_destroy", "kahan_sgd_adam_selfcheck",
    "kahan_sgd_import", "kahan_sgd_export", "kahan_sgd_classifier_bits",
    "kahan_sgd_last_cuda_error", "kahan_sgd_launch_count",
)


class ksgd_tensor_desc(ctypes.Structure):
    _fields_ = [("theta", ctypes.c_void_p), ("comp", ctypes.c_void_p), ("numel", ctypes.c_int64),
                ("theta_bits", ctypes.c_int32), ("comp_bits", ctypes.c_int32),
                ("overlap_k", ctypes.c_int32), ("exp_theta", ctypes.c_int32),
                ("exp_theta_next", ctypes.c_int32)]


class ksgd_momentum_desc(ctypes.Structure):
    _fields_ = [("mom", ctypes.c_void_p), ("mom_bits", ctypes.c_int32), ("exp_mom", ctypes.c_int32),
                ("exp_mom_next", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class ksgd_adam_desc(ctypes.Structure):
    _fields_ = [("mom1", ctypes.c_void_p), ("mom2", ctypes.c_void_p), ("exp_m", ctypes.c_int32),
                ("exp_m_next", ctypes.c_int32), ("exp_v", ctypes.c_int32), ("exp_v_next", ctypes.c_int32)]


_ADAM_STATS_FIELDS = ("amax_theta", "amax_comp", "amax_m", "amax_v", "exp_theta_cur", "exp_theta_next",
                      "exp_m_cur", "exp_m_next", "exp_v_cur", "exp_v_next", "n_sat_theta", "n_sat_comp",
                      "n_sat_m", "n_sat_v", "n_nonfinite")


class ksgd_adam_stats(ctypes.Structure):
    _fields_ = [(name, ctypes.c_void_p) for name in _ADAM_STATS_FIELDS]


class KahanSgdError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"kahan_sgd error {code}: {text}")
        self.code = code


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIBRARY):
        raise ImportError(
            f"{LIBRARY} is missing: build it with `python -m paper_1810_05486_b200.build` "
            "(nvcc, sm_100a).  There is no CPU fallback.")
    lib = ctypes.CDLL(LIBRARY)
    P = ctypes.POINTER
    lib.kahan_sgd_workspace_bytes.restype = ctypes.c_size_t
    lib.kahan_sgd_workspace_bytes.argtypes = [P(ksgd_tensor_desc), ctypes.c_int32]
    lib.kahan_sgd_workspace_error_offset.restype = ctypes.c_size_t
    lib.kahan_sgd_workspace_error_offset.argtypes = [P(ksgd_tensor_desc), ctypes.c_int32]
    lib.kahan_sgd_tile_table.restype = ctypes.c_int64
    lib.kahan_sgd_tile_table.argtypes = [P(ksgd_tensor_desc), ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                         P(ctypes.c_int64), ctypes.c_int64]
    lib.kahan_sgd_init.restype = ctypes.c_int
    lib.kahan_sgd_init.argtypes = [P(ctypes.c_void_p), P(ksgd_tensor_desc), ctypes.c_int32,
                                   ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
    lib.kahan_sgd_step.restype = ctypes.c_int
    lib.kahan_sgd_step.argtypes = [ctypes.c_void_p, P(ctypes.c_void_p), P(ctypes.c_float)]
    lib.kahan_sgd_step_qgrad.restype = ctypes.c_int
    lib.kahan_sgd_step_qgrad.argtypes = [ctypes.c_void_p, P(ctypes.c_void_p), ctypes.c_int32,
                                         P(ctypes.c_int32), P(ctypes.c_float)]
    lib.kahan_sgd_strict_workspace_bytes.restype = ctypes.c_size_t
    lib.kahan_sgd_strict_workspace_bytes.argtypes = [P(ksgd_tensor_desc), P(ctypes.c_int32), ctypes.c_int32]
    lib.kahan_sgd_strict_init.restype = ctypes.c_int
    lib.kahan_sgd_strict_init.argtypes = [P(ctypes.c_void_p), P(ksgd_tensor_desc), P(ctypes.c_int32),
                                          P(ctypes.c_int32), ctypes.c_int32, ctypes.c_int, ctypes.c_void_p,
                                          ctypes.c_size_t, ctypes.c_void_p]
    lib.kahan_sgd_strict_exponents.restype = ctypes.c_int
    lib.kahan_sgd_strict_exponents.argtypes = [ctypes.c_void_p, P(ctypes.c_int32), P(ctypes.c_int32)]
    lib.kahan_sgd_step_host.restype = ctypes.c_int
    lib.kahan_sgd_step_host.argtypes = [ctypes.c_void_p, P(ctypes.c_void_p), P(ctypes.c_void_p),
                                        P(ctypes.c_void_p), P(ctypes.c_float), ctypes.c_void_p,
                                        ctypes.c_size_t]
    lib.kahan_sgd_amax.restype = ctypes.c_int
    lib.kahan_sgd_amax.argtypes = [ctypes.c_void_p] + [ctypes.c_void_p] * 7
    lib.kahan_sgd_set_exponents.restype = ctypes.c_int
    lib.kahan_sgd_set_exponents.argtypes = [ctypes.c_void_p, P(ctypes.c_int32)]
    lib.kahan_sgd_step_static.restype = ctypes.c_int
    lib.kahan_sgd_step_static.argtypes = [P(ksgd_tensor_desc), ctypes.c_int32, ctypes.c_int,
                                          P(ctypes.c_void_p), P(ctypes.c_float)] + \
        [ctypes.c_void_p] * 7 + [ctypes.c_void_p]
    lib.kahan_sgd_momentum_workspace_bytes.restype = ctypes.c_size_t
    lib.kahan_sgd_momentum_workspace_bytes.argtypes = [P(ksgd_tensor_desc), P(ksgd_momentum_desc),
                                                       ctypes.c_int32]
    lib.kahan_sgd_momentum_init.restype = ctypes.c_int
    lib.kahan_sgd_momentum_init.argtypes = [P(ctypes.c_void_p), P(ksgd_tensor_desc), P(ksgd_momentum_desc),
                                            ctypes.c_int32, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t,
                                            ctypes.c_void_p]
    lib.kahan_sgd_momentum_step.restype = ctypes.c_int
    lib.kahan_sgd_momentum_step.argtypes = [ctypes.c_void_p, P(ctypes.c_void_p), P(ctypes.c_float),
                                            P(ctypes.c_float)]
    lib.kahan_sgd_momentum_amax.restype = ctypes.c_int
    lib.kahan_sgd_momentum_amax.argtypes = [ctypes.c_void_p] + [ctypes.c_void_p] * 11
    lib.kahan_sgd_momentum_destroy.restype = ctypes.c_int
    lib.kahan_sgd_momentum_destroy.argtypes = [ctypes.c_void_p]
    lib.kahan_sgd_adam_workspace_bytes.restype = ctypes.c_size_t
    lib.kahan_sgd_adam_workspace_bytes.argtypes = [P(ksgd_tensor_desc), P(ksgd_adam_desc), ctypes.c_int32]
    lib.kahan_sgd_adam_init.restype = ctypes.c_int
    lib.kahan_sgd_adam_init.argtypes = [P(ctypes.c_void_p), P(ksgd_tensor_desc), P(ksgd_adam_desc),
                                        ctypes.c_int32, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t,
                                        ctypes.c_void_p]
    lib.kahan_sgd_adam_step.restype = ctypes.c_int
    lib.kahan_sgd_adam_step.argtypes = [ctypes.c_void_p, P(ctypes.c_void_p), P(ctypes.c_float),
                                        ctypes.c_float, ctypes.c_float, ctypes.c_float]
    lib.kahan_sgd_adam_amax.restype = ctypes.c_int
    lib.kahan_sgd_adam_amax.argtypes = [ctypes.c_void_p, P(ksgd_adam_stats)]
    lib.kahan_sgd_adam_destroy.restype = ctypes.c_int
    lib.kahan_sgd_adam_destroy.argtypes = [ctypes.c_void_p]
    lib.kahan_sgd_adam_selfcheck.restype = ctypes.c_int
    lib.kahan_sgd_adam_selfcheck.argtypes = [P(ctypes.c_uint64), P(ctypes.c_uint64), ctypes.c_void_p]
    lib.kahan_sgd_step_qgrad_dev.restype = ctypes.c_int
    lib.kahan_sgd_step_qgrad_dev.argtypes = [ctypes.c_void_p, P(ctypes.c_void_p), ctypes.c_int32,
                                             ctypes.c_void_p, P(ctypes.c_float)]
    lib.kahan_sgd_import_dev.restype = ctypes.c_int
    lib.kahan_sgd_import_dev.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int64] + [ctypes.c_int32] * 3 + \
        [ctypes.c_void_p] * 3
    lib.kahan_sgd_import.restype = ctypes.c_int
    lib.kahan_sgd_import.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int64] + [ctypes.c_int32] * 4 + \
        [P(ctypes.c_int32), ctypes.c_void_p, ctypes.c_void_p]
    lib.kahan_sgd_export.restype = ctypes.c_int
    lib.kahan_sgd_export.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int64] + [ctypes.c_int32] * 4 + \
        [ctypes.c_void_p]
    lib.kahan_sgd_classifier_bits.restype = ctypes.c_int32
    lib.kahan_sgd_classifier_bits.argtypes = [ctypes.c_int64, ctypes.c_double]
    lib.kahan_sgd_destroy.restype = ctypes.c_int
    lib.kahan_sgd_destroy.argtypes = [ctypes.c_void_p]
    lib.kahan_sgd_strerror.restype = ctypes.c_char_p
    lib.kahan_sgd_strerror.argtypes = [ctypes.c_int]
    lib.kahan_sgd_last_cuda_error.restype = ctypes.c_char_p
    lib.kahan_sgd_last_cuda_error.argtypes = []
    lib.kahan_sgd_launch_count.restype = ctypes.c_uint64
    lib.kahan_sgd_launch_count.argtypes = []
    return lib


lib = _load()


def _check(code: int) -> None:
    if code != KSGD_OK:
        text = lib.kahan_sgd_strerror(code).decode()
        if code == KSGD_ERR_CUDA:
            text += ": " + lib.kahan_sgd_last_cuda_error().decode()
        raise KahanSgdError(code, text)


def make_descs(tensors: Sequence[dict]):
    """ctypes array of ksgd_tensor_desc from dicts with the struct's field names
    (theta / comp are integer device addresses; comp None or 0 when comp_bits == 0)."""
    arr = (ksgd_tensor_desc * len(tensors))()
    for d, t in zip(arr, tensors):
        d.theta = t["theta"]
        d.comp = t.get("comp") or None
        d.numel = t["numel"]
        d.theta_bits = t["theta_bits"]
        d.comp_bits = t["comp_bits"]
        d.overlap_k = t.get("overlap_k", 0)
        d.exp_theta = t["exp_theta"]
        d.exp_theta_next = t.get("exp_theta_next", t["exp_theta"])
    return arr


def kahan_sgd_workspace_bytes(descs) -> int:
    return int(lib.kahan_sgd_workspace_bytes(descs, len(descs)))


def kahan_sgd_workspace_error_offset(descs) -> int:
    """Byte offset of the sticky device-error word inside this list's workspace."""
    off = int(lib.kahan_sgd_workspace_error_offset(descs, len(descs)))
    if off == ctypes.c_size_t(-1).value:
        raise KahanSgdError(KSGD_ERR_NUMEL, "invalid tensor list")
    return off


def kahan_sgd_tile_table(descs, sms: int, which: int = 0):
    """The tile table of this list on a device with `sms` multiprocessors, as a list of
    (tensor, first element, number of elements); which = 1: the table of steps on 8-bit gradients."""
    n = int(lib.kahan_sgd_tile_table(descs, len(descs), sms, which, None, 0))
    if n < 0:
        _check(n)
    out = (ctypes.c_int64 * (3 * max(n, 1)))()
    _check(min(0, int(lib.kahan_sgd_tile_table(descs, len(descs), sms, which, out, n))))
    return [(int(out[3 * i]), int(out[3 * i + 1]), int(out[3 * i + 2])) for i in range(n)]


def kahan_sgd_init(descs, mode: int, workspace: int, workspace_bytes: int, stream: int = 0):
    """Returns the opaque handle (a ctypes.c_void_p)."""
    h = ctypes.c_void_p()
    _check(lib.kahan_sgd_init(ctypes.byref(h), descs, len(descs), mode,
                              ctypes.c_void_p(workspace), workspace_bytes,
                              ctypes.c_void_p(stream)))
    return h


def _ptr_array(addresses: Sequence[Optional[int]]):
    return (ctypes.c_void_p * len(addresses))(*[a or None for a in addresses])


def _float_array(values: Sequence[float]):
    return (ctypes.c_float * len(values))(*values)


def kahan_sgd_step(h, grads, lrs) -> None:
    """grads: device addresses (or a prebuilt ctypes pointer array); lrs: floats (or a
    prebuilt ctypes float array)."""
    g = grads if isinstance(grads, ctypes.Array) else _ptr_array(grads)
    l = lrs if isinstance(lrs, ctypes.Array) else _float_array(lrs)
    _check(lib.kahan_sgd_step(h, g, l))


def _int_array(values):
    return (ctypes.c_int32 * len(values))(*[int(v) for v in values])


def kahan_sgd_strict_workspace_bytes(descs, exp_comp) -> int:
    return int(lib.kahan_sgd_strict_workspace_bytes(descs, _int_array(exp_comp), len(descs)))


def kahan_sgd_strict_init(descs, exp_comp, exp_comp_next, mode: int, workspace: int, workspace_bytes: int,
                          stream: int = 0):
    """Strict Algorithm 1: exp_comp / exp_comp_next are the compensation's own exponents."""
    h = ctypes.c_void_p()
    nxt = _int_array(exp_comp_next) if exp_comp_next is not None else None
    _check(lib.kahan_sgd_strict_init(ctypes.byref(h), descs, _int_array(exp_comp), nxt, len(descs), mode,
                                     ctypes.c_void_p(workspace), workspace_bytes, ctypes.c_void_p(stream)))
    return h


def kahan_sgd_strict_exponents(h, n_tensors: int) -> dict:
    cur, nxt = (ctypes.c_int32 * n_tensors)(), (ctypes.c_int32 * n_tensors)()
    _check(lib.kahan_sgd_strict_exponents(h, cur, nxt))
    return {"exp_comp_cur": list(cur), "exp_comp_next": list(nxt)}


def kahan_sgd_step_qgrad(h, grads, grad_bits: int, exp_grad, lrs) -> None:
    """grads: device addresses of int8 / int16 gradient mantissas; exp_grad: their exponents."""
    g = grads if isinstance(grads, ctypes.Array) else _ptr_array(grads)
    e = exp_grad if isinstance(exp_grad, ctypes.Array) else (ctypes.c_int32 * len(exp_grad))(*exp_grad)
    l = lrs if isinstance(lrs, ctypes.Array) else _float_array(lrs)
    _check(lib.kahan_sgd_step_qgrad(h, g, grad_bits, e, l))


def kahan_sgd_step_qgrad_dev(h, grads, grad_bits: int, exp_grad_dev: int, lrs) -> None:
    """As kahan_sgd_step_qgrad, the exponents in a device int32 array (address exp_grad_dev)."""
    g = grads if isinstance(grads, ctypes.Array) else _ptr_array(grads)
    l = lrs if isinstance(lrs, ctypes.Array) else _float_array(lrs)
    _check(lib.kahan_sgd_step_qgrad_dev(h, g, grad_bits, ctypes.c_void_p(exp_grad_dev), l))


def kahan_sgd_step_host(h, theta_host, comp_host, grads_host, lrs, grad_staging: int,
                        grad_staging_bytes: int) -> None:
    """theta_host / comp_host / grads_host: host addresses per tensor."""
    th = theta_host if isinstance(theta_host, ctypes.Array) else _ptr_array(theta_host)
    ch = comp_host if isinstance(comp_host, ctypes.Array) else _ptr_array(comp_host)
    gh = grads_host if isinstance(grads_host, ctypes.Array) else _ptr_array(grads_host)
    l = lrs if isinstance(lrs, ctypes.Array) else _float_array(lrs)
    _check(lib.kahan_sgd_step_host(h, th, ch, gh, l, ctypes.c_void_p(grad_staging),
                                   grad_staging_bytes))


def kahan_sgd_amax(h, n_tensors: int) -> dict:
    """Per-tensor results of the most recent step as lists (synchronises the stream)."""
    a_t = (ctypes.c_uint32 * n_tensors)()
    a_c = (ctypes.c_uint32 * n_tensors)()
    e_c = (ctypes.c_int32 * n_tensors)()
    e_n = (ctypes.c_int32 * n_tensors)()
    s_t = (ctypes.c_uint64 * n_tensors)()
    s_c = (ctypes.c_uint64 * n_tensors)()
    nf = (ctypes.c_uint64 * n_tensors)()
    _check(lib.kahan_sgd_amax(h, a_t, a_c, e_c, e_n, s_t, s_c, nf))
    return {"amax_theta": list(a_t), "amax_comp": list(a_c), "exp_theta_cur": list(e_c),
            "exp_theta_next": list(e_n), "n_sat_theta": list(s_t), "n_sat_comp": list(s_c),
            "n_nonfinite": list(nf)}


def kahan_sgd_set_exponents(h, exp_theta_next: Sequence[int]) -> None:
    arr = (ctypes.c_int32 * len(exp_theta_next))(*exp_theta_next)
    _check(lib.kahan_sgd_set_exponents(h, arr))


KSGD_STATIC_SCRATCH_BYTES = 192 * 1024
KSGD_STATIC_MAX_TENSORS = 256


def kahan_sgd_step_static(descs, mode: int, grads, lrs, stream: int = 0) -> dict:
    """One self-contained step that allocates no device memory (scratch inside the library).

    For callers that cannot obtain a device workspace when they need one.  Returns the same
    dictionary as kahan_sgd_amax (counters: this call only); put exp_theta_cur and
    exp_theta_next back into the descs for the next call.  Calls must not overlap on the GPU.
    """
    n = len(descs)
    g = grads if isinstance(grads, ctypes.Array) else _ptr_array(grads)
    l = lrs if isinstance(lrs, ctypes.Array) else _float_array(lrs)
    a_t = (ctypes.c_uint32 * n)()
    a_c = (ctypes.c_uint32 * n)()
    e_c = (ctypes.c_int32 * n)()
    e_n = (ctypes.c_int32 * n)()
    s_t = (ctypes.c_uint64 * n)()
    s_c = (ctypes.c_uint64 * n)()
    nf = (ctypes.c_uint64 * n)()
    _check(lib.kahan_sgd_step_static(descs, n, mode, g, l, a_t, a_c, e_c, e_n, s_t, s_c, nf,
                                     ctypes.c_void_p(stream)))
    return {"amax_theta": list(a_t), "amax_comp": list(a_c), "exp_theta_cur": list(e_c),
            "exp_theta_next": list(e_n), "n_sat_theta": list(s_t), "n_sat_comp": list(s_c),
            "n_nonfinite": list(nf)}


def kahan_sgd_destroy(h) -> None:
    _check(lib.kahan_sgd_destroy(h))


def make_momentum_descs(tensors: Sequence[dict]):
    """ctypes array of ksgd_momentum_desc from dicts with keys mom, mom_bits, exp_mom
    (and optionally exp_mom_next)."""
    arr = (ksgd_momentum_desc * len(tensors))()
    for d, t in zip(arr, tensors):
        d.mom = t["mom"]
        d.mom_bits = t["mom_bits"]
        d.exp_mom = t["exp_mom"]
        d.exp_mom_next = t.get("exp_mom_next", t["exp_mom"])
        d.reserved = 0
    return arr


def kahan_sgd_momentum_workspace_bytes(descs, mdescs) -> int:
    return int(lib.kahan_sgd_momentum_workspace_bytes(descs, mdescs, len(descs)))


def kahan_sgd_momentum_init(descs, mdescs, mode: int, workspace: int, workspace_bytes: int,
                            stream: int = 0):
    h = ctypes.c_void_p()
    _check(lib.kahan_sgd_momentum_init(ctypes.byref(h), descs, mdescs, len(descs), mode,
                                       ctypes.c_void_p(workspace), workspace_bytes,
                                       ctypes.c_void_p(stream)))
    return h


def kahan_sgd_momentum_step(h, grads, lrs, mus) -> None:
    g = grads if isinstance(grads, ctypes.Array) else _ptr_array(grads)
    l = lrs if isinstance(lrs, ctypes.Array) else _float_array(lrs)
    m = mus if isinstance(mus, ctypes.Array) else _float_array(mus)
    _check(lib.kahan_sgd_momentum_step(h, g, l, m))


def kahan_sgd_momentum_amax(h, n_tensors: int) -> dict:
    u32 = lambda: (ctypes.c_uint32 * n_tensors)()   # noqa: E731
    i32 = lambda: (ctypes.c_int32 * n_tensors)()    # noqa: E731
    u64 = lambda: (ctypes.c_uint64 * n_tensors)()   # noqa: E731
    a_t, a_c, a_v, e_c, e_n, ev_c, ev_n = u32(), u32(), u32(), i32(), i32(), i32(), i32()
    s_t, s_c, s_v, nf = u64(), u64(), u64(), u64()
    _check(lib.kahan_sgd_momentum_amax(h, a_t, a_c, a_v, e_c, e_n, ev_c, ev_n, s_t, s_c, s_v, nf))
    return {"amax_theta": list(a_t), "amax_comp": list(a_c), "amax_mom": list(a_v),
            "exp_theta_cur": list(e_c), "exp_theta_next": list(e_n), "exp_mom_cur": list(ev_c),
            "exp_mom_next": list(ev_n), "n_sat_theta": list(s_t), "n_sat_comp": list(s_c),
            "n_sat_mom": list(s_v), "n_nonfinite": list(nf)}


def kahan_sgd_momentum_destroy(h) -> None:
    _check(lib.kahan_sgd_momentum_destroy(h))


def make_adam_descs(tensors: Sequence[dict]):
    """ctypes array of ksgd_adam_desc from dicts with keys mom1, mom2, exp_m, exp_v (and
    optionally exp_m_next, exp_v_next)."""
    arr = (ksgd_adam_desc * len(tensors))()
    for d, t in zip(arr, tensors):
        d.mom1, d.mom2 = t["mom1"], t["mom2"]
        d.exp_m, d.exp_m_next = t["exp_m"], t.get("exp_m_next", t["exp_m"])
        d.exp_v, d.exp_v_next = t["exp_v"], t.get("exp_v_next", t["exp_v"])
    return arr


def kahan_sgd_adam_workspace_bytes(descs, adescs) -> int:
    return int(lib.kahan_sgd_adam_workspace_bytes(descs, adescs, len(descs)))


def kahan_sgd_adam_init(descs, adescs, mode: int, workspace: int, workspace_bytes: int, stream: int = 0):
    h = ctypes.c_void_p()
    _check(lib.kahan_sgd_adam_init(ctypes.byref(h), descs, adescs, len(descs), mode,
                                   ctypes.c_void_p(workspace), workspace_bytes, ctypes.c_void_p(stream)))
    return h


def kahan_sgd_adam_step(h, grads, lrs, beta1: float, beta2: float, eps: float) -> None:
    g = grads if isinstance(grads, ctypes.Array) else _ptr_array(grads)
    l = lrs if isinstance(lrs, ctypes.Array) else _float_array(lrs)
    _check(lib.kahan_sgd_adam_step(h, g, l, beta1, beta2, eps))


def kahan_sgd_adam_amax(h, n_tensors: int) -> dict:
    arrays = {}
    st = ksgd_adam_stats()
    for name in _ADAM_STATS_FIELDS:
        ctype = ctypes.c_uint32 if name.startswith("amax") else (
            ctypes.c_int32 if name.startswith("exp") else ctypes.c_uint64)
        arrays[name] = (ctype * n_tensors)()
        setattr(st, name, ctypes.addressof(arrays[name]))
    _check(lib.kahan_sgd_adam_amax(h, ctypes.byref(st)))
    return {name: list(a) for name, a in arrays.items()}


def kahan_sgd_adam_destroy(h) -> None:
    _check(lib.kahan_sgd_adam_destroy(h))


def kahan_sgd_adam_selfcheck(stream: int = 0):
    """(division mismatches, square-root mismatches) of the fast path's sequences."""
    d, q = ctypes.c_uint64(), ctypes.c_uint64()
    _check(lib.kahan_sgd_adam_selfcheck(ctypes.byref(d), ctypes.byref(q), ctypes.c_void_p(stream)))
    return int(d.value), int(q.value)


KSGD_EXP_AUTO = -(2 ** 31)


def kahan_sgd_import(src: int, theta: int, comp, numel: int, theta_bits: int, comp_bits: int,
                     overlap_k: int = 0, exp_theta: int = KSGD_EXP_AUTO, scratch: int = 0,
                     stream: int = 0) -> int:
    """fp32 -> dynamic fixed-point on the device; returns the exponent used."""
    e = ctypes.c_int32()
    _check(lib.kahan_sgd_import(ctypes.c_void_p(src), ctypes.c_void_p(theta), ctypes.c_void_p(comp or None),
                                numel, theta_bits, comp_bits, overlap_k, exp_theta, ctypes.byref(e),
                                ctypes.c_void_p(scratch or None), ctypes.c_void_p(stream)))
    return int(e.value)


def kahan_sgd_import_dev(src: int, theta: int, comp, numel: int, theta_bits: int, comp_bits: int,
                         overlap_k: int, exp_theta_dev: int, scratch: int, stream: int = 0) -> None:
    """fp32 -> dynamic fixed-point without a host round trip: max scan, exponent chosen on the
    device and left in the device int32 at exp_theta_dev, quantization.  Enqueues only."""
    _check(lib.kahan_sgd_import_dev(ctypes.c_void_p(src), ctypes.c_void_p(theta), ctypes.c_void_p(comp or None),
                                    numel, theta_bits, comp_bits, overlap_k, ctypes.c_void_p(exp_theta_dev),
                                    ctypes.c_void_p(scratch), ctypes.c_void_p(stream)))


def kahan_sgd_export(theta: int, comp, dst: int, numel: int, theta_bits: int, comp_bits: int,
                     overlap_k: int, exp_theta: int, stream: int = 0) -> None:
    """Dynamic fixed-point -> fp32 on the device (theta + c rounded once)."""
    _check(lib.kahan_sgd_export(ctypes.c_void_p(theta), ctypes.c_void_p(comp or None), ctypes.c_void_p(dst),
                                numel, theta_bits, comp_bits, overlap_k, exp_theta, ctypes.c_void_p(stream)))


def kahan_sgd_classifier_bits(n_classes: int, alpha: float = 0.5) -> int:
    """Eq. 5: smallest bit-width larger than log2(n_classes - 1) + log2(2 / alpha)."""
    return int(lib.kahan_sgd_classifier_bits(n_classes, alpha))


def kahan_sgd_strerror(code: int) -> str:
    return lib.kahan_sgd_strerror(code).decode()


def kahan_sgd_launch_count() -> int:
    return int(lib.kahan_sgd_launch_count())
