"""Device-side set-up of a synthetic workload: host buffers, device buffers, descriptors,
handle.  Used by the benchmark and by the full-size parity tests so that both drive the
library in exactly the same launch configuration.  PyTorch supplies memory and streams
only; every step of the update runs in the CUDA library."""
import ctypes
from typing import List, Optional

import numpy as np

from . import binding as B
from . import workloads as W


def _carve(wl, itemsize_of):
    offs, off = [], 0
    for t in wl.tensors:
        offs.append(off)
        off += (t.numel * itemsize_of(t) + 15) // 16 * 16
    return offs, off


class HostInputs:
    """Host copies of theta, comp and n_sets gradient sets.  Each kind lives in one
    (optionally page-locked) buffer with every tensor at a 16-byte aligned offset."""

    def __init__(self, wl, seed: int = 0, n_sets: int = 1, pinned: bool = True,
                 threads: Optional[int] = None):
        import torch
        self.wl = wl
        self.th_offs, th_bytes = _carve(wl, lambda t: t.theta_bits // 8)
        self.c_offs, c_bytes = _carve(wl, lambda t: max(t.comp_bits, 8) // 8)
        self.g_offs, g_bytes = _carve(wl, lambda t: 4)
        alloc = lambda n: torch.zeros(n, dtype=torch.uint8, pin_memory=pinned)  # noqa: E731
        self.th_buf, self.c_buf = alloc(th_bytes), alloc(c_bytes)
        self.g_bufs = [alloc(g_bytes) for _ in range(n_sets)]
        self.thetas = self._views(self.th_buf, self.th_offs,
                                  lambda t: W.storage_dtype(t.theta_bits))
        self.comps = self._views(self.c_buf, self.c_offs,
                                 lambda t: W.storage_dtype(max(t.comp_bits, 8)))
        W.fill_theta(wl, self.thetas, seed, threads)
        self.grads: List[List[np.ndarray]] = []
        for k, gb in enumerate(self.g_bufs):
            gv = self._views(gb, self.g_offs, lambda t: np.float32)
            W.fill_grads(wl, k, gv, seed, threads)
            self.grads.append(gv)

    def _views(self, buf, offs, dtype_of):
        base = buf.numpy()
        return [base[o:o + t.numel * np.dtype(dtype_of(t)).itemsize].view(dtype_of(t))
                for o, t in zip(offs, self.wl.tensors)]


class DeviceRun:
    """Device buffers (same layout as HostInputs), descriptors, workspace and handle."""

    def __init__(self, host: HostInputs, mode: int = B.KSGD_EXP_AMAX, stream=None,
                 mom_bits: int = 0, mu: float = 0.9, adam: Optional[dict] = None, grad_bits: int = 32,
                 strict: bool = False):
        """mom_bits = 8 or 16 selects the momentum optimizer (velocity buffers start at zero,
        on a grid 8 binades below theta's).  adam = dict(beta1, beta2, eps, eta) selects ADAM
        (both 16-bit moments start at zero, on grids that just hold what the first step makes of
        the largest gradient of the first set; the step size carries the bias correction of the
        step count).  grad_bits = 8 or 16 (plain optimizer only): every resident gradient set is
        turned into fixed-point tensors of that width on the device (exponent from the tensor's
        maximum) and the steps read those.  strict (plain optimizer only): strict Algorithm 1, the
        compensation starting on the grid the ordinary mode ties it to."""
        import torch
        self.torch = torch
        self.host = host
        wl = self.wl = host.wl
        self.n = len(wl.tensors)
        self.dev_th = host.th_buf.cuda(non_blocking=True)
        self.dev_c = host.c_buf.cuda(non_blocking=True)
        self.dev_g = [g.cuda(non_blocking=True) for g in host.g_bufs]
        torch.cuda.synchronize()
        self.descs = B.make_descs([
            dict(theta=self.dev_th.data_ptr() + host.th_offs[i],
                 comp=(self.dev_c.data_ptr() + host.c_offs[i]) if t.comp_bits else None,
                 numel=t.numel, theta_bits=t.theta_bits, comp_bits=t.comp_bits,
                 overlap_k=t.overlap_k, exp_theta=t.exp_theta)
            for i, t in enumerate(wl.tensors)])
        self.stream = stream if stream is not None else torch.cuda.Stream()
        self.mom_bits = mom_bits
        self.adam = adam
        self.t = 0
        if adam:
            assert not mom_bits
            self.m_offs, m_bytes = _carve(wl, lambda t: 2)
            self.dev_m1 = torch.zeros(m_bytes, dtype=torch.uint8, device="cuda")
            self.dev_m2 = torch.zeros(m_bytes, dtype=torch.uint8, device="cuda")
            adescs = []
            for i, g in enumerate(host.grads[0]):
                gmax = max(float(np.abs(g[:1 << 20]).max()), 1e-30)
                e_m = int(np.clip(np.ceil(np.log2((1.0 - adam["beta1"] + 1e-9) * gmax / 32767.0)), -64, 64))
                e_v = int(np.clip(np.ceil(np.log2((1.0 - adam["beta2"] + 1e-9) * gmax * gmax / 32767.0)),
                                  -64, 64))
                adescs.append(dict(mom1=self.dev_m1.data_ptr() + self.m_offs[i],
                                   mom2=self.dev_m2.data_ptr() + self.m_offs[i], exp_m=e_m, exp_v=e_v))
            self.adescs = B.make_adam_descs(adescs)
            self.ws_bytes = B.kahan_sgd_adam_workspace_bytes(self.descs, self.adescs)
            self.workspace = torch.zeros(self.ws_bytes, dtype=torch.uint8, device="cuda")
            torch.cuda.synchronize()     # the fills above ran on torch's stream, the library works on self.stream
            self.handle = B.kahan_sgd_adam_init(self.descs, self.adescs, mode, self.workspace.data_ptr(),
                                                self.ws_bytes, self.stream.cuda_stream)
        elif mom_bits:
            self.v_offs, v_bytes = _carve(wl, lambda t: mom_bits // 8)
            self.dev_v = torch.zeros(v_bytes, dtype=torch.uint8, device="cuda")
            self.mdescs = B.make_momentum_descs([
                dict(mom=self.dev_v.data_ptr() + self.v_offs[i], mom_bits=mom_bits,
                     exp_mom=t.exp_theta - 8) for i, t in enumerate(wl.tensors)])
            self.ws_bytes = B.kahan_sgd_momentum_workspace_bytes(self.descs, self.mdescs)
            self.workspace = torch.zeros(self.ws_bytes, dtype=torch.uint8, device="cuda")
            torch.cuda.synchronize()     # the fills above ran on torch's stream, the library works on self.stream
            self.handle = B.kahan_sgd_momentum_init(self.descs, self.mdescs, mode,
                                                    self.workspace.data_ptr(), self.ws_bytes,
                                                    self.stream.cuda_stream)
            self.mus = (ctypes.c_float * self.n)(*([mu] * self.n))
        elif strict:
            ec = [t.exp_theta - (t.comp_bits - 1 - t.overlap_k) for t in wl.tensors]
            self.ws_bytes = B.kahan_sgd_strict_workspace_bytes(self.descs, ec)
            self.workspace = torch.zeros(self.ws_bytes, dtype=torch.uint8, device="cuda")
            torch.cuda.synchronize()     # the fills above ran on torch's stream, the library works on self.stream
            self.handle = B.kahan_sgd_strict_init(self.descs, ec, None, mode, self.workspace.data_ptr(),
                                                  self.ws_bytes, self.stream.cuda_stream)
        else:
            self.ws_bytes = B.kahan_sgd_workspace_bytes(self.descs)
            self.workspace = torch.zeros(self.ws_bytes, dtype=torch.uint8, device="cuda")
            torch.cuda.synchronize()     # the fills above ran on torch's stream, the library works on self.stream
            self.handle = B.kahan_sgd_init(self.descs, mode, self.workspace.data_ptr(),
                                           self.ws_bytes, self.stream.cuda_stream)
        self.strict = strict
        self.grad_ptr_sets = [(ctypes.c_void_p * self.n)(*[g.data_ptr() + o for o in host.g_offs])
                              for g in self.dev_g]
        self.grad_bits = grad_bits
        if grad_bits != 32:
            assert grad_bits in (8, 16) and not mom_bits and not adam
            self.q_offs, q_bytes = _carve(wl, lambda t: grad_bits // 8)
            scratch = torch.zeros(64, dtype=torch.uint8, device="cuda")
            self.dev_gq, self.gq_ptr_sets, self.gq_exp_sets = [], [], []
            for gset in self.dev_g:
                q = torch.zeros(q_bytes, dtype=torch.uint8, device="cuda")
                torch.cuda.synchronize()     # the fill must not overtake the import kernels on self.stream
                exps = [B.kahan_sgd_import(gset.data_ptr() + host.g_offs[i], q.data_ptr() + self.q_offs[i], None,
                                           t.numel, grad_bits, 0, 0, B.KSGD_EXP_AUTO, scratch.data_ptr(),
                                           self.stream.cuda_stream) for i, t in enumerate(wl.tensors)]
                self.dev_gq.append(q)
                self.gq_ptr_sets.append((ctypes.c_void_p * self.n)(*[q.data_ptr() + o for o in self.q_offs]))
                self.gq_exp_sets.append((ctypes.c_int32 * self.n)(*exps))
            self.dev_g = self.dev_g[:1]            # the binary32 copies are no longer needed ...
            self.grad_ptr_sets = self.grad_ptr_sets[:1]   # ... and their addresses must not outlive them
            torch.cuda.empty_cache()
        self.lrs = (ctypes.c_float * self.n)(*([wl.lr] * self.n))

    def adam_lrs(self, t: int):
        """Step sizes of ADAM step t (1-based): eta * sqrt(1 - beta2^t) / (1 - beta1^t)."""
        a = self.adam
        c1 = 1.0 - a["beta1"] ** t if a["beta1"] < 1.0 else 1.0
        c2 = 1.0 - a["beta2"] ** t if a["beta2"] < 1.0 else 1.0
        lr = float(np.float32(a["eta"] * np.sqrt(c2) / c1))
        return (ctypes.c_float * self.n)(*([lr] * self.n))

    def step(self, grad_set: int) -> None:
        if self.adam:
            self.t += 1
            B.kahan_sgd_adam_step(self.handle, self.grad_ptr_sets[grad_set], self.adam_lrs(self.t),
                                  self.adam["beta1"], self.adam["beta2"], self.adam["eps"])
        elif self.mom_bits:
            B.kahan_sgd_momentum_step(self.handle, self.grad_ptr_sets[grad_set], self.lrs, self.mus)
        elif self.grad_bits != 32:
            B.kahan_sgd_step_qgrad(self.handle, self.gq_ptr_sets[grad_set], self.grad_bits,
                                   self.gq_exp_sets[grad_set], self.lrs)
        else:
            B.kahan_sgd_step(self.handle, self.grad_ptr_sets[grad_set], self.lrs)

    def stats(self) -> dict:
        if self.adam:
            return B.kahan_sgd_adam_amax(self.handle, self.n)
        if self.mom_bits:
            return B.kahan_sgd_momentum_amax(self.handle, self.n)
        return B.kahan_sgd_amax(self.handle, self.n)

    @property
    def bytes_per_step(self) -> int:
        """Algorithmic HBM bytes of one step, velocity or moments included."""
        if self.adam:
            return self.wl.bytes_per_step + 8 * self.wl.numel
        if self.grad_bits != 32:
            return self.wl.bytes_per_step - (4 - self.grad_bits // 8) * self.wl.numel
        return self.wl.bytes_per_step + 2 * (self.mom_bits // 8) * self.wl.numel

    def theta(self, i: int) -> np.ndarray:
        t = self.wl.tensors[i]
        nb = t.numel * (t.theta_bits // 8)
        o = self.host.th_offs[i]
        return self.dev_th[o:o + nb].cpu().numpy().view(W.storage_dtype(t.theta_bits))

    def comp(self, i: int) -> np.ndarray:
        t = self.wl.tensors[i]
        nb = t.numel * (t.comp_bits // 8)
        o = self.host.c_offs[i]
        return self.dev_c[o:o + nb].cpu().numpy().view(W.storage_dtype(t.comp_bits))

    def velocity(self, i: int) -> np.ndarray:
        """Momentum mode: the velocity mantissas of tensor i."""
        nb = self.wl.tensors[i].numel * (self.mom_bits // 8)
        o = self.v_offs[i]
        return self.dev_v[o:o + nb].cpu().numpy().view(W.storage_dtype(self.mom_bits))

    def moments(self, i: int):
        """ADAM mode: (first, second) moment mantissas of tensor i."""
        nb = self.wl.tensors[i].numel * 2
        o = self.m_offs[i]
        return (self.dev_m1[o:o + nb].cpu().numpy().view(np.int16),
                self.dev_m2[o:o + nb].cpu().numpy().view(np.int16))

    def host_pointer_arrays(self):
        """ctypes arrays of host addresses for kahan_sgd_step_host."""
        n = self.n
        th = (ctypes.c_void_p * n)(*[a.ctypes.data for a in self.host.thetas])
        c = (ctypes.c_void_p * n)(*[a.ctypes.data for a in self.host.comps])
        g = [(ctypes.c_void_p * n)(*[a.ctypes.data for a in gs]) for gs in self.host.grads]
        return th, c, g

    def step_host(self, th, c, g) -> None:
        staging = self.dev_g[0]
        B.kahan_sgd_step_host(self.handle, th, c, g, self.lrs, staging.data_ptr(), staging.numel())

    def close(self) -> None:
        if self.handle is not None:
            if self.adam:
                B.kahan_sgd_adam_destroy(self.handle)
            elif self.mom_bits:
                B.kahan_sgd_momentum_destroy(self.handle)
            else:
                B.kahan_sgd_destroy(self.handle)
            self.handle = None
