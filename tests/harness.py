"""Shared plumbing of the GPU parity tests: device buffers with guard bands around every
tensor, a runner that drives the C ABI, and the matching oracle state."""
from typing import List, Optional, Sequence

import numpy as np

GUARD = 256          # bytes of canary before and after every device tensor
CANARY = 0xA5


def storage_dtype(bits: int):
    return np.int8 if bits <= 8 else np.int16


class DeviceArena:
    """One torch uint8 buffer carved into 256-byte aligned slots separated by canaries."""

    def __init__(self, sizes_bytes: Sequence[int], device="cuda"):
        import torch
        self.offsets = []
        off = GUARD
        for nb in sizes_bytes:
            self.offsets.append(off)
            off += (nb + 255) // 256 * 256 + GUARD
        self.sizes = list(sizes_bytes)
        self.buf = torch.full((off,), CANARY, dtype=torch.uint8, device=device)
        self.base = self.buf.data_ptr()
        assert self.base % 256 == 0

    def ptr(self, i: int) -> int:
        return self.base + self.offsets[i]

    def view(self, i: int):
        return self.buf[self.offsets[i]:self.offsets[i] + self.sizes[i]]

    def upload(self, i: int, arr: np.ndarray) -> None:
        import torch
        src = torch.from_numpy(np.ascontiguousarray(arr).view(np.uint8).reshape(-1))
        assert src.numel() == self.sizes[i]
        self.view(i).copy_(src)

    def download(self, i: int, dtype) -> np.ndarray:
        return self.view(i).cpu().numpy().view(dtype).copy()

    def guards_intact(self) -> bool:
        import torch
        mask = torch.ones(self.buf.numel(), dtype=torch.bool, device=self.buf.device)
        for off, nb in zip(self.offsets, self.sizes):
            mask[off:off + nb] = False
        return bool((self.buf[mask] == CANARY).all().item())


class LibraryRun:
    """Drives kahan_sgd_* on device copies of the given tensors."""

    def __init__(self, specs: Sequence[dict], thetas: Sequence[np.ndarray],
                 comps: Sequence[Optional[np.ndarray]], mode: int, stream=None, strict: bool = False):
        import torch
        from paper_1810_05486_b200 import binding as B
        self.B = B
        self.torch = torch
        self.specs = [dict(s) for s in specs]
        self.n = len(specs)
        self.theta_arena = DeviceArena([s["numel"] * (s["theta_bits"] // 8) for s in specs])
        self.comp_arena = DeviceArena([max(16, s["numel"] * (s["comp_bits"] // 8)) for s in specs])
        self.grad_arena = DeviceArena([s["numel"] * 4 for s in specs])
        descs = []
        for i, s in enumerate(specs):
            self.theta_arena.upload(i, thetas[i])
            if s["comp_bits"]:
                self.comp_arena.sizes[i] = s["numel"] * (s["comp_bits"] // 8)
                self.comp_arena.upload(i, comps[i])
            descs.append(dict(theta=self.theta_arena.ptr(i),
                              comp=self.comp_arena.ptr(i) if s["comp_bits"] else None,
                              numel=s["numel"], theta_bits=s["theta_bits"],
                              comp_bits=s["comp_bits"], overlap_k=s.get("overlap_k", 0),
                              exp_theta=s["exp_theta"],
                              exp_theta_next=s.get("exp_theta_next", s["exp_theta"])))
        self.descs = B.make_descs(descs)
        self.strict = strict
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        if strict:
            ec = [s["exp_comp"] for s in specs]
            ec_next = [s.get("exp_comp_next", s["exp_comp"]) for s in specs]
            nbytes = B.kahan_sgd_strict_workspace_bytes(self.descs, ec)
            assert nbytes > 0
            self.workspace = torch.zeros(nbytes + 256, dtype=torch.uint8, device="cuda")
            self.handle = B.kahan_sgd_strict_init(self.descs, ec, ec_next, mode, self.workspace.data_ptr(), nbytes,
                                                  self.stream.cuda_stream)
        else:
            nbytes = B.kahan_sgd_workspace_bytes(self.descs)
            assert nbytes > 0
            self.workspace = torch.zeros(nbytes + 256, dtype=torch.uint8, device="cuda")
            self.handle = B.kahan_sgd_init(self.descs, mode, self.workspace.data_ptr(), nbytes,
                                           self.stream.cuda_stream)
        self.grad_ptrs = [self.grad_arena.ptr(i) for i in range(self.n)]

    def step(self, grads: Sequence[np.ndarray], lrs: Sequence[float]) -> None:
        for i, g in enumerate(grads):
            self.grad_arena.upload(i, g)
        self.B.kahan_sgd_step(self.handle, self.grad_ptrs, list(lrs))

    def step_qgrad(self, grads_q: Sequence[np.ndarray], exp_grads: Sequence[int],
                   lrs: Sequence[float], exponents_on_device: bool = False) -> None:
        """Fixed-point gradients (all int8 or all int16), in a guarded arena of their own;
        their exponents from the host, or from a device array the step reads when it runs."""
        bits = 8 * grads_q[0].dtype.itemsize
        if getattr(self, "qgrad_arena", None) is None:
            self.qgrad_arena = DeviceArena([s["numel"] * 2 for s in self.specs])
        for i, g in enumerate(grads_q):
            assert g.dtype == storage_dtype(bits) and g.size == self.specs[i]["numel"]
            if g.nbytes < self.qgrad_arena.sizes[i]:      # narrower gradients than last time: the rest is guard again
                self.qgrad_arena.view(i)[g.nbytes:] = CANARY
            self.qgrad_arena.sizes[i] = g.nbytes
            self.qgrad_arena.upload(i, g)
        ptrs = [self.qgrad_arena.ptr(i) for i in range(self.n)]
        if exponents_on_device:
            self.exp_grad_dev = self.torch.tensor([int(e) for e in exp_grads], dtype=self.torch.int32, device="cuda")
            self.torch.cuda.current_stream().synchronize()      # the upload is torch's; the step may run on another stream
            self.B.kahan_sgd_step_qgrad_dev(self.handle, ptrs, bits, self.exp_grad_dev.data_ptr(), list(lrs))
        else:
            self.B.kahan_sgd_step_qgrad(self.handle, ptrs, bits, [int(e) for e in exp_grads], list(lrs))

    def set_exponents(self, exps: Sequence[int]) -> None:
        self.B.kahan_sgd_set_exponents(self.handle, list(exps))

    def stats(self) -> dict:
        st = self.B.kahan_sgd_amax(self.handle, self.n)
        if self.strict:
            st.update(self.B.kahan_sgd_strict_exponents(self.handle, self.n))
        return st

    def thetas(self) -> List[np.ndarray]:
        self.torch.cuda.synchronize()
        return [self.theta_arena.download(i, storage_dtype(s["theta_bits"]))
                for i, s in enumerate(self.specs)]

    def comps(self) -> List[Optional[np.ndarray]]:
        self.torch.cuda.synchronize()
        return [self.comp_arena.download(i, storage_dtype(s["comp_bits"])) if s["comp_bits"]
                else None for i, s in enumerate(self.specs)]

    def guards_intact(self) -> bool:
        self.torch.cuda.synchronize()
        arenas = [self.theta_arena, self.comp_arena, self.grad_arena]
        if getattr(self, "qgrad_arena", None) is not None:
            arenas.append(self.qgrad_arena)
        return all(a.guards_intact() for a in arenas)

    def close(self) -> None:
        if self.handle is not None:
            self.B.kahan_sgd_destroy(self.handle)
            self.handle = None


def make_oracle_state(specs, thetas, comps, mode, n_threads=1):
    from oracle import OracleState, OracleTensor
    ts = []
    for s, th, c in zip(specs, thetas, comps):
        ts.append(OracleTensor(th.copy(), None if c is None else c.copy(), s["theta_bits"],
                               s["comp_bits"], s.get("overlap_k", 0), s["exp_theta"],
                               s.get("exp_theta_next", s["exp_theta"]),
                               exp_comp=s.get("exp_comp", 0),
                               exp_comp_next=s.get("exp_comp_next", s.get("exp_comp", 0))))
    return OracleState(ts, mode, n_threads)


def assert_same_state(gpu: LibraryRun, ost, where="") -> None:
    """Bit-exact comparison of everything a step produces."""
    st = gpu.stats()
    got_t, got_c = gpu.thetas(), gpu.comps()
    for i, t in enumerate(ost.tensors):
        tag = f"{where} tensor {i}"
        assert np.array_equal(got_t[i], t.theta), \
            f"{tag}: theta differs at {np.flatnonzero(got_t[i] != t.theta)[:8]}"
        if t.comp_bits:
            assert np.array_equal(got_c[i], t.comp), \
                f"{tag}: comp differs at {np.flatnonzero(got_c[i] != t.comp)[:8]}"
        assert st["exp_theta_cur"][i] == t.exp_theta, tag
        assert st["exp_theta_next"][i] == t.exp_theta_next, tag
        assert st["amax_theta"][i] == t.amax_theta, tag
        assert st["amax_comp"][i] == t.amax_comp, tag
        assert st["n_sat_theta"][i] == t.n_sat_theta, tag
        assert st["n_sat_comp"][i] == t.n_sat_comp, tag
        assert st["n_nonfinite"][i] == t.n_nonfinite, tag
        if gpu.strict:
            assert (st["exp_comp_cur"][i], st["exp_comp_next"][i]) == (t.exp_comp, t.exp_comp_next), tag


def specs_of(wl) -> List[dict]:
    return [dict(numel=t.numel, theta_bits=t.theta_bits, comp_bits=t.comp_bits,
                 overlap_k=t.overlap_k, exp_theta=t.exp_theta) for t in wl.tensors]
