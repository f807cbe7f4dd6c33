"""kahan_sgd_step_static: the step for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits at step time (all memory
already handed to a host program's pool, a loop that cannot afford the device-wide
synchronisation an allocation implies, a thread next to an ongoing stream capture), so they
cannot give kahan_sgd_init the workspace it asks for.  The static entry point keeps that
scratch inside the library.  This file checks, through the C ABI, that two such calls in a
row give exactly the bits that the ordinary init/step/amax path gives on the same inputs,
and that both agree with the CPU oracle (a mistake shared by the two entry points would
otherwise pass).

It is collected last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest

from harness import DeviceArena, LibraryRun, make_oracle_state, storage_dtype

pytestmark = pytest.mark.gpu

FORMATS = [(8, 8, 0), (16, 8, 0), (16, 16, 0), (8, 16, 0), (8, 0, 0), (16, 0, 0), (8, 8, 3)]
SIZES = [70001, 8192, 33, 250000, 12345, 16384, 99999]


def make_inputs(seed):
    rng = np.random.default_rng(seed)
    specs, thetas, comps = [], [], []
    for (tb, cb, k), n in zip(FORMATS, SIZES):
        q = 2 ** (tb - 1) - 1
        thetas.append(rng.integers(-q, q + 1, n).astype(storage_dtype(tb)))
        s = cb - 1 - k if cb else 0
        comps.append(rng.integers(-2 ** max(s - 1, 0), 2 ** max(s - 1, 0) + 1, n)
                     .astype(storage_dtype(cb)) if cb else None)
        specs.append(dict(numel=n, theta_bits=tb, comp_bits=cb, overlap_k=k, exp_theta=-12))
    grads = []
    for step in range(2):
        gs = []
        for sp in specs:
            s = sp["comp_bits"] - 1 - sp["overlap_k"] if sp["comp_bits"] else 0
            g = (rng.standard_t(3, sp["numel"]) * 2.0 ** (-12 - s) * 400).astype(np.float32)
            g[:: 997] *= np.float32(1e4)          # some saturation
            g[5 % sp["numel"]] = np.float32(np.inf) if step else np.float32(np.nan)
            gs.append(g)
        grads.append(gs)
    lrs = [0.5, 0.25, 1.0, 0.125, 0.5, 0.75, 0.3]
    return specs, thetas, comps, grads, lrs


def test_static_entry_point_matches_the_workspace_path_twice_in_a_row():
    import torch
    from paper_1810_05486_b200 import binding as B
    from oracle import EXP_AMAX, oracle_step
    specs, thetas, comps, grads, lrs = make_inputs(2024)
    n = len(specs)

    # the oracle on the same inputs
    ost = make_oracle_state(specs, thetas, comps, EXP_AMAX)
    oracle_states = []
    for step in range(2):
        before = [(t.n_sat_theta, t.n_sat_comp, t.n_nonfinite) for t in ost.tensors]
        oracle_step(ost, grads[step], lrs)
        oracle_states.append(dict(
            theta=[t.theta.copy() for t in ost.tensors],
            comp=[None if t.comp is None else t.comp.copy() for t in ost.tensors],
            exp_theta_cur=[t.exp_theta for t in ost.tensors],
            exp_theta_next=[t.exp_theta_next for t in ost.tensors],
            amax_theta=[t.amax_theta for t in ost.tensors],
            amax_comp=[t.amax_comp for t in ost.tensors],
            n_sat_theta=[t.n_sat_theta - b[0] for t, b in zip(ost.tensors, before)],
            n_sat_comp=[t.n_sat_comp - b[1] for t, b in zip(ost.tensors, before)],
            n_nonfinite=[t.n_nonfinite - b[2] for t, b in zip(ost.tensors, before)]))

    # reference: the ordinary path with a caller-provided workspace
    ref = LibraryRun(specs, thetas, comps, B.KSGD_EXP_AMAX)
    ref_states = []
    prev = ref.stats()
    for step in range(2):
        ref.step(grads[step], lrs)
        st = ref.stats()
        per_call = dict(st)
        for key in ("n_sat_theta", "n_sat_comp", "n_nonfinite"):
            per_call[key] = [a - b for a, b in zip(st[key], prev[key])]
        prev = st
        ref_states.append((ref.thetas(), ref.comps(), per_call))
    ref.close()

    # the static entry point on its own copies of the same inputs
    th_arena = DeviceArena([s["numel"] * (s["theta_bits"] // 8) for s in specs])
    c_arena = DeviceArena([max(16, s["numel"] * (s["comp_bits"] // 8)) for s in specs])
    g_arena = DeviceArena([s["numel"] * 4 for s in specs])
    for i, s in enumerate(specs):
        th_arena.upload(i, thetas[i])
        if s["comp_bits"]:
            c_arena.sizes[i] = s["numel"] * (s["comp_bits"] // 8)
            c_arena.upload(i, comps[i])
    exp_cur = [s["exp_theta"] for s in specs]
    exp_next = list(exp_cur)
    stream = torch.cuda.current_stream().cuda_stream

    def descs_now():
        return B.make_descs([
            dict(theta=th_arena.ptr(i), comp=c_arena.ptr(i) if s["comp_bits"] else None,
                 numel=s["numel"], theta_bits=s["theta_bits"], comp_bits=s["comp_bits"],
                 overlap_k=s["overlap_k"], exp_theta=exp_cur[i], exp_theta_next=exp_next[i])
            for i, s in enumerate(specs)])

    # One untimed call first, on copies that are thrown away: the first call on a device
    # looks up the scratch array's address and sets the kernel's shared-memory attribute.
    # After it, the free device memory the driver reports must not move: that figure sees a
    # cudaMalloc by anybody, the library included, which torch's own counters would not.
    warm_t = [th_arena.view(i).clone() for i in range(n)]
    warm_c = [c_arena.view(i).clone() for i in range(n)]
    for i in range(n):
        g_arena.upload(i, grads[0][i])
    torch.cuda.synchronize()
    B.kahan_sgd_step_static(descs_now(), B.KSGD_EXP_AMAX, [g_arena.ptr(i) for i in range(n)], lrs, stream)
    for i in range(n):
        th_arena.view(i).copy_(warm_t[i])
        c_arena.view(i).copy_(warm_c[i])
    staged = [[torch.from_numpy(g).cuda() for g in gs] for gs in grads]   # no allocation inside the window
    host_t = [torch.empty(th_arena.sizes[i], dtype=torch.uint8).pin_memory() for i in range(n)]
    host_c = [torch.empty(c_arena.sizes[i], dtype=torch.uint8).pin_memory() for i in range(n)]
    torch.cuda.synchronize()
    launches0 = B.kahan_sgd_launch_count()
    mem0 = torch.cuda.memory_allocated()
    free0 = torch.cuda.mem_get_info()[0]
    for step in range(2):
        for i in range(n):
            g_arena.view(i).copy_(staged[step][i].view(torch.uint8))
        torch.cuda.synchronize()
        out = B.kahan_sgd_step_static(descs_now(), B.KSGD_EXP_AMAX, [g_arena.ptr(i) for i in range(n)],
                                      lrs, stream)
        for i in range(n):                                     # device -> page-locked host, no allocation
            host_t[i].copy_(th_arena.view(i))
            host_c[i].copy_(c_arena.view(i))
        torch.cuda.synchronize()
        want_t, want_c, want = ref_states[step]
        orc = oracle_states[step]
        for i, s in enumerate(specs):
            got_t = host_t[i].numpy().view(storage_dtype(s["theta_bits"]))
            assert np.array_equal(got_t, want_t[i]), (step, i)
            assert np.array_equal(got_t, orc["theta"][i]), (step, i, "oracle")
            if s["comp_bits"]:
                got_c = host_c[i].numpy().view(storage_dtype(s["comp_bits"]))
                assert np.array_equal(got_c, want_c[i]), (step, i)
                assert np.array_equal(got_c, orc["comp"][i]), (step, i, "oracle")
        assert out == want, step
        for key in out:
            assert list(out[key]) == orc[key], (step, key, "oracle")
        exp_cur, exp_next = out["exp_theta_cur"], out["exp_theta_next"]
    assert sum(ref_states[1][2]["n_nonfinite"]) == n          # the planted Inf per tensor
    assert B.kahan_sgd_launch_count() - launches0 == 2
    assert torch.cuda.memory_allocated() == mem0               # torch allocated nothing on the way ...
    assert torch.cuda.mem_get_info()[0] >= free0               # ... and neither did anybody else
    assert th_arena.guards_intact() and c_arena.guards_intact() and g_arena.guards_intact()


def test_static_entry_point_rejects_what_does_not_fit():
    import torch
    from paper_1810_05486_b200 import binding as B
    # real (small) device buffers behind every address, and a length derived from the
    # array's size, so that neither case could ever reach a launch on a wild pointer
    buf = torch.zeros(3 * 4096, dtype=torch.uint8, device="cuda")
    th, c, g = buf.data_ptr(), buf.data_ptr() + 4096, buf.data_ptr() + 8192
    too_many = B.make_descs([dict(theta=th, comp=c, numel=100, theta_bits=8,
                                  comp_bits=8, exp_theta=-11)] * (B.KSGD_STATIC_MAX_TENSORS + 1))
    # 8 bytes of tile table per 8192 elements: four times what the whole array could describe
    numel = 4 * (B.KSGD_STATIC_SCRATCH_BYTES // 8) * 8192
    too_big = B.make_descs([dict(theta=th, comp=c, numel=numel, theta_bits=8,
                                 comp_bits=8, exp_theta=-11)])
    for descs in (too_many, too_big):
        with pytest.raises(B.KahanSgdError) as ei:
            B.kahan_sgd_step_static(descs, B.KSGD_EXP_AMAX, [g] * len(descs),
                                    [0.1] * len(descs))
        assert ei.value.code == B.KSGD_ERR_WORKSPACE
    assert bool((buf == 0).all())
