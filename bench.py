#!/usr/bin/env python
"""Benchmark of the lazy-update step (SGD with Kahan summation, dynamic fixed-point).

A "step" is one pass of the whole hot path over one synthetic parameter list: gradient
quantization, compensated update, requantization, compensation store, per-tensor max
scans and the exponent choice, i.e. one kahan_sgd_step call.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints one JSON line.  `value` is parameters updated per second with every input
resident in device memory; `e2e` is the same metric through kahan_sgd_step_host with
page-locked host buffers (host->device and device->host copies inside the timed region);
`roofline` relates the step kernel to the measured HBM copy bandwidth; `cpu_baseline` is
the CPU oracle timed on this machine's cores.  With N > 1 (torchrun) every rank updates
its own parameter list of the same shape (weak scaling, no data-path collective: the
update of one tensor never needs another tensor).
"""
import argparse
import ctypes
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "parameters updated/sec and achieved HBM GB/s (% of B200 peak) per Kahan SGD step"
UNIT = "parameters/s"
FALLBACK_HBM_GBS = 6650.0
# Gradient sets kept resident and used in turn: c5 alternates two sets (its recipe), the
# other workloads draw a fresh gradient for every step of their recipe.
L2_BYTES = 126 << 20     # B200 L2 capacity
GRAD_SETS = {"c5_sweep": 2, "c1_single": 100, "c2_resnet20": 200, "c3_resnet50": 50, "c4_alexnet": 20}


# DRAM traffic of ksgd_step_kernel from ncu captures (dram__bytes_read.sum +
# dram__bytes_write.sum per launch, divided by the parameters of the captured launch; see
# profiles/).  "cold": caches flushed before the launch (ncu's default); c5_sweep was captured
# at 2e8 parameters and its traffic is proportional to the parameter count, so a full launch
# is this figure times its parameters.  "warm": the launch as it runs in the benchmark's loop,
# caches left as the preceding steps left them (--cache-control none): the steady state,
# which is what counts for a list whose theta and c partly stay in L2 from step to step (a
# warm launch also writes back lines the preceding step left dirty, a cold one leaves some
# of its own behind).  The record only counts while the kernel sources (kahan_sgd_ring.cuh,
# kahan_sgd_kernels.cuh) still hash to the value below.
TRAFFIC_RECORD = {
    "sources_sha256": "36afd64ba1344e8e6c095c1faaecfc39d6ecfad7b9634488069076cebcd439bf",
    "dram_bytes_per_parameter": {
        "c5_sweep": {"cold": 2351.837e6 / 2e8, "warm": None},
        "c4_alexnet": {"cold": 463.616e6 / 61100840, "warm": 464.885e6 / 61100840},
        "c3_resnet50": {"cold": 200.816e6 / 25557032, "warm": 219.663e6 / 25557032},
    },
}


def kernel_sources_sha256():
    import hashlib
    h = hashlib.sha256()
    for name in ("kahan_sgd_ring.cuh", "kahan_sgd_kernels.cuh"):
        with open(os.path.join(ROOT, "paper_1810_05486_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def recorded_traffic(wl, kind="cold"):
    """DRAM bytes of one launch from the ncu record, or None once the kernel has changed."""
    try:
        if kernel_sources_sha256() != TRAFFIC_RECORD["sources_sha256"]:
            return None
        per = TRAFFIC_RECORD["dram_bytes_per_parameter"].get(wl.name, {}).get(kind)
        return None if per is None else per * wl.numel
    except Exception:
        return None


def state_bytes_of(wl):
    return sum(t.numel * (t.theta_bits + t.comp_bits) // 8 for t in wl.tensors)


def l2_resident_state(wl):
    """True if theta and c of the whole list stay in L2 from step to step (the library marks
    the gradient loads evict-first under the same condition)."""
    return state_bytes_of(wl) <= 0.8 * L2_BYTES


def l2_note(wl, n_sets):
    """How the timed steps relate to the 126 MB L2.  What decides is the state (theta and c)
    plus ONE gradient set, not the bytes a step touches: a state that fits stays resident
    while the gradients stream through."""
    state = state_bytes_of(wl)
    grads = wl.bytes_per_step - 2 * state
    if state + n_sets * grads <= L2_BYTES:
        return "working set %.1f MB fits L2: a launch-latency figure, not a DRAM one" % ((state + n_sets * grads) / 1e6)
    if l2_resident_state(wl):
        return ("L2-assisted: theta and c (%.1f MB) stay resident in L2 from step to step; a fresh gradient "
                "set every step (%d sets, %.0f MB each) streams from DRAM, so a step moves fewer DRAM bytes "
                "than its %.0f MB of algorithmic bytes" % (state / 1e6, n_sets, grads / 1e6, wl.bytes_per_step / 1e6))
    return "inputs larger than L2 (state %.0f MB + %.0f MB of gradients per step)" % (state / 1e6, grads / 1e6)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0,
                    help="timed steps (default: 500 for c5_sweep, about a second, the recipe's own step count otherwise)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c5_sweep")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--sweep-total", type=int, default=0,
                    help="with --workload c5_sweep: scaled-down total parameter count (profiling)")
    ap.add_argument("--sweep-tensors", type=int, default=0)
    ap.add_argument("--momentum-bits", type=int, default=0, choices=[0, 8, 16],
                    help="8 or 16: time the momentum optimizer (mu 0.9) with a velocity tensor of that width")
    ap.add_argument("--adam", action="store_true",
                    help="time ADAM (beta1 0.9, beta2 0.999, eps 1e-8, two int16 moment tensors; the step "
                         "size is 1e-3 of the first tensor's range)")
    ap.add_argument("--grad-bits", type=int, default=32, choices=[8, 16, 32],
                    help="8 or 16: the gradients are fixed-point tensors of that width (made on the device "
                         "from the binary32 ones before the timed region)")
    ap.add_argument("--strict", action="store_true",
                    help="strict Algorithm 1: every statement rounded into the stored format, the "
                         "compensation with its own exponent")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-buckets", action="store_true",
                    help="skip the per-size-bucket timing of c5_sweep")
    ap.add_argument("--no-extra-workloads", action="store_true",
                    help="skip the c3_resnet50 / c4_alexnet legs that the default run adds to its line")
    ap.add_argument("--no-optimizers", action="store_true",
                    help="skip the momentum / ADAM / int8-gradient legs that the default run adds to its line")
    ap.add_argument("--no-convert", action="store_true",
                    help="skip the fp32 <-> fixed-point conversion leg that the default run adds to its line")
    ap.add_argument("--convert-only", action="store_true",
                    help="time the fp32 <-> fixed-point conversion leg alone and print it as one JSON line")
    ap.add_argument("--sustained-s", type=float, default=0.35,
                    help="length of the sustained leg (the same steps repeated for about this long, with the "
                         "clocks sampled inside it); 0 skips it")
    return ap.parse_args()


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """nvidia-smi clock samples; only those stamped inside the timed region are kept."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "50"], stdout=f,
                stderr=subprocess.DEVNULL)
            f.close()
        except Exception:
            self.proc = None

    def stop(self, t_begin: float, t_end: float) -> dict:
        """t_begin / t_end: time.time() around the timed region."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = []
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(parts[1]), float(parts[2]),
                                 [n for n, v in zip(names, parts[5:9]) if v.lower().startswith("active")]))
                except ValueError:
                    continue
            os.unlink(self.path)
        except Exception:
            pass
        inside = [r for r in rows if t_begin <= r[0] <= t_end + 0.05]
        if not inside and rows:
            # a timed region shorter than the sampling period: the samples closest to it
            out["window"] = "no sample inside the timed region; samples within 0.3 s of it"
            inside = [r for r in rows if t_begin - 0.3 <= r[0] <= t_end + 0.3]
        if inside:
            out.update(sm_mhz=statistics.median(r[1] for r in inside), sm_max_mhz=max(r[2] for r in inside),
                       samples=len(inside))
            out["reasons"] = sorted({n for r in inside for n in r[3]})
        return out


def pick_workload(W, args):
    if args.workload == "c5_sweep" and args.sweep_total:
        return W.scaled_sweep(args.sweep_total, args.sweep_tensors or 256)
    return W.workload(args.workload)


def timed_region(torch, B, run, n_sets, steps, first_set, barrier, sampler=None):
    """`steps` back-to-back steps on the handle's stream between two CUDA events (recorded on
    that stream), a barrier and a device synchronisation on both sides.  Returns total ms,
    the per-step ms of each quarter of the region, launches of the library's kernels, and
    the clock record if a sampler was given."""
    stream = run.stream
    if sampler is not None:
        sampler.start()
        time.sleep(0.2)
    launches0 = B.kahan_sgd_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    wall0 = time.time()
    ev0.record(stream)
    marks = []          # events at the quarters of the timed region (clock-regime record)
    for i in range(steps):
        run.step((first_set + i) % n_sets)
        if steps >= 40 and (i + 1) % (steps // 4) == 0 and len(marks) < 3:
            marks.append(torch.cuda.Event(enable_timing=True))
            marks[-1].record(stream)
    ev1.record(stream)
    barrier()
    wall1 = time.time()
    launches = B.kahan_sgd_launch_count() - launches0
    ms_total = ev0.elapsed_time(ev1)
    quarters = None
    if len(marks) == 3:
        pts = [ev0] + marks + [ev1]
        q = steps // 4
        counts = [q, q, q, steps - 3 * q]
        quarters = [round(pts[j].elapsed_time(pts[j + 1]) / counts[j], 6) for j in range(4)]
    clocks = sampler.stop(wall0, wall1) if sampler is not None else None
    return ms_total, quarters, int(launches), clocks


def sustained_leg(torch, B, run, n_sets, ms_step, seconds, first_set, barrier, gpu_index, bytes_per_step, peak):
    """The same steps repeated for about `seconds` (gradient sets reused in turn), with the
    clocks sampled inside the region: the figure a long training run sees, and the one a
    timed region of a few milliseconds cannot carry a clock record for."""
    steps = max(40, int(seconds / max(ms_step * 1e-3, 1e-6)))
    steps = min(steps, 200000)
    ms_total, quarters, _, clocks = timed_region(torch, B, run, n_sets, steps, first_set, barrier,
                                                 ClockSampler(gpu_index))
    ms = ms_total / steps
    gbs = bytes_per_step / (ms * 1e-3) / 1e9
    out = {"steps": steps, "ms_per_step": ms, "ms_per_step_quarters": quarters, "algorithmic_gbs": gbs,
           "frac": gbs / peak, "clocks": clocks}
    if clocks and clocks.get("sm_mhz"):
        # time x clock: how the step depends on the SM clock the box happened to run at
        out["us_x_ghz"] = round(ms * 1e3 * clocks["sm_mhz"] / 1e3, 2)
    return out


def roofline_of(wl, bytes_per_step, ms_step, peak, peak_src, kernel, plain):
    """The roofline object of one workload.  `achieved` counts the ALGORITHMIC bytes of a
    step (2m/8 + 2n/8 + 4 per parameter); `traffic` is what DRAM really moved per launch
    (ncu), `dram_gbs` that traffic over the same time.  For a list whose state stays in L2
    the two differ, and `dram_gbs` is the DRAM-side figure."""
    achieved = bytes_per_step / (ms_step * 1e-3) / 1e9
    r = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
         "traffic": None, "peak_source": peak_src, "frac_of_nominal_8000": achieved / 8000.0,
         "kernel": kernel, "launch_ms": ms_step, "l2_assisted": l2_resident_state(wl)}
    if plain:
        kind = "warm" if TRAFFIC_RECORD["dram_bytes_per_parameter"].get(wl.name, {}).get("warm") else "cold"
        traffic = recorded_traffic(wl, kind)
        r["traffic"] = traffic
        r["traffic_capture"] = ("ncu --cache-control none (caches as the preceding steps left them)"
                                if kind == "warm" else "ncu default (caches flushed before the launch)")
        if traffic is not None:
            r["dram_gbs"] = traffic / (ms_step * 1e-3) / 1e9
            r["frac_dram"] = r["dram_gbs"] / peak
    return r


def convert_leg(torch, B, peak, numel=64 * 1024 * 1024, iters=10):
    """fp32 <-> dynamic fixed-point on one tensor of `numel` elements (256 MB of binary32,
    twice the L2): kahan_sgd_import_dev (max scan, exponent chosen on the device, quantization:
    the source is read twice) and kahan_sgd_export, each timed over `iters` back-to-back calls
    after two warm-up calls.  Algorithmic bytes per element: import 4 + 4 + m/8 + n/8, export
    m/8 + n/8 + 4."""
    st = torch.cuda.current_stream()
    gen = torch.Generator(device="cuda").manual_seed(7)
    src = torch.randn(numel, generator=gen, device="cuda", dtype=torch.float32) * 0.05
    dst = torch.empty(numel, dtype=torch.float32, device="cuda")
    scratch = torch.zeros(4, dtype=torch.int32, device="cuda")
    exp_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = []
    for tb, cb, what in ((8, 0, "int8 gradients"), (16, 0, "int16 gradients"), (16, 8, "int16 theta + int8 c"),
                         (8, 8, "int8 theta + int8 c"), (16, 16, "int16 theta + int16 c")):
        th = torch.empty(numel * (tb // 8), dtype=torch.uint8, device="cuda")
        c = torch.empty(numel * (cb // 8), dtype=torch.uint8, device="cuda") if cb else None
        torch.cuda.synchronize()

        def imp():
            B.kahan_sgd_import_dev(src.data_ptr(), th.data_ptr(), c.data_ptr() if cb else None, numel, tb, cb, 0,
                                   exp_dev.data_ptr(), scratch.data_ptr(), st.cuda_stream)

        def exp():
            B.kahan_sgd_export(th.data_ptr(), c.data_ptr() if cb else None, dst.data_ptr(), numel, tb, cb, 0,
                               e_used, st.cuda_stream)
        row = {"format": what, "elements": numel}
        imp()
        torch.cuda.synchronize()
        e_used = int(exp_dev.item())
        for name, fn, nbytes in (("import", imp, 8 + (tb + cb) // 8), ("export", exp, 4 + (tb + cb) // 8)):
            fn()
            fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(st)
            for _ in range(iters):
                fn()
            e1.record(st)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / iters
            gbs = numel * nbytes / (ms * 1e-3) / 1e9
            row[name] = {"ms": round(ms, 4), "bytes_per_element": nbytes, "gbs": round(gbs, 1),
                         "frac": round(gbs / peak, 3), "elements_per_s": numel / (ms * 1e-3)}
        row["exponent"] = e_used
        out.append(row)
        del th, c
    return out


OPTIMIZER_KERNELS = {"sgd": "ksgd_step_kernel", "sgd, int8 gradients": "ksgd_step_qgrad_kernel",
                     "momentum 0.9, int16 velocity": "ksgd_momentum_step_kernel",
                     "momentum 0.9, int8 velocity": "ksgd_momentum_step_kernel",
                     "adam 0.9/0.999/1e-8, int16 moments": "ksgd_adam_step_kernel"}


def extra_workload(torch, B, W, name, args, peak, peak_src, barrier, gpu_index, host=None, optimizer="sgd"):
    """One of the other workloads of at least 25 M parameters, timed like the headline: the
    recipe's own number of steps (a fresh gradient set each), then the sustained leg.
    optimizer: "sgd" (the path of the headline), or one of the optimizers and gradient formats
    built around the same update (their extra arrays count as algorithmic bytes)."""
    from paper_1810_05486_b200.runner import DeviceRun, HostInputs
    wl = W.workload(name)
    n_sets = GRAD_SETS[name]
    if host is None:
        host = HostInputs(wl, args.seed, n_sets, pinned=False)
    kw = {}
    if optimizer.startswith("momentum"):
        kw["mom_bits"] = 16 if "int16" in optimizer else 8
    elif optimizer.startswith("adam"):
        t0_ = wl.tensors[0]
        kw["adam"] = dict(beta1=0.9, beta2=0.999, eps=1e-8,
                          eta=1e-3 * 2.0 ** t0_.exp_theta * (2 ** (t0_.theta_bits - 1) - 1))
    elif "int8 gradients" in optimizer:
        kw["grad_bits"] = 8
    run = DeviceRun(host, B.KSGD_EXP_AMAX, **kw)
    with torch.cuda.stream(run.stream):
        for i in range(args.warmup):
            run.step(i % n_sets)
        barrier()
        ms_total, quarters, launches, _ = timed_region(torch, B, run, n_sets, wl.steps, args.warmup, barrier)
        ms_step = ms_total / wl.steps
        out = {"workload": name, "optimizer": optimizer, "tensors": len(wl.tensors), "parameters": wl.numel,
               "bytes_per_step": run.bytes_per_step, "steps": wl.steps, "warmup": args.warmup,
               "ms_per_step": ms_step, "value": wl.numel / (ms_step * 1e-3), "unit": UNIT,
               "gpu_launches": launches, "l2": l2_note(wl, n_sets),
               "roofline": roofline_of(wl, run.bytes_per_step, ms_step, peak, peak_src,
                                       OPTIMIZER_KERNELS[optimizer], optimizer == "sgd")}
        if args.sustained_s > 0:
            out["sustained"] = sustained_leg(torch, B, run, n_sets, ms_step, args.sustained_s,
                                             args.warmup + wl.steps, barrier, gpu_index, run.bytes_per_step, peak)
    st = run.stats()
    out["counters"] = {"n_sat_theta": int(sum(st["n_sat_theta"])), "n_sat_comp": int(sum(st["n_sat_comp"])),
                       "n_nonfinite": int(sum(st["n_nonfinite"]))}
    run.close()
    del run
    torch.cuda.empty_cache()
    return out


def run_ours(args, rank, world, local_rank):
    import torch
    import __graft_entry__ as entry
    if not os.path.exists(os.path.join(ROOT, "paper_1810_05486_b200", "libkahan_sgd.so")):
        entry.build()
    from paper_1810_05486_b200 import binding as B
    from paper_1810_05486_b200 import workloads as W
    from paper_1810_05486_b200 import multi
    from paper_1810_05486_b200.runner import DeviceRun, HostInputs

    torch.cuda.set_device(local_rank)
    if args.convert_only:
        if rank == 0:
            peak, peak_src = hbm_peak()
            with torch.cuda.stream(torch.cuda.Stream()):
                rows = convert_leg(torch, B, peak)
            print(json.dumps({"convert": rows, "peak": peak, "peak_source": peak_src, "unit": "GB/s",
                              "gpu_launches": B.kahan_sgd_launch_count()}), flush=True)
        return
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    wl = pick_workload(W, args)
    n = len(wl.tensors)
    n_sets = GRAD_SETS.get(wl.name, 4)
    if not args.steps:
        args.steps = 500 if wl.name == "c5_sweep" else wl.steps
    t0 = time.time()
    host = HostInputs(wl, multi.rank_seed(args.seed, rank), n_sets, pinned=True)
    gen_s = time.time() - t0
    adam = None
    if args.adam:
        t0_ = wl.tensors[0]
        adam = dict(beta1=0.9, beta2=0.999, eps=1e-8,
                    eta=1e-3 * 2.0 ** t0_.exp_theta * (2 ** (t0_.theta_bits - 1) - 1))
    run = DeviceRun(host, B.KSGD_EXP_AMAX, mom_bits=args.momentum_bits, adam=adam, grad_bits=args.grad_bits,
                    strict=args.strict)
    other = bool(args.momentum_bits or args.adam or args.grad_bits != 32 or args.strict)
    if other:
        args.no_e2e = args.no_cpu_baseline = True      # those legs describe the plain step
    stream = run.stream

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident throughput ---------------------------------------------------
    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            run.step(i % n_sets)
        barrier()
        ms_total, quarters, launches, clocks = timed_region(
            torch, B, run, n_sets, args.steps, args.warmup, barrier,
            ClockSampler(local_rank) if rank == 0 else None)
    stats = run.stats()

    ms_total = multi.max_over_ranks(ms_total, dist, "cuda")
    ms_step = ms_total / args.steps
    value = multi.whole_job_throughput(wl.numel, world, ms_step * 1e-3)

    peak, peak_src = hbm_peak()
    sustained = None
    if args.sustained_s > 0 and world == 1:
        with torch.cuda.stream(stream):
            sustained = sustained_leg(torch, B, run, n_sets, ms_step, args.sustained_s, args.warmup + args.steps,
                                      barrier, local_rank, run.bytes_per_step, peak)

    # ---- end to end through host buffers ------------------------------------------------
    e2e = None
    if not args.no_e2e:
        th_h, c_h, g_h = run.host_pointer_arrays()
        run.step_host(th_h, c_h, g_h[0])
        barrier()
        t0 = time.perf_counter()
        for i in range(args.e2e_steps):
            run.step_host(th_h, c_h, g_h[(i + 1) % n_sets])
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt = multi.max_over_ranks(dt, dist, "cuda")
        state_bytes = sum(t.numel * (t.theta_bits + t.comp_bits) // 8 for t in wl.tensors)
        e2e = {"value": multi.whole_job_throughput(wl.numel * args.e2e_steps, world, dt), "unit": UNIT,
               "h2d_bytes_per_step": state_bytes + 4 * wl.numel,
               "d2h_bytes_per_step": state_bytes, "steps": args.e2e_steps,
               "ms_per_step": dt / args.e2e_steps * 1e3}
    graph_us = None
    if wl.bytes_per_step < (64 << 20) and world == 1 and not other:
        # small lists are bound by the host's launch rate: also time the same steps recorded
        # once into a CUDA graph and replayed (kahan_sgd_step only enqueues work)
        with torch.cuda.stream(stream):
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for i in range(args.steps):
                    run.step(i % n_sets)
            graph.replay()
            stream.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(stream)
            graph.replay()
            g1.record(stream)
            stream.synchronize()
            graph_us = g0.elapsed_time(g1) * 1e3 / args.steps
    buckets = None
    if wl.name == "c5_sweep" and rank == 0 and not other and not args.no_buckets:
        buckets = time_size_buckets(torch, B, run, wl)
    run.close()
    bytes_per_step = run.bytes_per_step
    run.dev_th = run.dev_c = run.dev_g = run.workspace = None      # give the device memory back

    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    kernel = ("ksgd_momentum_step_kernel" if args.momentum_bits
              else ("ksgd_adam_step_kernel" if args.adam else
                    (("ksgd_strict_step" if args.strict else "ksgd_step") +
                     ("_kernel" if args.grad_bits == 32 else "_qgrad_kernel"))))
    roofline = roofline_of(wl, bytes_per_step, ms_step, peak, peak_src, kernel, not other)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "tensors": n, "parameters": wl.numel,
                   "bytes_per_step": bytes_per_step, "grad_sets": n_sets,
                   "optimizer": "momentum 0.9, int%d velocity" % args.momentum_bits if args.momentum_bits
                   else ("adam 0.9/0.999/1e-8, int16 moments" if args.adam else
                         (("sgd" if args.grad_bits == 32 else "sgd, int%d gradients" % args.grad_bits) +
                          (", strict Algorithm 1" if args.strict else ""))),
                   "l2": l2_note(wl, n_sets),
                   "exponent_mode": "amax", "input_generation_s": round(gen_s, 1)},
        # algorithmic bytes per second (not DRAM bytes: see roofline.dram_gbs / roofline.l2_assisted)
        "achieved_hbm_gbs": roofline["achieved"],
        # ms per step in each quarter of the timed region: under sustained load the power cap
        # lowers the SM clock within a few tenths of a second, and the step gets faster with it
        "ms_per_step_quarters": quarters,
        "roofline": roofline,
        "sustained": sustained,
        "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
        "counters": {"n_sat_theta": int(sum(stats["n_sat_theta"])),
                     "n_sat_comp": int(sum(stats["n_sat_comp"])),
                     "n_nonfinite": int(sum(stats["n_nonfinite"]))},
    }
    if buckets is not None:
        line["size_buckets"] = buckets
    if graph_us is not None:
        line["cuda_graph"] = {"us_per_step": graph_us,
                              "note": "the same %d steps recorded once into a CUDA graph and replayed" % args.steps}
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl, host, budget_core_s=20.0)
    if (wl.name == "c5_sweep" and not args.sweep_total and not other and world == 1
            and not args.no_extra_workloads):
        # the other two workloads of at least 25 M parameters, on the same line
        run.host = None
        del host        # page-locked host copies of the sweep (12 GB) go before the next workloads come
        torch.cuda.empty_cache()
        from paper_1810_05486_b200.runner import HostInputs
        line["workloads"], line["optimizers"] = [], []
        for name, others in (("c3_resnet50", ("adam 0.9/0.999/1e-8, int16 moments",)),
                             ("c4_alexnet", ("momentum 0.9, int16 velocity", "sgd, int8 gradients"))):
            h2 = HostInputs(W.workload(name), args.seed, GRAD_SETS[name], pinned=False)
            line["workloads"].append(extra_workload(torch, B, W, name, args, peak, peak_src, barrier, local_rank, h2))
            if not args.no_optimizers:
                # the optimizers of Section 4 and the all-fixed-point gradient format, on the same inputs
                for opt in others:
                    line["optimizers"].append(extra_workload(torch, B, W, name, args, peak, peak_src, barrier,
                                                             local_rank, h2, opt))
            del h2
        if not args.no_convert:
            line["convert"] = convert_leg(torch, B, peak)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def time_size_buckets(torch, B, run, wl, steps=20):
    """GB/s of the step on the sub-list of every tensor-size bucket [2^j, 2^(j+1)) of the
    sweep, on the device buffers of the full run (each sub-list gets its own handle)."""
    import math
    out = []
    by_bucket = {}
    for i, t in enumerate(wl.tensors):
        by_bucket.setdefault(int(math.log2(t.numel)), []).append(i)
    for j in sorted(by_bucket):
        idx = by_bucket[j]
        sub = [dict(theta=run.descs[i].theta, comp=run.descs[i].comp, numel=run.descs[i].numel,
                    theta_bits=run.descs[i].theta_bits, comp_bits=run.descs[i].comp_bits,
                    overlap_k=run.descs[i].overlap_k, exp_theta=wl.tensors[i].exp_theta) for i in idx]
        descs = B.make_descs(sub)
        nb = B.kahan_sgd_workspace_bytes(descs)
        ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()      # the fill ran on torch's stream, the library works on run.stream
        h = B.kahan_sgd_init(descs, B.KSGD_EXP_AMAX, ws.data_ptr(), nb, run.stream.cuda_stream)
        gp = [(ctypes.c_void_p * len(idx))(*[run.grad_ptr_sets[k][i] for i in idx]) for k in range(2)]
        lr = (ctypes.c_float * len(idx))(*([wl.lr] * len(idx)))
        for k in range(3):
            B.kahan_sgd_step(h, gp[k % 2], lr)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        run.stream.synchronize()
        ev0.record(run.stream)
        for k in range(steps):
            B.kahan_sgd_step(h, gp[k % 2], lr)
        ev1.record(run.stream)
        run.stream.synchronize()
        ms = ev0.elapsed_time(ev1) / steps
        B.kahan_sgd_destroy(h)
        params = sum(wl.tensors[i].numel for i in idx)
        out.append({"log2_size": j, "tensors": len(idx), "parameters": params,
                    "us_per_step": round(ms * 1e3, 2), "gbs": round(params * 12 / (ms * 1e-3) / 1e9, 1)})
    return out


def cpu_baseline(wl, host, budget_core_s):
    """Time the oracle, as it stands, with all host cores on a bounded sample: one step of
    the largest tensors of the workload until about budget_core_s core-seconds are spent."""
    from oracle import oracle_step_tensor, oracle_max_threads
    cores = oracle_max_threads()
    done, t_used, k = 0, 0.0, 0
    order = sorted(range(len(wl.tensors)), key=lambda i: -wl.tensors[i].numel)
    for i in order:
        t = wl.tensors[i]
        th = host.thetas[i].copy()
        c = host.comps[i].copy() if t.comp_bits else None
        g = host.grads[0][i]
        t0 = time.perf_counter()
        oracle_step_tensor(th, c, g, t.theta_bits, t.comp_bits, t.overlap_k, t.exp_theta,
                           t.exp_theta, wl.lr, cores)
        t_used += time.perf_counter() - t0
        done += t.numel
        k += 1
        if t_used * cores >= budget_core_s:
            break
    # one thread, on the largest tensor alone (a few seconds at most)
    i = order[0]
    t = wl.tensors[i]
    n1 = min(t.numel, 40_000_000)
    th = host.thetas[i][:n1].copy()
    c = host.comps[i][:n1].copy() if t.comp_bits else None
    t0 = time.perf_counter()
    oracle_step_tensor(th, c, np.ascontiguousarray(host.grads[0][i][:n1]), t.theta_bits, t.comp_bits,
                       t.overlap_k, t.exp_theta, t.exp_theta, wl.lr, 1)
    t1 = time.perf_counter() - t0
    return {"value": done / t_used, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "one step of the %d largest tensors of %s (%d of %d parameters), OpenMP "
                      "static split over elements" % (k, wl.name, done, wl.numel),
            "seconds": round(t_used, 3),
            "one_thread": {"value": n1 / t1, "unit": UNIT, "cores": 1,
                           "sample": "%d parameters of the largest tensor" % n1}}


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle on the same workload, bounded sample per step."""
    if rank != 0:
        return
    from oracle import build as oracle_build
    oracle_build.build()
    from paper_1810_05486_b200 import workloads as W
    from oracle import oracle_step_tensor, oracle_max_threads
    wl = pick_workload(W, args)
    if not args.steps:
        args.steps = 3
    cores = oracle_max_threads()
    # sample: the largest tensors up to ~64M parameters per step
    order = sorted(range(len(wl.tensors)), key=lambda i: -wl.tensors[i].numel)
    pick, tot = [], 0
    for i in order:
        if tot + wl.tensors[i].numel > 64_000_000 and pick:
            break
        pick.append(i)
        tot += wl.tensors[i].numel
    thetas = [W.theta_slice(wl, i, 0, wl.tensors[i].numel, args.seed) for i in pick]
    comps = [np.zeros(wl.tensors[i].numel, W.storage_dtype(max(wl.tensors[i].comp_bits, 8)))
             for i in pick]
    grads = [W.grad_slice(wl, i, 0, 0, wl.tensors[i].numel, args.seed) for i in pick]

    def one_step():
        for j, i in enumerate(pick):
            t = wl.tensors[i]
            oracle_step_tensor(thetas[j], comps[j] if t.comp_bits else None, grads[j],
                               t.theta_bits, t.comp_bits, t.overlap_k, t.exp_theta, t.exp_theta,
                               wl.lr, cores)
    for _ in range(args.warmup):
        one_step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_step()
    dt = time.perf_counter() - t0
    value = tot * args.steps / dt
    sample = "each step = the %d largest tensors of %s (%d of %d parameters)" % (
        len(pick), wl.name, tot, wl.numel)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": wl.name, "tensors": len(wl.tensors), "parameters": wl.numel,
                       "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started without a launcher: start one rank per GPU ourselves (whole-list replicas,
        # one process per GPU, rendezvous on the loopback address)
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        os.execv(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                                  "--nproc-per-node", str(args.gpus), "--master-addr", "127.0.0.1",
                                  "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:])
    if world > 1 and args.gpus != world:
        if rank == 0:
            print("bench.py: --gpus %d does not match the %d ranks of the launcher" % (args.gpus, world),
                  file=sys.stderr)
        sys.exit(2)
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.impl == "ours":
        import torch
        if torch.cuda.device_count() < max(world, 1):
            print("bench.py: %d ranks but %d visible GPUs" % (world, torch.cuda.device_count()), file=sys.stderr)
            sys.exit(2)
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
