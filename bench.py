#!/usr/bin/env python
"""DES-LOC step benchmark: G param-updates/s and fraction of the HBM roofline on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

With --gpus N > 1 and no torchrun environment the program starts N ranks of itself (one per
GPU); under torchrun it is one of the ranks.  After the headline workload (default: workload 4)
the single-GPU run times every other workload of the benchmark definition and reports them in
"all_configs".

One "step" is one call of desloc_step(): the whole hot path (clip, desynced averaging,
optimizer update for all M worker replicas) over the full synthetic parameter/gradient set.
Steps run t = 0, 1, 2, ... under the workload's own (K_x, K_u, K_v), so the timed region mixes
sync and local steps as a run would; per-mask timings (local, x-only, all-sync) are taken
separately afterwards and reported in "by_mask".

--impl reference times the CPU oracle (the only "reference implementation" this paper has:
it ships no code) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "desloc_step_param_updates_per_s"
UNIT = "G param-updates/s"
NOMINAL_HBM_GBS = 8000.0


def bytes_per_param(w) -> int:
    """Algorithmic HBM bytes per worker-parameter per step: gradient + read and write of each
    state array (x, u, v fp32; SGDM has no v)."""
    g = 2 if w.grad_dtype == "bf16" else 4
    return g + (16 if w.opt == "sgdm" else 24)


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 200 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "200", "-i", str(self.idx)], stdout=subprocess.PIPE,
                stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for ln in self.proc.stdout:
            self.lines.append((time.time(), ln.strip()))

    def stop(self, t_begin: float, t_end: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        allrows = []
        for ts, ln in self.lines:
            f = [a.strip() for a in ln.split(",")]
            if len(f) < 9:
                continue
            allrows.append((ts, f))
        rows = [r for r in allrows if t_begin <= r[0] <= t_end + 0.2] or allrows
        for ts, f in rows:
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); pw.append(float(f[3]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w": float(np.median(pw)) if pw else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------ CPU oracle leg
def time_oracle(w, seconds_target: float = 15.0, threads: int | None = None):
    """Times the oracle as it stands on this host: `threads` threads, each stepping its own
    disjoint slice of the workload (same M, optimizer and hyper-parameters, gradients of the
    workload's distribution), one local step and one all-sync step per round."""
    import torch
    import desloc_inputs as di
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    oid = {"adam": oracle.ADAM, "adopt": oracle.ADOPT, "sgdm": oracle.SGDM}[w.opt]
    threads = threads or max(1, (os.cpu_count() or 1))
    f32 = lambda a: float(np.float32(a))

    def make_slice(n, seed):
        ws = w.replace(numel=(n,), seed=seed)
        x0 = di.init_params(ws).numpy()
        x = np.ascontiguousarray(np.tile(x0, (w.M, 1)))
        u = np.zeros_like(x)
        v = np.zeros_like(x) if w.opt != "sgdm" else None
        g = torch.empty(w.M, n, dtype=torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32)
        for m in range(w.M):
            di.fill_grads_(ws, 0, m, g[m])
        return x, u, v, np.ascontiguousarray(g.float().numpy())

    def cfg_for(K):
        return oracle.make_cfg(w.M, oid, beta1=f32(w.beta1), beta2=f32(w.beta2), eps=f32(w.eps),
                               weight_decay=f32(w.weight_decay), clip_rho=f32(w.clip_rho),
                               Kx=K[0], Ku=K[1], Kv=K[2],
                               flags=oracle.FLAG_ADOPT_NORM_CLIP if w.adopt_norm_clip else 0)

    def work(args):
        x, u, v, g = args
        # t = 1 with the workload's periods is a local step; t = 0 syncs every array
        oracle.step(cfg_for(w.K if min(w.K) > 1 else (0, 0, 0)), 1, f32(w.lr), x, u, v, g, clip_bound=1.0)
        oracle.step(cfg_for(w.K), 0, f32(w.lr), x, u, v, g, clip_bound=1.0)

    # calibrate on a small slice, then size the sample: slices of at most 4 Mi params per
    # thread (and ~8 GB in total), repeated until ~seconds_target of wall time has passed
    cal_n = 1 << 15
    sl = make_slice(cal_n, 1)
    t0 = time.perf_counter(); work(sl); dt = time.perf_counter() - t0
    per_elem = dt / (2 * cal_n * w.M)
    n = int(min(1 << 22, (8 << 30) // (threads * w.M * 16)))
    n = max(n, 1 << 12)
    reps = int(max(1, round(seconds_target / (2 * n * w.M * per_elem))))
    slices = [make_slice(n, 100 + i) for i in range(threads)]

    def work_reps(a):
        for _ in range(reps):
            work(a)

    with ThreadPoolExecutor(max_workers=threads) as ex:
        t0 = time.perf_counter()
        list(ex.map(work_reps, slices))
        dt = time.perf_counter() - t0
    updates = 2 * reps * n * w.M * threads
    return {"value": updates / dt / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{threads} threads x {n} params x M={w.M} x {2 * reps} steps (alternating "
                      f"local / all-sync) of {w.name}, {dt:.1f} s", "seconds": dt,
            "sample_params": n * threads}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    vals, info = [], None
    per_step_target = max(2.0, min(20.0, 90.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        info = time_oracle(w, seconds_target=per_step_target)
        if i >= args.warmup:
            vals.append(info)
    value = float(np.mean([v["value"] for v in vals]))
    # one full-workload step at this rate would take:
    ms_per_step = w.M * w.N / (value * 1e9) * 1e3
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": w.name, "M": w.M, "params": w.N, "opt": w.opt,
                   "note": "CPU oracle on host cores; each step is a bounded sample of the "
                           "workload; ms_per_step extrapolates to the full parameter set"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": info["cores"], "kind": "oracle",
                         "sample": info["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------ GPU leg
class Resident:
    """One workload resident in HBM: M replicas of x, u, v, one gradient set, and views per
    tensor.  torch is used for the memory and the stream only."""

    def __init__(self, w, dev, rank=0):
        import torch
        import desloc_inputs as di
        self.w, self.dev = w, dev
        align = 4
        self.nflat = di.flat_size(w.numel, align)
        self.offs = di.offsets_of(w.numel, align)
        gdt = torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32
        x0 = di.init_params(w.replace(seed=w.seed + rank), device=dev, align=align)
        self.X = [x0.clone() for _ in range(w.M - 1)] + [x0]
        self.U = [torch.zeros(self.nflat, dtype=torch.float32, device=dev) for _ in range(w.M)]
        self.V = [torch.zeros(self.nflat, dtype=torch.float32, device=dev) for _ in range(w.M)] \
            if w.opt != "sgdm" else None
        self.G = [torch.empty(self.nflat, dtype=gdt, device=dev) for _ in range(w.M)]
        for m in range(w.M):
            di.fill_grads_(w.replace(seed=w.seed + rank), 0, m, self.G[m], align=align)

    def views(self, bufs):
        return [[b[o:o + n] for o, n in zip(self.offs, self.w.numel)] for b in bufs]

    def engine(self, d, w=None, post=False):
        w = w or self.w
        flags = d.DESLOC_FLAG_ADOPT_NORM_CLIP if w.adopt_norm_clip else 0
        if post:
            flags |= d.DESLOC_FLAG_POST_AVERAGE
        return d.DesLoc(self.views(self.X), self.views(self.U),
                        self.views(self.V) if self.V is not None else None, opt=w.opt,
                        grad_dtype=w.grad_dtype, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                        weight_decay=w.weight_decay, clip_rho=w.clip_rho, K=w.K, flags=flags)


def timed_loop(stream, fn, reps):
    """CUDA-event time per call of fn over `reps` back-to-back calls, in ms."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(reps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def timed_median(stream, fn, steps=20, repeats=5):
    """Median (and spread) over `repeats` CUDA-event timings of `steps` back-to-back calls."""
    ms = sorted(timed_loop(stream, fn, steps) for _ in range(repeats))
    return ms[len(ms) // 2], {"ms_min": ms[0], "ms_max": ms[-1], "steps_per_repeat": steps, "repeats": repeats}


def rates(w, ms, peak, nbytes=None):
    nbytes = nbytes if nbytes is not None else w.M * w.N * bytes_per_param(w)
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"ms": ms, "gups": w.M * w.N / (ms * 1e-3) / 1e9, "gbs": gbs,
            "frac_of_measured_peak": gbs / peak, "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS}


def per_mask_and_variants(w, eng, g, stream, peak, reps):
    """Local, x-only and all-sync steps timed in isolation (median of five timings of at least
    twenty back-to-back steps of the same mask), then the norm-clipped step (one more read of the
    gradients) and the diagnostics step (same bytes as the plain step)."""
    out = {"by_mask": {}}
    for mk in [0, 1, 3 if w.opt == "sgdm" else 7]:
        if w.M == 1 and mk:
            continue
        fn = lambda: eng.step_masked(mk, w.lr, g, clip_bound=1.0)
        fn(); fn()
        ms, spread = timed_median(stream, fn, steps=max(reps, 20), repeats=5)
        out["by_mask"][str(mk)] = dict(rates(w, ms, peak), **spread)
    gbytes = 2 if w.grad_dtype == "bf16" else 4
    fn = lambda: eng.step_normclip(1, w.lr, g, 1.0, clip_bound=1.0)
    fn(); fn()
    nc_bytes = w.M * w.N * (bytes_per_param(w) + gbytes)
    ms, spread = timed_median(stream, fn, steps=max(reps, 20), repeats=3)
    out["normclip_step"] = dict(rates(w, ms, peak, nc_bytes), launches_per_step=3,
                                algorithmic_bytes=nc_bytes, **spread)
    fn = lambda: eng.step_diag(1, w.lr, g, clip_bound=1.0)
    fn(); fn()
    ms, spread = timed_median(stream, fn, steps=max(reps, 20), repeats=3)
    out["diag_step"] = dict(rates(w, ms, peak), **spread,
                            note="same step, plus per-(worker, tensor) norms of g, x, d fused in")
    return out


def graph_window(w, eng, g, stream, eager_us):
    """Small, launch-bound workloads: a CUDA graph of one lcm(K) window of steps."""
    import math
    import torch
    L = math.lcm(*[k for k in w.K if k > 0])
    if L > 256:
        return None
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for t in range(L):
                eng.step(t, w.lr, g, clip_bound=w.clip_bound(t))
    stream.wait_stream(side)
    for _ in range(3):
        graph.replay()
    us = timed_loop(stream, graph.replay, 50) * 1e3 / L
    return {"window_steps": L, "us_per_step": us, "gups": w.M * w.N / (us * 1e-6) / 1e9,
            "eager_us_per_step": eager_us}


PARITY_TESTS = {
    "cfg1_adam_n4096": "tests/test_parity_gpu.py::test_cfg1_adam_n4096_full_run (every element, T = 64)",
    "cfg2_adam_135m": "tests/test_parity_fullsize_gpu.py::test_fullsize_sampled_parity[cfg2_adam_135m-*]",
    "cfg3_adopt_360m": "tests/test_parity_fullsize_gpu.py::test_fullsize_sampled_parity[cfg3_adopt_360m-*]",
    "cfg4_adam_1p7b": "tests/test_parity_fullsize_gpu.py::test_fullsize_sampled_parity[cfg4_adam_1p7b-*]",
}


def parity_test_of(name):
    """The -m gpu test that checks this workload at full size, in this launch configuration,
    against the oracle (this program may run the oracle only for its CPU-baseline leg)."""
    return PARITY_TESTS.get(
        name, f"tests/test_parity_fullsize_gpu.py::test_fullsize_sampled_parity[{name}-*]")


def time_config(d, w, res, steps, warmup, peak, rank=0, world=1, barrier=None, sampler=None,
                post=False):
    """The timed region of one workload: exactly `steps` steps under its own schedule, placed so
    that an x-sync step falls inside; then the per-mask and variant timings."""
    import torch
    dev = res.dev
    stream = torch.cuda.current_stream(dev)
    eng = res.engine(d, w, post)
    g = eng.bind_grads(res.views(res.G))
    step = lambda t: eng.step(t, w.lr, g, clip_bound=w.clip_bound(t))
    t_next = 0
    for _ in range(max(3, warmup)):
        step(t_next); t_next += 1
    barrier()
    Kx = w.K[0]
    if Kx > 1:
        t_next = max(t_next, (t_next // Kx + 1) * Kx - steps // 2)
    if sampler is not None:
        sampler.start()
        time.sleep(0.3)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    masks = []
    launches0 = eng.launches()
    barrier()
    wall0 = time.time()
    ev[0].record(stream)
    for i in range(steps):
        masks.append(step(t_next)); t_next += 1
        ev[i + 1].record(stream)
    barrier()
    wall1 = time.time()
    launches = eng.launches() - launches0
    total_ms = ev[0].elapsed_time(ev[-1])
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    clocks = sampler.stop(wall0, wall1) if sampler is not None else None
    total_ms = d.dist.max_over_ranks(total_ms, dev)
    launches = d.dist.sum_over_ranks(launches, dev)
    out = {"eng": eng, "g": g, "masks": masks, "per_step": per_step, "total_ms": total_ms,
           "launches": launches, "clocks": clocks,
           "value": world * w.M * w.N * steps / (total_ms * 1e-3) / 1e9}
    out.update(per_mask_and_variants(w, eng, g, stream, peak, max(3, min(steps, 10))))
    return out


def config_entry(w, r, steps):
    ms = r["total_ms"] / steps
    e = {"workload": w.name, "opt": w.opt, "M": w.M, "params": w.N, "K": list(w.K),
         "grad_dtype": w.grad_dtype, "steps": steps, "ms_per_step": ms, "value": r["value"],
         "unit": UNIT, "masks_in_timed_region": r["masks"], "by_mask": r["by_mask"],
         "normclip_step": r["normclip_step"], "diag_step": r["diag_step"],
         "parity_test": parity_test_of(w.name)}
    gbs = w.M * w.N * bytes_per_param(w) / (ms * 1e-3) / 1e9
    e["gbs"] = gbs
    e["frac_of_nominal_8tbs"] = gbs / NOMINAL_HBM_GBS
    return e


def run_all_configs(d, dev, steps, warmup, peak, skip):
    """Every other workload of the benchmark definition, one after the other on the same GPU:
    workload 1 (latency-bound: eager and CUDA-graph microseconds per step), workload 2,
    workload 3, and workload 5's two optimizers under its three schedules."""
    import torch
    import desloc_inputs as di
    stream = torch.cuda.current_stream(dev)
    out = []
    no_barrier = torch.cuda.synchronize
    groups = [["cfg1_adam_n4096"], ["cfg2_adam_135m"], ["cfg3_adopt_360m"], ["cfg4_adam_1p7b"],
              ["cfg5_sgdm_ddp", "cfg5_sgdm_local", "cfg5_sgdm_desloc"],
              ["cfg5_adam_ddp", "cfg5_adam_local", "cfg5_adam_desloc"]]
    for names in groups:
        names = [n for n in names if n != skip]
        if not names:
            continue
        w0 = di.WORKLOADS[names[0]]
        free, _ = torch.cuda.mem_get_info(dev)
        need = w0.N * w0.M * (14 if w0.opt != "sgdm" else 10) + (4 << 30)
        if free < need:
            out += [{"workload": n, "skipped": f"needs {need >> 30} GiB, {free >> 30} GiB free"}
                    for n in names]
            continue
        res = Resident(w0, dev)            # the schedules of a group share one resident state
        for n in names:
            w = di.WORKLOADS[n]
            r = time_config(d, w, res, steps, warmup, peak, barrier=no_barrier)
            e = config_entry(w, r, steps)
            e["frac_of_measured_peak"] = e["gbs"] / peak
            if w.M * w.N * 14 < (126 << 20) and w.M * len(w.numel) <= 32 and min(w.K) > 0:
                e["graph_window"] = graph_window(w, r["eng"], r["g"], stream,
                                                 r["total_ms"] * 1e3 / steps)
                e["note"] = "fits in L2: latency-bound, microseconds per step are the figure"
            r["eng"].close()
            out.append(e)
        del res, r
        torch.cuda.empty_cache()
    return out


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    import paper_2505_22549_b200 as d

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the DES-LOC step has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peak, peak_kind = measured_peak()
    # ---- resident state: every rank holds its own M replicas of the whole tensor list -------
    res = Resident(w, dev, rank)
    bpp = bytes_per_param(w)
    launch_bytes = w.M * w.N * bpp
    stream = torch.cuda.current_stream(dev)
    r = time_config(d, w, res, args.steps, args.warmup, peak, rank, world, barrier,
                    ClockSampler(local_rank) if rank == 0 else None, args.post_average)
    eng, g = r["eng"], r["g"]

    resident = w.M * w.N * (bpp - (8 if w.opt == "sgdm" else 12))
    graph_info = None
    if resident < (126 << 20) and w.M * len(w.numel) <= 32 and min(w.K) > 0:
        graph_info = graph_window(w, eng, g, stream, r["total_ms"] * 1e3 / args.steps)

    # ---- roofline of the dominant kernel (the local-step kernel), from the timed region -------
    local_ms = [ms for ms, mk in zip(r["per_step"], r["masks"]) if mk == 0] or r["per_step"]
    avg_local_ms = float(np.mean(local_ms))
    achieved = launch_bytes / (avg_local_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak,
                "traffic": (TRAFFIC_PER_ALGORITHMIC_BYTE[(w.opt, w.M)] * launch_bytes
                            if (w.opt, w.M) in TRAFFIC_PER_ALGORITHMIC_BYTE else None),
                "traffic_source": "ncu dram__bytes_read+write on a 44M-parameter case, scaled by "
                                  "parameter count (profiles/)",
                "peak_source": f"{peak_kind} copy bandwidth", "kernel": "desloc_step_kernel (local step)",
                "algorithmic_bytes_per_launch": launch_bytes,
                "frac_of_nominal_8tbs": achieved / NOMINAL_HBM_GBS,
                "avg_launch_ms": avg_local_ms, "launches_averaged": len(local_ms)}

    # ---- end to end: gradients start in pinned host memory, a result is read back -------------
    e2e = None if args.skip_e2e else run_e2e(args, w, eng, res.G, res.X, res.offs, dev, world, barrier)
    eng.close()
    headline = config_entry(w, r, args.steps)
    value, total_ms, launches, clocks = r["value"], r["total_ms"], r["launches"], r["clocks"]
    del res, r, eng, g
    torch.cuda.empty_cache()

    all_configs = None
    if rank == 0 and world == 1 and not args.skip_all_configs:
        all_configs = run_all_configs(d, dev, max(4, min(args.steps, 20)), args.warmup, peak,
                                      skip=w.name)

    if rank == 0:
        cpu = (time_oracle(w, seconds_target=15.0) if not args.skip_cpu else
               {"value": None, "unit": UNIT, "cores": 0, "kind": "oracle", "sample": "skipped"})
        if not args.skip_cpu:   # the same routine on one core, for the per-core figure
            cpu["single_thread"] = time_oracle(w, seconds_target=4.0, threads=1)["value"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": w.name, "opt": w.opt, "M": w.M, "params": w.N,
                       "tensors": len(w.numel), "grad_dtype": w.grad_dtype, "K": list(w.K),
                       "resident_gb": resident / 1e9,
                       "l2": ("inputs larger than L2 (no flush needed)" if resident > (126 << 20)
                              else "workload fits in L2: latency-bound, see graph_window"),
                       "parallelism": f"{world} independent replica set(s), no collective",
                       "ordering": "post-average" if args.post_average else "pre-average",
                       "masks_in_timed_region": headline["masks_in_timed_region"],
                       "parity_test": headline["parity_test"]},
            "roofline": roofline, "by_mask": headline["by_mask"],
            "normclip_step": headline["normclip_step"], "diag_step": headline["diag_step"],
            "graph_window": graph_info,
            "cpu_baseline": {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample",
                                                 "single_thread") if k in cpu},
            "e2e": e2e, "gpu_launches": launches, "clocks": clocks, "all_configs": all_configs,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


# DRAM bytes (read + write) per algorithmic byte of one launch of the local-step kernel, from
# the ncu captures summarised under profiles/ (44 M-parameter stand-ins of the workloads: the
# full sizes are too large for a multi-pass capture; each byte is touched once, so traffic grows
# in proportion to the parameter count).  Keyed by (optimizer, M).
TRAFFIC_PER_ALGORITHMIC_BYTE = {("adam", 4): 0.9875, ("adopt", 8): 0.9937}


def run_e2e(args, w, eng, G, X, offs, dev, world, barrier):
    """Same step, but every step's gradients are copied from pinned host memory first and a
    small result (worker 0's last tensor of x) is read back to the host afterwards."""
    import torch
    esz = G[0].element_size()
    nflat = G[0].numel()
    h2d = w.M * nflat * esz
    try:
        import psutil
        avail = psutil.virtual_memory().available
    except Exception:
        avail = 0
    share = h2d + (8 << 30) < avail / max(1, world)
    try:
        if share:
            H = [torch.empty(nflat, dtype=G[0].dtype).pin_memory() for _ in range(w.M)]
        else:
            H = [torch.empty(nflat, dtype=G[0].dtype).pin_memory()] * w.M
        for h, g in zip(H[:w.M if share else 1], G):
            h.copy_(g)
    except Exception as ex:  # not enough pinnable memory on this host
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 0,
                "note": f"pinned host buffer unavailable: {type(ex).__name__}"}
    stream = torch.cuda.current_stream(dev)
    views = lambda bufs: [[b[o:o + n] for o, n in zip(offs, w.numel)] for b in bufs]
    gv = views(G)
    last = (offs[-1], w.numel[-1])
    out = torch.empty(last[1], dtype=torch.float32).pin_memory()
    steps = max(2, min(args.steps, 6))
    t_next = 1000

    hv = views(H)

    def one(t):
        # desloc_step_host: the C-ABI call that takes HOST gradient buffers, copies them group by
        # group and pipelines the step behind the copies; then the result read-back
        eng.step_host(t, w.lr, hv, gv, clip_bound=w.clip_bound(t))
        out.copy_(X[0][last[0]:last[0] + last[1]], non_blocking=True)
        stream.synchronize()

    one(t_next); t_next += 1
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        one(t_next); t_next += 1
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    import paper_2505_22549_b200 as d
    ms = d.dist.max_over_ranks(ms, dev)
    return {"value": world * w.M * w.N * steps / (ms * 1e-3) / 1e9, "unit": UNIT,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": last[1] * 4, "steps": steps,
            "ms_per_step": ms / steps,
            "note": "desloc_step_host: gradients copied from pinned host memory every step, "
                    "pipelined with the step in 8 tensor groups; result slice read back"
                    + ("" if share else " (one host buffer re-sent for each worker)")}


def launcher_command(gpus: int, argv, port: int | None = None):
    """The command that starts `gpus` ranks of this program on this node (one process per GPU,
    rendezvous on 127.0.0.1), as the benchmark contract launches it."""
    if port is None:
        import socket
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port),
            os.path.abspath(__file__)] + list(argv)


def main(argv=None):
    argv = sys.argv[1:] if argv is None else list(argv)
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4_adam_1p7b")
    ap.add_argument("--post-average", action="store_true",
                    help="average after the update (ordering of Algorithms 4-5) instead of before")
    ap.add_argument("--skip-e2e", action="store_true", help="omit the host-buffer leg (profiling)")
    ap.add_argument("--skip-cpu", action="store_true", help="omit the CPU oracle leg (profiling)")
    ap.add_argument("--skip-all-configs", action="store_true",
                    help="time the named workload only, not the other workloads after it")
    args = ap.parse_args(argv)
    import desloc_inputs as di
    w = di.WORKLOADS[args.workload]
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain program: become N ranks, one per GPU (replicas only, no collective
        # on the data path; NCCL carries the barrier and the max over ranks of the timing)
        return subprocess.call(launcher_command(args.gpus, argv))
    if args.impl == "reference":
        return run_reference(args, w)
    return run_ours(args, w)


if __name__ == "__main__":
    sys.exit(main())
