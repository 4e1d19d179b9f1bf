#!/usr/bin/env python
"""Throughput of the C-step on B200: parameters per second and achieved HBM GB/s.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 5] [--impl ours|reference]

A step is one whole C-step call (ranking, projection, multiplier update) over
one synthetic weight set. With N > 1 (launched by torch.distributed.run, one
process per GPU) every rank runs the same workload on its own GPU: the method
ranks one global list on one GPU, so the ranks are independent replicas and
`value` is the sum of what they processed over the slowest rank's time.

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

L2_BYTES = 126 * 1024 * 1024
NOMINAL_HBM_GBS = 8000.0      # the B200's nominal HBM3e rate, beside the measured copy rate


def ncu_traffic_per_param(kernel: str, fuse) -> "float | None":
    """dram__bytes_read.sum + dram__bytes_write.sum per parameter of the projection kernel, from the
    ncu captures summarised under profiles/ (taken on smaller cases; the traffic grows in proportion
    to the parameters). profiles/traffic.json holds one entry per (kernel, fuse); an entry is null
    once the kernel has changed since its capture."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            table = json.load(f)
        return table.get("%s|%s" % (kernel, "+".join(fuse)))
    except Exception:
        return None


FALLBACK_HBM_GBS = 6650.0


def algorithmic_bytes_per_param(fuse) -> int:
    """Minimal traffic of one C-step: read w and lambda, write theta, mask, lambda
    (+ the penalty gradient, + the fp16 copy when they are asked for)."""
    b = 4 + 4 + 4 + 1 + 4
    if "penalty" in fuse:
        b += 4
    return b


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier copy measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def dist_max(value: float, world: int, device=None) -> float:
    """Largest `value` over the ranks of the default process group (identity for one rank)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(total_ms_local: float, steps: int, n_params: int, world: int, device=None):
    """Whole-job params/s of `world` independent replicas: what all ranks processed over the
    slowest rank's time. Returns (value, ms_per_step)."""
    total_ms = dist_max(total_ms_local, world, device)
    ms_per_step = total_ms / steps
    return world * n_params / (ms_per_step * 1e-3), ms_per_step


def workload_name(ws) -> str:
    return "%s: %s s=%.2f fuse=%s, %d tensors, %d params" % (
        ws.name, ws.op, ws.sparsity, "+".join(ws.fuse) or "none", len(ws.w), ws.numel)


# --------------------------------------------------------------------------- oracle arm
def time_oracle(ws, steps: int, warmup: int):
    import oracle
    for _ in range(warmup):
        oracle.run_config(ws)
    t0 = time.perf_counter()
    out = None
    for _ in range(steps):
        out = oracle.run_config(ws)
    dt = time.perf_counter() - t0
    return dt / max(steps, 1), out


def run_reference(args):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_1911_02497_b200 import workloads as W
    scale = args.ref_scale
    if scale <= 0.0:
        # the whole configuration per step when K + W oracle calls end within about two minutes
        # (the oracle sorts about 3e7 units per second), else every dimension shrunk to fit
        n_full = W.config_numel(args.config)
        calls = max(args.steps + args.warmup, 1)
        budget = 150.0 * 3.0e7 / calls
        scale = 1.0 if n_full <= budget else max(0.05, (budget / n_full) ** 0.5)
    ws = W.config(args.config, scale=scale)
    sec, _ = time_oracle(ws, args.steps, args.warmup)
    value = ws.numel / sec
    sample = ("the whole configuration %s (%d params), one oracle call per step" % (args.config, ws.numel)
              if scale == 1.0 else
              "config %s with every dimension scaled by %.3g (%d params), one oracle call per step" % (
                  args.config, scale, ws.numel))
    line = {"impl": "reference", "metric": "cstep_params_per_s", "value": value, "unit": "params/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_name(ws), "sample": sample},
            "cpu_baseline": {"value": value, "unit": "params/s", "cores": 1, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "params/s", "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def run_lstep(args, ws, ctx, local, world):
    """Standalone timing of the fused penalty-gradient + optimizer step (not the headline)."""
    import torch
    from paper_1911_02497_b200 import cstep
    dev = torch.device("cuda", local)
    adam = args.op == "lstep_adam"
    mk = lambda a: torch.from_numpy(np.ascontiguousarray(a).reshape(-1)).to(dev)
    w = [mk(a) for a in ws.w]
    th = [torch.where(t.abs() > 0.05, t, torch.zeros_like(t)) for t in w]
    lam = [mk(a) for a in ws.lam]
    grad = [torch.randn_like(t) for t in w]
    b1 = [torch.zeros_like(t) for t in w]
    b2 = [torch.zeros_like(t) for t in w] if adam else None
    tab = cstep.opt_table(w, th, lam, grad, b1, b2)
    N = ws.numel
    bpp = 36 if adam else 28             # read w, theta, lambda, grad, moments; write w, moments
    kw = dict(kind="adam", lr=1e-4, step=3) if adam else dict(kind="sgd", lr=0.1, momentum=0.9)
    for _ in range(max(args.warmup, 3)):
        ctx.lstep_update(tab, len(w), ws.mu, **kw)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = ctx.launch_count()
    a.record()
    for _ in range(args.steps):
        ctx.lstep_update(tab, len(w), ws.mu, **kw)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.steps
    peak, src = measured_peak()
    gbs = N * bpp / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "lstep_params_per_s", "value": N / (ms * 1e-3), "unit": "params/s", "n_gpus": world,
                      "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
                      "higher_is_better": True, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": "%s on %s" % (args.op, workload_name(ws))},
                      "gpu_launches": ctx.launch_count() - l0,
                      "roofline": {"bound": "hbm", "kernel": "k_" + args.op, "achieved": gbs, "peak": peak,
                                   "unit": "GB/s", "frac": gbs / peak, "traffic": None, "peak_source": src,
                                   "algorithmic_bytes_per_launch": N * bpp}}))
    return 0


def run_thin(args, ws, ctx, local, world):
    """Standalone timing of thinning after filter pruning (not the headline): zero-filter flags,
    compaction along the chain of conv layers, and the non-zero count of the whole list."""
    import torch
    from paper_1911_02497_b200.device_set import DeviceSet
    ds = DeviceSet(ws.w, ws.lam, device="cuda:%d" % local)
    ds.run(ctx, "filter", ws.sparsity, ws.mu, ("lambda",), ws.block)
    convs = [t for t in range(len(ws.w)) if len(ws.shapes[t]) == 4]
    keep = [torch.empty(ws.shapes[t][0], dtype=torch.uint8, device=ds.device) for t in convs]
    dst = [torch.empty(int(np.prod(ws.shapes[t])), dtype=torch.float32, device=ds.device) for t in convs]
    dims = [torch.zeros(2, dtype=torch.int64, device=ds.device) for t in convs]
    counts = torch.zeros(len(ws.w) + 1, dtype=torch.int64, device=ds.device)
    flush = torch.empty(2 * L2_BYTES // 4, dtype=torch.float32, device=ds.device)

    layers = [dict(src=ds.theta[t], d0=ws.shapes[t][0], d1=ws.shapes[t][1], inner=ws.shapes[t][2] * ws.shapes[t][3],
                   keep0=keep[i], remove_axis0=True, keep1_from=i - 1, dst=dst[i], dims_out=dims[i])
              for i, t in enumerate(convs)]

    def step_per_layer():
        for i, t in enumerate(convs):
            Fo, Ci, kh, kw = ws.shapes[t]
            ctx.thin_flags(ds.theta[t], Fo, Ci, kh * kw, 0, keep[i])
            ctx.thin_compact(ds.theta[t], Fo, Ci, kh * kw, keep[i], keep[i - 1] if i else None, dst[i], dims[i])
        ctx.count_nonzero(ds.theta, counts)

    def step():
        ctx.thin_list(layers)
        ctx.count_nonzero(ds.theta, counts)

    def timed(fn):
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        l0 = ctx.launch_count()
        for a, b in ev:
            flush.fill_(1.0)
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in ev) / args.steps, (ctx.launch_count() - l0) // args.steps

    ms_layer, launches_layer = timed(step_per_layer)
    ms, launches = timed(step)
    N = sum(int(np.prod(ws.shapes[t])) for t in convs)
    kept = sum(int(d[0]) * int(d[1]) * ws.shapes[t][2] * ws.shapes[t][3] for d, t in zip(dims, convs))
    algo = 4 * N + 8 * kept + 4 * ws.numel        # flags read theta; compaction reads and writes the kept part; count reads
    peak, src = measured_peak()
    gbs = algo / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "thin_params_per_s", "value": ws.numel / (ms * 1e-3), "unit": "params/s",
                      "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
                      "higher_is_better": True, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": "thin (one list call: flags + chain compaction; non-zero count) on %s" % workload_name(ws),
                                 "l2": "L2 flushed between steps by writing a 252 MB buffer"},
                      "gpu_launches": launches * args.steps, "kept_params": kept,
                      "per_layer_calls": {"ms_per_step": ms_layer, "launches_per_step": launches_layer}, "nonzero": int(counts[-1]),
                      "roofline": {"bound": "hbm", "kernel": "thin step", "achieved": gbs, "peak": peak, "unit": "GB/s",
                                   "frac": gbs / peak, "traffic": None, "peak_source": src,
                                   "algorithmic_bytes_per_launch": algo}}))
    return 0


# --------------------------------------------------------------------------- CUDA arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_1911_02497_b200 import cstep, workloads as W
    from paper_1911_02497_b200.device_set import DeviceSet

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the C-step has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    ws = W.config(args.config, scale=args.scale)
    if args.block_size and ws.op == "block":
        ws.block = (args.block_size, args.block_size)
        ws.name += "-bs%d" % args.block_size
    if args.op:      # a standalone operation on the configuration's weight set (not the headline)
        ws.op = args.op
        ws.fuse = ("lambda", "penalty") if args.op == "lagrange" else ("lambda",)
        args.skip_cpu = True
    fuse = ws.fuse + (("no_sampling",) if args.no_sampling else ())
    with_grad = "penalty" in ws.fuse
    ds = DeviceSet(ws.w, ws.lam, device="cuda:%d" % local, with_grad=with_grad, with_theta_h=False)
    ctx = cstep.Context(local)
    N = ws.numel
    bpp = algorithmic_bytes_per_param(ws.fuse)
    if args.op == "lagrange":
        bpp = 4 + 4 + 4 + 4 + 4          # read w, theta, lambda; write lambda, g
    if args.op in ("lstep_sgd", "lstep_adam"):
        return run_lstep(args, ws, ctx, local, world)
    if args.op == "thin":
        return run_thin(args, ws, ctx, local, world)
    stream = torch.cuda.current_stream()

    calls = [0]

    def step():
        # The sample positions of the single-pass path come from the context's seed; the step time
        # depends a little on how close the sample's guess lands to the threshold (how many
        # provisional decisions have to be rewritten), so the seed changes from step to step and
        # the mean is one over seeds, not the luck of one draw.
        ctx.set_seed(1000 + calls[0])
        calls[0] += 1
        ds.run(ctx, ws.op, ws.sparsity, ws.mu, fuse, ws.block)

    flush = None
    if N * 8 < 2 * L2_BYTES:       # small workloads fit the L2: evict it between steps
        flush = torch.empty(2 * L2_BYTES // 4, dtype=torch.float32, device=ds.device)

    def between_steps():
        ds.reset_lambda()
        if flush is not None:
            flush.fill_(1.0)

    for _ in range(max(args.warmup, 3)):
        between_steps()
        step()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(args.steps)]
    launches0 = ctx.launch_count()
    barrier()
    with ClockSampler(physical_gpu_index(local)) as clocks:
        for a, b in ev:
            between_steps()
            a.record(stream)
            step()
            b.record(stream)
        barrier()
    launches = ctx.launch_count() - launches0
    per_step_ms = [a.elapsed_time(b) for a, b in ev]
    value, ms_per_step = replica_throughput(float(sum(per_step_ms)), args.steps, N, world, ds.device)
    # the same steps once more without the flush: what a caller sees whose weights are still in the L2
    warm_ms = None
    if flush is not None and rank == 0:
        evw = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in evw:
            ds.reset_lambda()
            a.record(stream)
            step()
            b.record(stream)
        torch.cuda.synchronize()
        warm_ms = [a.elapsed_time(b) for a, b in evw]

    line = None
    if rank == 0:
        res = ctx.get_result() if ws.op in ("prune", "filter", "block") else None
        # second pass over the same call with an event pair around every kernel
        ctx.profile_enable(True)
        for _ in range(args.steps):
            between_steps()
            step()
        torch.cuda.synchronize()
        prof = ctx.profile_read()
        ctx.profile_enable(False)
        peak, peak_src = measured_peak()
        kernels = {k: {"launches": n, "avg_us": 1e3 * ms / n} for k, (n, ms) in prof.items()}
        # the kernel that does the projection (reads w, lambda; writes theta, mask, lambda):
        # its algorithmic bytes are the step's
        names = ("k_fused", "k_apply", "k_quantize", "k_lagrange", "k_select_all", "k_prune_small")   # the last two: one-launch routes
        movers = {k: v for k, v in prof.items() if k.startswith(names)
                  and v[1] / v[0] > 0.02}          # launches that return at once do not count
        if not movers:                             # small sets: every launch is short
            movers = {k: v for k, v in prof.items() if k.startswith(names)}
        dom = max(movers.items(), key=lambda kv: kv[1][1])
        dom_name, (dom_n, dom_ms) = dom
        achieved = (N * bpp) / (dom_ms / dom_n * 1e-3) / 1e9
        traffic = None
        per_param = ncu_traffic_per_param(dom_name, ws.fuse)
        if args.scale == 1.0 and per_param is not None:
            traffic = per_param * N
        step_gbs = (N * bpp) / (ms_per_step * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": dom_name, "achieved": achieved, "peak": peak,
                    "unit": "GB/s", "frac": achieved / peak, "traffic": traffic,
                    "peak_source": peak_src, "algorithmic_bytes_per_launch": N * bpp,
                    "frac_nominal": achieved / NOMINAL_HBM_GBS, "peak_nominal": NOMINAL_HBM_GBS,
                    "step_achieved": step_gbs, "step_frac": step_gbs / peak,
                    "step_frac_nominal": step_gbs / NOMINAL_HBM_GBS,
                    "kernels": kernels}

        # end to end: host buffers through the host entry point (pinned memory)
        hw = [torch.from_numpy(a).pin_memory() for a in ws.w]
        hl = [torch.from_numpy(a.copy()).pin_memory() for a in ws.lam]
        ht = [torch.empty_like(a).pin_memory() for a in hw]
        hm = [torch.empty(a.shape, dtype=torch.uint8).pin_memory() for a in hw]
        hg = [torch.empty_like(a).pin_memory() for a in hw] if with_grad else None
        tab = cstep.tensor_table(hw, hl, ht, hm, hg, None, shapes=ws.shapes)
        opn = {"prune": cstep.OP_PRUNE, "filter": cstep.OP_FILTER, "block": cstep.OP_BLOCK,
               "quantize": cstep.OP_QUANTIZE, "lagrange": cstep.OP_LAGRANGE}[ws.op]
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        lam0 = [torch.from_numpy(a.copy()) for a in ws.lam]

        def e2e_step():
            ctx.cstep_host(opn, tab, len(hw), ws.sparsity, ws.mu, ws.block[0], ws.block[1], fuse)

        e2e_step()
        e2e_ms = 0.0
        for _ in range(e2e_steps):
            for a, b in zip(hl, lam0):
                a.copy_(b)
            t0 = time.perf_counter()
            e2e_step()                       # returns after the stream has finished
            e2e_ms += (time.perf_counter() - t0) * 1e3
        e2e_ms /= e2e_steps
        h2d = 8 * N
        d2h = (9 + (4 if with_grad else 0)) * N
        e2e = {"value": N / (e2e_ms * 1e-3), "unit": "params/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps}

        # CPU oracle on the same workload (bounded), and a parity check of this very run
        cpu = None
        if not args.skip_cpu:
            small = N > args.cpu_max_params
            ows = W.config(args.config, scale=args.cpu_scale * args.scale) if small else ws
            sec, out = time_oracle(ows, 1, 0)
            cpu = {"value": ows.numel / sec, "unit": "params/s", "cores": 1, "kind": "oracle",
                   "sample": ("whole workload, one call" if not small else
                              "config scaled by %.3g (%d params), one call" % (args.cpu_scale, ows.numel)),
                   "seconds": sec}
            if not small:
                got_mask = [m.cpu().numpy().reshape(s) for m, s in zip(hm, ws.shapes)]
                cpu["parity_mask_equal"] = bool(all(np.array_equal(a, b) for a, b in zip(got_mask, out.mask)))
                key_ok = res.tau_key == out.result.tau_key
                if ws.op == "filter" and not key_ok:
                    # filter norms: the fp64 summation order differs from the oracle's sequential one
                    a, b = (np.array([k], np.uint64).view(np.float64)[0] for k in (res.tau_key, out.result.tau_key))
                    key_ok = bool(abs(a - b) <= 1e-12 * abs(b))
                    cpu["tau_key_rel_err"] = float(abs(a - b) / abs(b)) if b else 0.0
                cpu["parity_tau_equal"] = bool(key_ok and res.tau_id == out.result.tau_id)
        line = {"metric": "cstep_params_per_s", "value": value, "unit": "params/s", "n_gpus": world,
                "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic",
                "config": {"workload": workload_name(ws),
                           "l2": ("inputs (%.0f MB) larger than L2" % (N * 8 / 1e6)) if flush is None
                           else "L2 flushed between steps by writing a 252 MB buffer",
                           "parallelism": "replicas" if world > 1 else "single GPU",
                           "lambda": "restored between steps outside the timed windows",
                           "seed": "sample seed 1000 + call number (a new one every step)"},
                "ms_per_step_median": float(np.median(per_step_ms)), "ms_per_step_min": float(min(per_step_ms)),
                "l2_warm": None if warm_ms is None else {"ms_per_step": float(np.mean(warm_ms)),
                                                         "ms_per_step_median": float(np.median(warm_ms)),
                                                         "ms_per_step_min": float(min(warm_ms)),
                                                         "note": "same steps without the L2 flush (rank 0)"},
                "hbm_gbs": (N * bpp) / (ms_per_step * 1e-3) / 1e9,
                "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": launches,
                "roofline": roofline, "cpu_baseline": cpu,
                "result": None if res is None else {"passes": res.passes, "sampled": res.sampled,
                                                     "n_candidates": res.n_candidates, "n_units": res.n_units,
                                                     "n_repaired": res.n_repaired}}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="5", help="1..5 or 5t; 5 (the largest) is the headline")
    ap.add_argument("--no-sampling", action="store_true")
    ap.add_argument("--op", default=None, choices=["prune", "quantize", "lagrange", "lstep_sgd", "lstep_adam", "thin"],
                    help="time a standalone operation on the configuration's weights instead of its C-step")
    ap.add_argument("--block-size", type=int, default=0, help="block side for the block configs (default 4)")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-max-params", type=int, default=200_000_000)
    ap.add_argument("--cpu-scale", type=float, default=0.25)
    ap.add_argument("--ref-scale", type=float, default=0.0,
                    help="reference arm: shrink every dimension; 0 = the whole configuration when that fits two minutes")
    ap.add_argument("--scale", type=float, default=1.0,
                    help="shrink every dimension (profiling captures only; not a bench value)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
