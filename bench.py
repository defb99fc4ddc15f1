#!/usr/bin/env python
"""Throughput of the n-softsync parameter-server update on B200.

A step is one pass of the whole server path for one weight update of the large-net softsync
workload (60,965,224 fp32 parameters, lambda = 18 learners, n = 4, c = 4 fp32 gradients per
update): the learners' timestamp pulls, c gradient pushes (timestamp check, staleness, grouping),
the scale table, ONE fused sumGradients+applyUpdate kernel launch, and the timestamp advance.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints one JSON line.  `value` is gradient elements applied per second (c * N * K / time) with
the gradients already resident in HBM; `e2e` is the same metric with every gradient copied from
pinned host memory and the updated weights copied back to the host inside the timed region.
With N > 1 (torchrun, one process per GPU) every rank runs an independent server replica: the
path has no exchange step, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from workloads import arrivals, configs, generators as G

METRIC = "ps_gradient_elements_per_sec"
UNIT = "grad-elements/s"
FALLBACK_HBM_GBS = 6650.0
POOL_BUFFERS = 8
L2_BYTES = 126 * 1024 * 1024


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(num_params: int, entries: int, grad_bytes: int) -> int:
    """Bytes one kernel launch must move: every gradient once, theta and v read and written once."""
    return num_params * (entries * grad_bytes + 16)


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs (read-only NVML)."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:                                   # CUDA_VISIBLE_DEVICES may renumber: match by UUID
                uuid = "GPU-" + str(torch.cuda.get_device_properties(index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _reason_names(self, mask: int):
        nv = self.nv
        table = {
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        return [k for k, bit in table.items() if mask & bit]

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.reasons.update(self._reason_names(mask))
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return False

    def summary(self):
        if self.nv is None or not self.samples:
            return self._smi_once()
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": float(self.max_mhz),
                "reasons": sorted(self.reasons), "samples": len(self.samples)}

    def _smi_once(self):
        try:
            out = subprocess.run(["nvidia-smi", "-i", str(self.index), "--query-gpu=clocks.sm,clocks.max.sm",
                                  "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10).stdout
            a, b = [float(x) for x in out.strip().split(",")]
            return {"sm_mhz": a, "sm_max_mhz": b, "reasons": [], "samples": 1, "note": "sampled after the timed region"}
        except Exception:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}


def max_over_ranks(values, device, world: int):
    """Slowest rank decides: element-wise maximum of per-rank timings (the only cross-rank exchange)."""
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_value(world: int, elems_per_step: int, steps: int, elapsed_ms: float) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return world * elems_per_step * steps / (elapsed_ms * 1e-3)


def step_events(cfg, num_steps: int):
    """Per step, the list of trace events up to and including the push that completes a group."""
    kinds, learners = arrivals.make_trace(cfg.arrival_model, cfg.num_learners, num_steps * cfg.c, cfg.seed)
    steps, cur, pushes = [], [], 0
    for k, l in zip(kinds.tolist(), learners.tolist()):
        cur.append((k, l))
        if k == arrivals.PUSH:
            pushes += 1
            if pushes % cfg.c == 0:
                steps.append(cur)
                cur = []
    return steps


# ----------------------------------------------------------------------------- our arm
NOMINAL_HBM_GBS = 8000.0

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) that ncu counted for one kernel
# instantiation on one workload, with the summary under profiles/ that records the capture.  A run reports
# a figure only when it launches that same instantiation in the same way; anything else gets null and why.
TRAFFIC_CAPTURES = {
    ("large_softsync", "vector", "fp32", 4, 1, 128, False, False):
        (1.9124e9, "profiles/softsync_update_fp32_c4_large_softsync.md"),
    ("large_stale_bf16", "vector", "bf16", 1, 8, 128, False, False):
        (1.9147e9, "profiles/softsync_update_bf16_c1_T8_large_stale_bf16.md"),
}


def traffic_for(cfg_name, kernel, grad_dtype, c, fuse_t, threads, mirror, layers):
    key = (cfg_name, kernel, grad_dtype, c, fuse_t, threads or 128, bool(mirror), bool(layers))
    if key in TRAFFIC_CAPTURES:
        v, src = TRAFFIC_CAPTURES[key]
        return v, src
    return None, "no ncu capture of this kernel instantiation / launch shape is recorded under profiles/"


def build_server(P, cfg, args, dev, rank, fuse_t):
    layout = cfg.layout()
    n = layout.num_params
    ps = P.ParameterServer(n, cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay,
                           cfg.modulation, cfg.grad_dtype, fuse_t, device=dev)
    ps.init_weights(G.initial_weights(layout, cfg.seed + rank, cfg.weight_std, device=dev))
    # every gradient buffer exists before the first update, so consecutive update kernels may overlap
    # their launch ramps (the option's contract)
    ps.set_option(P.PS_OPT_OVERLAP_LAUNCH, 0 if args.no_overlap else 1)
    ps.set_option(P.PS_OPT_KERNEL, P.binding.KERNELS[args.kernel])
    if args.block_threads:
        ps.set_option(P.PS_OPT_BLOCK_THREADS, args.block_threads)
    if args.no_zigzag:
        ps.set_option(P.PS_OPT_ZIGZAG, 0)
    if args.bulk_tile:
        ps.set_option(P.PS_OPT_BULK_TILE, args.bulk_tile)
    if args.bulk_stages:
        ps.set_option(P.PS_OPT_BULK_STAGES, args.bulk_stages)
    if args.layer_multipliers:                    # rate x2 / decay x0 on biases, x1 / x1 on weights
        bounds = [seg.offset for seg in layout.segments] + [n]
        ps.set_layer_multipliers(bounds, [2.0 if seg.is_bias else 1.0 for seg in layout.segments],
                                 [0.0 if seg.is_bias else 1.0 for seg in layout.segments])
    if args.bf16_mirror:
        ps.bind_weight_mirror()                    # every pass also writes theta as bf16 (2 more bytes per element)
    if args.replicas:                              # every pass also writes theta into R further fp32 buffers
        ps.bind_weight_replicas([torch.empty(n, dtype=torch.float32, device=dev) for _ in range(args.replicas)])
    return ps, n


def make_stepper(ps, cfg, events, groups_per_step, grads):
    """One step = the trace's pulls and pushes of `groups_per_step` groups, then ONE ps_apply_update."""
    cursor = {"i": 0}
    pulled = {}

    def one_step(step_index: int):
        for gi in range(groups_per_step):
            for k, l in events[step_index * groups_per_step + gi]:
                if k == arrivals.PULL:
                    pulled[l] = ps.pull_weights()
                else:
                    g = grads[cursor["i"] % len(grads)]
                    cursor["i"] += 1
                    ps.push_gradient(l, g, pulled[l])
        done = ps.apply_update()
        assert done == groups_per_step
    return one_step


def measure_device(P, cfg, args, dev, rank, world, local_rank, fuse_t, steps, warmup, repeats, pool=None):
    """Gradients resident in HBM.  The timed region (`steps` steps between two CUDA events on the server's
    stream, barrier + synchronize on both sides) is run `repeats` times; every repeat carries its own clock
    samples.  Returns (per-repeat list, server facts, gradient pool, the server)."""
    import torch.distributed as dist
    ps, n = build_server(P, cfg, args, dev, rank, fuse_t)
    tdt = torch.bfloat16 if cfg.grad_dtype == "bf16" else torch.float32
    pool_n = max(POOL_BUFFERS, 2 * cfg.c * fuse_t)
    if pool is None or len(pool) < pool_n:
        pool = [G.gradient(cfg.seed + rank, i, 0, n, cfg.grad_std, dtype=tdt, device=dev) for i in range(pool_n)]
    total_steps = warmup + steps * repeats
    one_step = make_stepper(ps, cfg, step_events(cfg, total_steps * fuse_t), fuse_t, pool)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for s in range(warmup):
        one_step(s)
    ps.synchronize()
    out = []
    done = warmup
    for r in range(repeats):
        applied_before = ps.timestamps()[0]
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        with ClockSampler(local_rank) as clocks:
            start.record()                             # torch's current stream is the server's stream
            for s in range(done, done + steps):
                one_step(s)
            stop.record()
            torch.cuda.synchronize(dev)
        barrier()
        done += steps
        # one update kernel per step and nothing else on the stream between the two events
        launches = (ps.timestamps()[0] - applied_before) // fuse_t
        assert launches == steps
        out.append({"ms": start.elapsed_time(stop), "clocks": clocks.summary()})
    facts = {"last_kernel": ps.get_option(P.PS_OPT_LAST_KERNEL),
             "launches": {k: ps.get_option(o) for k, o in (("scalar", P.PS_OPT_LAUNCHES_SCALAR),
                                                           ("vector", P.PS_OPT_LAUNCHES_VECTOR),
                                                           ("bulk", P.PS_OPT_LAUNCHES_BULK))},
             "num_params": n, "pool_n": len(pool)}
    ps.synchronize()
    return out, facts, pool, ps


def summarise(repeats_ms, steps):
    per_step = sorted(r["ms"] / steps for r in repeats_ms)
    return {"median": per_step[len(per_step) // 2], "min": per_step[0], "max": per_step[-1]}


def measure_e2e(P, ps, cfg, args, dev, rank, world, fuse_t, pool, e2e_steps):
    """Gradients from pinned host memory (one cudaMemcpyAsync per push into a recycled staging slot), the
    updated weights copied back to pinned host memory after every step.  Returns (seconds, details)."""
    import torch.distributed as dist
    layout = cfg.layout()
    n = layout.num_params
    tdt = torch.bfloat16 if cfg.grad_dtype == "bf16" else torch.float32
    host_pool = [torch.empty(n, dtype=tdt).pin_memory() for _ in range(min(4, len(pool)))]
    for hb, db in zip(host_pool, pool):
        hb.copy_(db)
    w_host = torch.empty(n, dtype=torch.float32).pin_memory()
    ps.bind_staging(2 * cfg.c * fuse_t)
    ps.init_weights(G.initial_weights(layout, cfg.seed + rank, cfg.weight_std, device=dev))
    events = step_events(cfg, (1 + e2e_steps) * fuse_t)
    one_step = make_stepper(ps, cfg, events, fuse_t, host_pool)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def e2e_step(s):
        one_step(s)
        ps.pull_weights(w_host, non_blocking=True)      # device -> host read of the step's result, overlapped
                                                        # with the next step's host -> device gradient copies
    e2e_step(0)
    ps.synchronize()
    barrier()
    t0 = time.perf_counter()
    for s in range(1, 1 + e2e_steps):
        e2e_step(s)
    ps.synchronize()                                   # every read-back has landed in host memory
    torch.cuda.synchronize(dev)
    seconds = time.perf_counter() - t0
    barrier()
    return seconds, {"w_host": w_host, "host_pool": host_pool, "events": events, "steps": 1 + e2e_steps,
                     "fuse_t": fuse_t, "seed": cfg.seed + rank}


def run_ours(args, cfg, rank, world, local_rank):
    from paper_1511_05950_b200 import build as lib_build
    if local_rank == 0:
        lib_build.ensure_built()                   # no-op when the in-tree library is current
    if world > 1:
        import torch.distributed as dist_
        dist_.barrier()
    import paper_1511_05950_b200 as P

    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    gbytes = 2 if cfg.grad_dtype == "bf16" else 4
    fuse_t = args.fuse_t or cfg.fuse_t
    peak, peak_kind = hbm_peak()

    reps, facts, pool, ps = measure_device(P, cfg, args, dev, rank, world, local_rank, fuse_t,
                                           args.steps, args.warmup, args.repeats)
    n = facts["num_params"]
    e2e_steps, e2e_s, e2e_detail = 0, 0.0, None
    if not args.no_e2e:
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        e2e_s, e2e_detail = measure_e2e(P, ps, cfg, args, dev, rank, world, fuse_t, pool, e2e_steps)
    ps.destroy()
    del pool

    # slowest rank decides, repeat by repeat
    maxed = max_over_ranks([r["ms"] for r in reps] + [e2e_s * 1e3], dev, world)
    for r, ms in zip(reps, maxed):
        r["ms"] = ms
    e2e_ms = maxed[-1]
    stat = summarise(reps, args.steps)
    median_ms = stat["median"] * args.steps

    elems_per_step = cfg.c * n * fuse_t
    if args.total_params:                              # sharded: the ranks together hold one vector
        value = whole_job_value(1, cfg.c * args.total_params * fuse_t, args.steps, median_ms)
        e2e_value = whole_job_value(1, cfg.c * args.total_params * fuse_t, e2e_steps, e2e_ms) if e2e_steps else None
    else:
        value = whole_job_value(world, elems_per_step, args.steps, median_ms)
        e2e_value = whole_job_value(world, elems_per_step, e2e_steps, e2e_ms) if e2e_steps else None
    abytes = algorithmic_bytes(n, cfg.c * fuse_t, gbytes) + (2 * n if args.bf16_mirror else 0) + 4 * n * args.replicas
    kern_ms = stat["median"]
    achieved = abytes / (kern_ms * 1e-3) / 1e9
    kernel_name = {1: "scalar", 2: "vector", 3: "bulk"}.get(facts["last_kernel"], "none")
    traffic, traffic_from = traffic_for(cfg.name, kernel_name, cfg.grad_dtype, cfg.c, fuse_t, args.block_threads,
                                        args.bf16_mirror or args.replicas, args.layer_multipliers)
    if (args.no_overlap or args.no_zigzag) and traffic is not None:
        traffic, traffic_from = None, "the recorded capture used programmatic dependent launches and alternating traversal"
    mid = sorted(reps, key=lambda r: r["ms"])[len(reps) // 2]
    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": stat["median"], "higher_is_better": True,
        "scaling": "strong" if args.total_params else "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": "%s: N=%d fp32 parameters (%s layout), lambda=%d, n=%d, c=%d %s gradients "
                        "per update, T=%d updates per kernel pass" % (cfg.name, n, cfg.layout().name, cfg.num_learners,
                                                                    cfg.n, cfg.c, cfg.grad_dtype, fuse_t),
            "num_params": n, "lambda": cfg.num_learners, "n": cfg.n, "c": cfg.c, "fuse_t": fuse_t,
            "grad_dtype": cfg.grad_dtype, "arrivals": cfg.arrival_model, "alpha0": cfg.alpha0,
            "momentum": cfg.momentum, "weight_decay": cfg.weight_decay, "modulation": cfg.modulation,
            "bf16_mirror": bool(args.bf16_mirror), "layer_multipliers": bool(args.layer_multipliers),
            "weight_replicas": args.replicas,
            "kernel": kernel_name, "kernel_launches": facts["launches"],
            "launch": "ordinary" if args.no_overlap else "programmatic dependent launch (PS_OPT_OVERLAP_LAUNCH=1)",
            "traversal": "forward" if args.no_zigzag else "alternating direction from launch to launch",
            "parallelism": ("%d contiguous shards of one %d-parameter vector, no data-path collective"
                            % (world, args.total_params)) if args.total_params else
                           ("replicas only (independent servers, no data-path collective)" if world > 1 else "1 GPU"),
            "l2": ("inputs larger than L2: each step streams %.2f GB from %d rotating gradient buffers"
                   % (abytes / 1e9, facts["pool_n"])) if abytes > 2 * L2_BYTES else
                  ("working set of %.1f MB per step stays in L2: a launch-latency figure, not an HBM one"
                   % (abytes / 1e6)),
        },
        "repeats": {"count": len(reps), "steps_each": args.steps,
                    "ms_per_step": stat,
                    "each": [{"ms_per_step": r["ms"] / args.steps, "sm_mhz": r["clocks"].get("sm_mhz"),
                              "reasons": r["clocks"].get("reasons")} for r in reps],
                    "note": "value, ms_per_step and roofline use the median repeat; ms_per_step x sm_mhz separates "
                            "a clock change from a kernel change"},
        "hbm_gbs": world * abytes / (stat["median"] * 1e-3) / 1e9,
        "gpu_launches": int(args.steps),
        "clocks": mid["clocks"],
        "e2e": {"value": e2e_value, "unit": UNIT, "steps": e2e_steps,
                "h2d_bytes_per_step": cfg.c * fuse_t * n * gbytes, "d2h_bytes_per_step": n * 4,
                "ms_per_step": e2e_ms / e2e_steps if e2e_steps else None},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "of": peak_kind,
                     "peak_is": "copy bandwidth (1 read : 1 write); not a ceiling for this read-heavy pass, "
                                "which may read a little above 1",
                     "nominal_peak": NOMINAL_HBM_GBS, "frac_of_nominal": achieved / NOMINAL_HBM_GBS,
                     "traffic": traffic, "traffic_from": traffic_from,
                     "kernel_ms": kern_ms, "algorithmic_bytes": abytes,
                     "how": "CUDA events around the %d back-to-back launches of a timed region / %d "
                            "(inter-launch gaps included), median of %d regions" % (args.steps, args.steps, len(reps))},
    }
    return result, e2e_detail


def second_config(args, rank, world, local_rank):
    """The other 61 M-parameter configuration (bf16 gradients, c = 1, T = 8 fused updates per pass), measured
    the same way in the same process, and its unfused form (T = 1) beside it."""
    import paper_1511_05950_b200 as P
    cfg = configs.LARGE_STALE_BF16
    dev = torch.device("cuda", local_rank)
    peak, peak_kind = hbm_peak()
    out = {}
    pool = None
    for label, fuse_t, steps in (("fused", cfg.fuse_t, max(1, args.steps // 2)), ("unfused", 1, args.steps)):
        reps, facts, pool, ps = measure_device(P, cfg, args, dev, rank, world, local_rank, fuse_t, steps,
                                               args.warmup, args.repeats, pool=pool)
        ps.destroy()
        maxed = max_over_ranks([r["ms"] for r in reps], dev, world)
        for r, ms in zip(reps, maxed):
            r["ms"] = ms
        stat = summarise(reps, steps)
        n = facts["num_params"]
        abytes = algorithmic_bytes(n, cfg.c * fuse_t, 2)
        gbs = abytes / (stat["median"] * 1e-3) / 1e9
        out[label] = {
            "fuse_t": fuse_t, "steps": steps, "us_per_pass": {k: v * 1e3 for k, v in stat.items()},
            "updates_per_s": world * fuse_t / (stat["median"] * 1e-3),
            "value": world * cfg.c * n * fuse_t / (stat["median"] * 1e-3), "unit": UNIT,
            "algorithmic_bytes": abytes, "hbm_gbs": gbs, "frac": gbs / peak, "of": peak_kind,
            "frac_of_nominal": gbs / NOMINAL_HBM_GBS,
            "each": [{"us_per_pass": r["ms"] / steps * 1e3, "sm_mhz": r["clocks"].get("sm_mhz"),
                      "reasons": r["clocks"].get("reasons")} for r in reps],
            "kernel_launches": facts["launches"],
        }
    tr, src = traffic_for(cfg.name, "vector", "bf16", cfg.c, cfg.fuse_t, args.block_threads, False, False)
    out["fused"]["traffic"], out["fused"]["traffic_from"] = tr, src
    out["workload"] = "%s: N=%d, lambda=%d, n=%d, c=%d bf16 gradients, T=%d" % (
        cfg.name, cfg.layout().num_params, cfg.num_learners, cfg.n, cfg.c, cfg.fuse_t)
    return out


# ----------------------------------------------------------------------------- oracle arms
def oracle_sample(cfg, sample_params: int, updates: int, rotate: int = 8, threads: int = 1):
    """Time the CPU reference, as it stands, on `updates` updates over the first `sample_params`
    elements of the workload.  threads > 1: that many unmodified reference servers, each on its own
    contiguous range of the vector (the update is element-wise, so the result is the same).
    Returns (grad elements per second, seconds)."""
    from concurrent.futures import ThreadPoolExecutor

    from oracle import reference as R

    layout = cfg.layout()
    idx_n = min(sample_params, layout.num_params)
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    tdt = torch.bfloat16 if cfg.grad_dtype == "bf16" else torch.float32
    w0 = G.initial_weights(layout, cfg.seed, cfg.weight_std, device=gen_dev)[:idx_n].cpu().numpy()
    grads = []
    for i in range(rotate):
        g = G.gradient(cfg.seed, i, 0, idx_n, cfg.grad_std, dtype=tdt, device=gen_dev).cpu()
        grads.append(g.view(torch.int16).numpy().view(np.uint16) if tdt == torch.bfloat16 else g.numpy())
    threads = max(1, min(threads, idx_n))
    bounds = [idx_n * t // threads for t in range(threads + 1)]
    mod = R.MOD_INV_STALENESS if cfg.modulation == "inv_staleness" else R.MOD_CONSTANT
    servers = []
    for a, b in zip(bounds[:-1], bounds[1:]):
        ref = R.ReferencePS(b - a, cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay, mod, 32)
        ref.set_weights(w0[a:b])
        servers.append((a, b, ref))
    steps = step_events(cfg, updates)

    def replay(part):
        a, b, ref = part
        i = 0
        for evs in steps:
            for k, l in evs:
                if k == arrivals.PULL:
                    ref.pull(l)
                else:
                    ref.push(l, grads[i % rotate][a:b])          # ctypes calls release the GIL
                    i += 1
        return ref.timestamp

    t0 = time.perf_counter()
    if threads == 1:
        done = [replay(servers[0])]
    else:
        with ThreadPoolExecutor(threads) as pool:
            done = list(pool.map(replay, servers))
    dt = time.perf_counter() - t0
    assert all(d == updates for d in done)
    return cfg.c * idx_n * updates / dt, dt


def cpu_baseline(cfg):
    # about 10 s of single-thread work at the reference's ~6e8 gradient elements/s, at most the whole workload
    n = cfg.layout().num_params
    per_update_s = cfg.c * n / 6e8
    updates = int(max(24, min(cfg.num_updates, 10.0 / per_update_s)))
    v, dt = oracle_sample(cfg, n, updates)
    cores = os.cpu_count() or 1
    out = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": "first %d updates of the workload at full size (%d parameters), fp32 reference, "
                     "single thread, %.1f s; host has %d cores" % (updates, n, dt, cores)}
    if cores > 1 and n >= (1 << 20):
        va, dta = oracle_sample(cfg, n, updates, threads=cores)
        out["all_cores"] = {"value": va, "unit": UNIT, "cores": cores,
                            "sample": "same updates, %d unmodified reference servers on contiguous ranges of the "
                                      "vector, one thread each, %.1f s" % (cores, dta)}
    return out


def check_e2e_result(cfg, detail, samples: int = 4096):
    """The weights the end-to-end leg read back, against a replay of the same steps through the CPU
    reference on a sample of the elements (the update is element-wise).  Outside every timed region."""
    from oracle import reference as R
    layout = cfg.layout()
    n = layout.num_params
    rng = np.random.default_rng(7)
    idx = np.unique(np.concatenate([rng.integers(0, n, size=samples), np.arange(0, 32), np.arange(n - 32, n)]))
    idx_t = torch.from_numpy(idx)
    mod = {"inv_staleness": R.MOD_INV_STALENESS, "constant": R.MOD_CONSTANT, "exp_staleness": R.MOD_EXP_STALENESS}[cfg.modulation]
    ref = R.ReferencePS(idx.size, cfg.num_learners, cfg.n, cfg.alpha0, cfg.momentum, cfg.weight_decay, mod, 32)
    ref.set_weights(G.initial_weights_at(layout, detail["seed"], idx_t, cfg.weight_std).numpy())
    grads = []
    for hb in detail["host_pool"]:
        g = hb[idx_t]
        grads.append(g.view(torch.int16).numpy().view(np.uint16) if g.dtype == torch.bfloat16 else g.numpy())
    i = 0
    for evs in detail["events"][: detail["steps"] * detail["fuse_t"]]:
        for k, l in evs:
            if k == arrivals.PULL:
                ref.pull(l)
            else:
                ref.push(l, grads[i % len(grads)])
                i += 1
    want = ref.state()[0].astype(np.float32)
    got = detail["w_host"][idx_t].numpy()
    return {"sampled_elements": int(idx.size), "updates": int(ref.timestamp),
            "bit_equal_to_reference": bool(np.array_equal(got, want))}


def run_reference(args, cfg):
    sample_params = 1 << 22
    v, dt = oracle_sample(cfg, sample_params, args.warmup)       # warm-up steps, untimed in the result
    v, dt = oracle_sample(cfg, sample_params, args.steps)
    layout = cfg.layout()
    sample = ("each step is one update over the first %d of %d parameters, fp32 reference, single thread"
              % (sample_params, layout.num_params))
    return {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3 / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "%s (CPU reference on a bounded sample)" % cfg.name, "num_params": layout.num_params,
                   "lambda": cfg.num_learners, "n": cfg.n, "c": cfg.c, "grad_dtype": cfg.grad_dtype},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def run_sweep(args):
    from paper_1511_05950_b200 import build as lib_build
    lib_build.ensure_built()
    return _run_sweep(args)


def _run_sweep(args):
    """Bandwidth sweep: flat fp32 vectors of 1M .. 1B parameters, c in {1,4,16,64}, fp32 and bf16
    gradients, staleness uniform in [1, 2c], 50 updates per point after 5 warm-up updates."""
    import paper_1511_05950_b200 as P

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, peak_kind = hbm_peak()
    l2_bytes = torch.cuda.get_device_properties(dev).L2_cache_size
    rng = np.random.default_rng(configs.SEED)
    points = []
    updates, warm = args.sweep_updates, 5
    sizes = [int(x) for x in args.sweep_sizes.split(",") if x] or list(configs.SWEEP_SIZES)
    group_sizes = [int(x) for x in args.sweep_c.split(",") if x] or list(configs.SWEEP_C)
    for n in sizes:
        for grad_dtype, tdt, gb in (("fp32", torch.float32, 4), ("bf16", torch.bfloat16, 2)):
            for c in group_sizes:
                abytes = algorithmic_bytes(n, c, gb)
                pool_n = max(c, min(64, -(-(4 * l2_bytes) // (n * gb))))
                need = n * 8 + pool_n * n * gb + (2 << 30)
                torch.cuda.empty_cache()
                free, _ = torch.cuda.mem_get_info(dev)
                point = {"num_params": n, "c": c, "grad_dtype": grad_dtype, "algorithmic_bytes": abytes,
                         "fits_l2": bool(abytes <= l2_bytes)}
                if need > free:
                    point["skipped"] = "does not fit: needs %.1f GB, %.1f GB free" % (need / 1e9, free / 1e9)
                    points.append(point)
                    continue
                ps = P.ParameterServer(n, c, 1, 0.01, 0.9, 5e-4, "inv_staleness", grad_dtype, 1, device=dev)
                ps.set_option(P.PS_OPT_QUEUE_GROUPS, 4)
                w0 = torch.empty(n, dtype=torch.float32, device=dev)
                G.normal_like(G.stream_key(configs.SEED, G.STREAM_WEIGHTS), 0, n, 0.01, out=w0)
                ps.init_weights(w0)
                del w0
                # start the clock at 2c so that every staleness drawn from [1, 2c] is reachable at once
                words = ps.export_state()
                words[5] = 2 * c
                ps.import_state(words)
                pool = []
                for i in range(pool_n):
                    buf = torch.empty(n, dtype=tdt, device=dev)
                    G.gradient(configs.SEED, i, 0, n, 1e-4, dtype=tdt, device=dev, out=buf)
                    pool.append(buf)
                k = 0
                start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                for u in range(warm + updates):
                    if u == warm:
                        torch.cuda.synchronize(dev)
                        start.record()
                    now = ps.pull_weights()
                    for l in range(c):
                        sigma = int(rng.integers(1, 2 * c + 1))
                        ps.push_gradient(l, pool[k % pool_n], now - sigma)
                        k += 1
                    ps.apply_update()
                stop.record()
                torch.cuda.synchronize(dev)
                ms = start.elapsed_time(stop) / updates
                point.update({"us_per_update": ms * 1e3, "gbs": abytes / ms / 1e6, "frac_of_%s_copy_peak" % peak_kind:
                              abytes / ms / 1e6 / peak, "grad_elements_per_s": c * n / (ms * 1e-3)})
                points.append(point)
                ps.destroy()
                del pool
                print("N=%-11d %s c=%-3d %9.1f us  %7.1f GB/s  %5.1f%% of %s copy peak%s" % (
                    n, grad_dtype, c, ms * 1e3, point["gbs"], 100 * point["gbs"] / peak, peak_kind,
                    "  (fits L2: not an HBM figure)" if point["fits_l2"] else ""), file=sys.stderr, flush=True)
    return {"metric": "hbm_gbs_per_softsync_update", "unit": "GB/s", "peak": peak, "of": peak_kind,
            "updates_per_point": updates, "warmup": warm, "sweep": points}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large_softsync", choices=sorted(configs.BY_NAME))
    ap.add_argument("--repeats", type=int, default=7, help="how many times the timed region of --steps steps is run")
    ap.add_argument("--kernel", default="auto", choices=["auto", "scalar", "vector", "bulk"],
                    help="PS_OPT_KERNEL: which update kernel the server launches")
    ap.add_argument("--block-threads", type=int, default=0, choices=[0, 128, 256, 512])
    ap.add_argument("--bulk-tile", type=int, default=0, help="PS_OPT_BULK_TILE (with --kernel bulk)")
    ap.add_argument("--bulk-stages", type=int, default=0, help="PS_OPT_BULK_STAGES (with --kernel bulk)")
    ap.add_argument("--layer-multipliers", action="store_true",
                    help="variant: per-layer rate / decay multipliers (x2 / x0 on biases)")
    ap.add_argument("--no-second-config", action="store_true",
                    help="skip the bf16 T=8 configuration that the default run measures beside the headline one")
    ap.add_argument("--e2e-steps", type=int, default=12)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-overlap", action="store_true", help="ordinary launches instead of programmatic dependent ones")
    ap.add_argument("--fuse-t", type=int, default=0, choices=range(0, 17),
                    help="variant: updates per kernel pass (PS_OPT_FUSE_T) instead of the workload's own; 0 = the workload's")
    ap.add_argument("--no-zigzag", action="store_true", help="every launch walks the vector forward (PS_OPT_ZIGZAG=0)")
    ap.add_argument("--bf16-mirror", action="store_true",
                    help="variant: keep a bf16 copy of the weights current in the same pass (+2 bytes per element)")
    ap.add_argument("--replicas", type=int, default=0, choices=range(0, 9),
                    help="variant: the update pass also stores theta into this many further fp32 buffers "
                         "(the fused weight broadcast of a sharded server; here all in this GPU's memory)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (for profiler captures)")
    ap.add_argument("--num-params", type=int, default=0,
                    help="run the workload's protocol on a flat vector of this many parameters (profiler captures)")
    ap.add_argument("--sharded", action="store_true",
                    help="with N > 1 ranks: one server over the workload's vector, a contiguous shard per rank "
                         "(strong scaling) instead of one replica per rank")
    ap.add_argument("--sweep", action="store_true", help="bandwidth sweep over sizes, group sizes and gradient types")
    ap.add_argument("--sweep-sizes", default="", help="comma-separated subset of the sweep's vector sizes")
    ap.add_argument("--sweep-c", default="", help="comma-separated subset of the sweep's group sizes")
    ap.add_argument("--sweep-updates", type=int, default=50, help="timed updates per sweep point")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.repeats = max(args.repeats, 1)
    cfg = configs.BY_NAME[args.workload]
    if args.num_params:
        from dataclasses import replace
        from workloads import layouts
        flat_n = args.num_params
        cfg = replace(cfg, name="%s@flat%d" % (cfg.name, flat_n), layout=lambda: layouts.flat(flat_n))

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args, cfg)), flush=True)
        return
    args.total_params = 0
    if args.sharded and world > 1:
        from dataclasses import replace
        from paper_1511_05950_b200.sharded import shard_bounds
        from workloads import layouts
        args.total_params = cfg.layout().num_params
        bounds = shard_bounds(args.total_params, world, grad_dtype=cfg.grad_dtype)
        local_n = bounds[rank + 1] - bounds[rank]
        cfg = replace(cfg, name="%s@shard%dof%d" % (cfg.name, rank, world), layout=lambda: layouts.flat(local_n))
    if args.sweep:
        if rank == 0:
            print(json.dumps(run_sweep(args)), flush=True)
        return

    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    result, e2e_detail = run_ours(args, cfg, rank, world, local_rank)
    default_run = (args.workload == "large_softsync" and not args.num_params and not args.total_params
                   and args.kernel == "auto" and not args.bf16_mirror and not args.layer_multipliers
                   and not args.no_zigzag and not args.replicas and not args.fuse_t)
    if default_run and not args.no_second_config:
        result["configs"] = {"large_stale_bf16": second_config(args, rank, world, local_rank)}
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            result["cpu_baseline"] = cpu_baseline(cfg)
            if e2e_detail is not None:
                result["e2e"]["check"] = check_e2e_result(cfg, e2e_detail)
        print(json.dumps(result), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
