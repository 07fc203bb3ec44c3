#!/usr/bin/env python
"""Benchmark of the mixed-tenant inference hot path.

One "step" = one mt_infer call: bucketing, one grouped launch per layer (the last one returns the rows to arrival
order), over one synthetic mixed batch.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

Without --config the headline (`value`, `roofline`, `e2e`, ...) is workload 2 (64 tenants x MLP 1024-4096-4096-1024,
4096 requests, Zipf 1.1) and `per_config` carries the same measurements for all five workloads.  With --config C only
that workload runs.

Timing: after W warm-up steps, EXACTLY K steps between two CUDA events on the launching stream (a synchronisation and,
with several ranks, a barrier on both sides): that block gives `value` and `ms_per_step`.  A block of K steps may last
only milliseconds, in which the GPU neither reaches its power cap nor gives the clock sampler a sample; so (one rank
only) the same block is repeated until about two seconds of device time have passed, and `sustained` reports the
per-step time of the blocks (min / median / max / first / last) with the SM clock sampled during each.

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank hosts all tenants and runs its own batch
(requests of different batches are independent; no collective on the data path): weak scaling.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1901_06887_b200 import synth  # noqa: E402

METRIC = "mixed-tenant requests/sec"
UNIT = "requests/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
HEADLINE_CONFIG = 2
DEFAULT_STEPS = {1: 2000, 2: 200, 3: 400, 4: 400, 5: 20}
SUSTAIN_MS = 2000.0          # repeat the timed block until this much device time has passed ...
MAX_BLOCKS = 400             # ... or this many blocks
N_INPUT_BUFFERS = 3
# Requests of the batch the reference arm (--impl reference) times per step.
REFERENCE_SAMPLE = {1: 64, 2: 512, 3: 4096, 4: 6, 5: 24}
# DRAM traffic of the dominant kernel, from the ncu captures summarised under profiles/.  "ratio": traffic over
# algorithmic bytes measured on a reduced case of the same kernel, scaled to the full launch (traffic grows with the
# weights of the tenants that have requests, as the algorithmic bytes do); "bytes": measured at full size, per step.
# An entry is deleted when its kernel changes and comes back with the next capture.
TRAFFIC = {
    2: {"ratio": 0.997, "source": "profiles/grouped_gemm_c2_reduced_ncu_full.md (16 tenants, 1024 requests: 843.0 MB "
                                  "measured / 845.8 MB algorithmic), scaled by algorithmic bytes"},
    3: {"ratio": 1.007, "source": "profiles/grouped_gemm128_c3_reduced_ncu_full.md (250 tenants, 4096 requests: 272.1 MB "
                                  "measured / 270.0 MB algorithmic), scaled by algorithmic bytes"},
    4: {"bytes": 720.7e6, "source": "profiles/grouped_conv3x3_pair_c4_full_ncu_full.md (full size, the four conv layers of a step in one launch)"},
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def env_int(name, default):
    return int(os.environ.get(name, default))


def aggregate(local_units: float, local_ms: float, world: int):
    """Whole-job numbers from per-rank ones: units add up, the time is the slowest rank's (device time).
    Uses torch.distributed when world > 1 (nccl on GPUs, gloo in the CPU tests)."""
    if world == 1:
        return float(local_units), float(local_ms)
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([local_units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(u.item()), float(t.item())


def result_line(metric_units: float, ms_total: float, n_steps: int, **extra):
    """units/s over the timed region and ms per step."""
    value = metric_units / (ms_total * 1e-3) if ms_total > 0 else 0.0
    d = {"metric": METRIC, "value": value, "unit": UNIT, "ms_per_step": ms_total / max(n_steps, 1),
         "higher_is_better": True}
    d.update(extra)
    return d


def gpu_selector(local_rank: int) -> str:
    """What `nvidia-smi -i` needs to find THIS process's GPU: its UUID (nvidia-smi counts physical devices and knows
    nothing of CUDA_VISIBLE_DEVICES, so the CUDA index would name another GPU on a shared host)."""
    try:
        import torch
        u = str(torch.cuda.get_device_properties(local_rank).uuid)
        return u if u.startswith("GPU-") else "GPU-" + u
    except Exception:
        return str(local_rank)


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs (read-only queries), with time
    stamps so that samples can be assigned to the timed blocks."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    REASONS = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, selector: str, period_ms: int = 20):
        self.selector = selector
        self.period_ms = period_ms
        self.proc = None
        self.path = None
        self.samples = []          # (unix time, sm MHz, max MHz, watts, [reasons])

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.selector, "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", str(self.period_ms)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 8:
                    continue
                try:
                    ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    sm, mx = float(parts[1]), float(parts[2])
                    watts = float(parts[3])
                except ValueError:
                    continue
                reasons = [nm for nm, v in zip(self.REASONS, parts[4:8]) if v.lower().startswith("active")]
                self.samples.append((ts, sm, mx, watts, reasons))
            os.unlink(self.path)
        except Exception:
            pass
        self.proc = None

    def summary(self, t0=None, t1=None):
        """Median SM clock, maximum, reasons seen and sample count over [t0, t1] (all samples by default)."""
        sel = [s for s in self.samples if (t0 is None or s[0] >= t0) and (t1 is None or s[0] <= t1)]
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": len(sel)}
        if sel:
            out.update(sm_mhz=float(np.median([s[1] for s in sel])), sm_max_mhz=float(max(s[2] for s in sel)),
                       power_w=float(np.median([s[3] for s in sel])),
                       reasons=sorted({r for s in sel for r in s[4]}))
        return out


def dominant_roofline(wl, kernel_ms_per_step, peaks, peaks_kind, config, long_run):
    """Roofline of the dominant kernel (the grouped layer executor), all its launches of one step together:
    algorithmic bytes (weights + bias of tenants with requests once, activations in, activations out) and flops of
    those layers, against the measured HBM and bf16 peaks; the larger time bounds it.  A tensor-bound kernel is held
    against the burst cuBLAS figure when its timed region was short and against the sustained one when the region
    lasted long enough for the power cap to act (long_run); the fraction of the other peak is given beside it."""
    per_layer_bytes = synth.workload_bytes(wl.models, wl.model_ids, per_layer=True)
    kinds = [l.kind for l in wl.models[0]]
    dom_kind = synth.CONV3X3 if synth.CONV3X3 in kinds else synth.DENSE
    counts = np.bincount(wl.model_ids, minlength=len(wl.models))
    byts = sum(b for b, k in zip(per_layer_bytes, kinds) if k == dom_kind)
    flops = sum(int(c) * sum(synth.layer_flops(l) for l in m if l.kind == dom_kind) for c, m in zip(counts, wl.models))
    burst = peaks["bf16_tflops"]
    sustained = peaks.get("bf16_tflops_sustained", burst)
    t_hbm = byts / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (burst * 1e12)
    sec = kernel_ms_per_step * 1e-3
    if t_hbm >= t_tc:
        ach = byts / sec / 1e9 if sec > 0 else 0.0
        roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"]}
    else:
        ach = flops / sec / 1e12 if sec > 0 else 0.0
        tc_peak = sustained if long_run else burst
        roof = {"bound": "tensor", "achieved": ach, "peak": tc_peak, "unit": "TFLOP/s", "frac": ach / tc_peak,
                "peak_kind": "sustained (timed inside a seconds-long loop)" if long_run else "burst (timed region under a second)",
                "frac_of_burst_peak": ach / burst, "frac_of_sustained_peak": ach / sustained}
    traffic, source = None, None
    t = TRAFFIC.get(config)
    if any(getattr(l, "residual", 0) for m in wl.models for l in m):
        t = None            # the captures are of the plain workload
    if t is not None:
        traffic = int(t["ratio"] * byts) if "ratio" in t else int(t["bytes"])
        source = t["source"]
    roof.update(traffic=traffic, traffic_source=source, peak_source="of " + peaks_kind,
                algorithmic_bytes_per_step=int(byts), flops_per_step=int(flops), kernel_ms_per_step=kernel_ms_per_step)
    return roof


def oracle_sample(wl, config):
    """Requests the CPU baseline times: the whole batch for workloads 1-4; for workload 5 the first 128 requests of
    every tenant (at least 1024 in all), whose time is extrapolated linearly since every request of a tenant costs the same."""
    if config != 5:
        return np.arange(wl.n), "the whole batch of %d requests" % wl.n
    pick = []
    for t in range(len(wl.models)):
        pick.append(np.flatnonzero(wl.model_ids == t)[:128])
    idx = np.sort(np.concatenate(pick))
    return idx, "%d of %d requests (the first 128 of every tenant); extrapolated from %d requests" % (len(idx), wl.n, len(idx))


def time_oracle(wl, config, repeats=3):
    import oracle
    oracle.build()
    idx, what = oracle_sample(wl, config)
    ids, x = wl.model_ids[idx], wl.inputs[idx]
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle.forward(wl.models, ids, x)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    flops = synth.workload_flops(wl.models, ids)
    return {"value": len(idx) / best, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
            "gflops": flops / best / 1e9,
            "sample": "%s, all tenants resident, best of %d, wall clock %.2f s" % (what, repeats, best)}


def run_reference(args, rank, world):
    """The reference arm: the fp64 CPU oracle as it stands, on the host cores, rank 0 only."""
    if rank != 0:
        return
    cfg = args.config or HEADLINE_CONFIG
    wl = synth.make_workload(cfg)
    n_s = min(wl.n, REFERENCE_SAMPLE[cfg])
    import oracle
    oracle.build()
    ids, x = wl.model_ids[:n_s], wl.inputs[:n_s]
    for _ in range(min(args.warmup, 1)):
        oracle.forward(wl.models, ids, x)
    steps = min(args.steps or 8, 8)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.forward(wl.models, ids, x)
    ms = (time.perf_counter() - t0) * 1e3
    line = result_line(n_s * steps, ms, steps, n_gpus=args.gpus, steps=steps, warmup=min(args.warmup, 1), scaling="weak",
                       vs_baseline=None, dtype="f64", data="synthetic", impl="reference",
                       config={"workload": synth.CONFIG_NAMES[cfg],
                               "sample": "each step = first %d of %d requests" % (n_s, wl.n)})
    line["cpu_baseline"] = {"value": line["value"], "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
                            "sample": "first %d of %d requests per step, %d steps" % (n_s, wl.n, steps)}
    line["e2e"] = {"value": line["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    print(json.dumps(line), flush=True)


def run_cache_sweep(args, ctx):
    """Weight-residency leg (the paper's Sec. 3.3 argument with this machine's numbers): workload 2's 64 tenants behind a
    device cache of a fraction of their total size, small batches through mt_infer_host_async on two streams; per
    fraction the request-level hit ratio, requests/s, bytes copied per step, and the time the copies alone would take
    at the PCIe rate measured in the same run."""
    torch, mt, harness = ctx["torch"], ctx["mt"], ctx["harness"]
    cfg = 2
    nb = args.requests or 64
    models = synth.make_models(cfg)
    n_batches = 48
    batches = [synth.make_requests(cfg, models, n=nb, salt=500 + b) for b in range(n_batches)]
    out_elems = models[0][-1].out_ch
    h_in = [torch.from_numpy(x.view(np.int16)).pin_memory() for _, x in batches]
    h_ids = [torch.from_numpy(i).pin_memory() for i, _ in batches]
    h_outs = [torch.empty((nb, out_elems), dtype=torch.float32).pin_memory() for _ in range(2)]
    two = [torch.cuda.Stream(), torch.cuda.Stream()]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # PCIe rate of this machine: a 512 MB pinned host -> device copy, best of 8
    probe_h = torch.empty(512 << 20, dtype=torch.uint8).pin_memory()
    probe_d = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    pcie = 0.0
    for _ in range(8):
        e0.record(); probe_d.copy_(probe_h, non_blocking=True); e1.record(); torch.cuda.synchronize()
        pcie = max(pcie, (512 << 20) / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    del probe_h, probe_d
    rows = []
    block = None
    for frac in (1.0, 0.97, 0.94, 0.9, 0.8, 0.7, 0.6, 0.5):
        mt.mt_shutdown()
        mt.mt_init(ctx["local_rank"], 64, nb)
        if block is None:      # size of one tenant's block: register one model under a generous cache and read the counter
            mt.mt_set_cache_bytes(1 << 30)
            mt.mt_register_model(models[0])
            block = mt.mt_get_cache_stats()["bytes_loaded"]
            mt.mt_shutdown()
            mt.mt_init(ctx["local_rank"], 64, nb)
        cap = int(frac * len(models) * block) + (1 << 20)
        mt.mt_set_cache_bytes(cap)
        harness.register_models(models)

        def step(i):
            b = i % n_batches
            mt.mt_infer_host_async(h_in[b], h_ids[b], nb, h_outs[i % 2], two[i % 2])

        try:
            for i in range(n_batches):       # one pass over all batches warms the cache into its steady state
                step(i)
            torch.cuda.synchronize()
            mt.mt_get_cache_stats(reset=True)
            steps = 4 * n_batches
            e0.record(two[0])
            for i in range(steps):
                step(i)
            two[0].wait_stream(two[1])
            e1.record(two[0])
            torch.cuda.synchronize()
        except mt.MtError as err:
            rows.append({"cache_fraction": frac, "error": str(err)})
            continue
        ms = e0.elapsed_time(e1)
        st = mt.mt_get_cache_stats()
        if mt.mt_get_async_status() != (0, -1):
            raise SystemExit("device status in the cache sweep")
        req = st["request_hits"] + st["request_misses"]
        ten = st["tenant_hits"] + st["tenant_misses"]
        rows.append({"cache_fraction": frac, "cache_bytes": cap,
                     "request_hit_ratio": st["request_hits"] / max(req, 1), "tenant_hit_ratio": st["tenant_hits"] / max(ten, 1),
                     "requests_per_s": nb * steps / (ms * 1e-3), "ms_per_step": ms / steps,
                     "h2d_weight_bytes_per_step": st["bytes_loaded"] / steps,
                     "pcie_ms_per_step_for_the_misses": st["bytes_loaded"] / steps / (pcie * 1e9) * 1e3,
                     "evictions_per_step": st["evictions"] / steps})
    mt.mt_shutdown()
    full = rows[0]
    line = {"cache_sweep": rows, "workload": synth.CONFIG_NAMES[cfg] + ", batches of %d requests" % nb,
            "tenant_block_bytes": block, "pcie_h2d_gbs": pcie,
            "note": "a miss copies one tenant's %.1f MB block: %.2f ms at the PCIe rate, against %.3f ms for a whole batch "
                    "with every tenant resident" % (block / 1e6, block / (pcie * 1e9) * 1e3, full.get("ms_per_step", 0.0))}
    print(json.dumps(line), flush=True)


def median(xs):
    return float(np.median(xs)) if len(xs) else None


def measure_config(cfg, args, ctx):
    """Everything the bench reports for one workload, as a dict in the layout of the JSON line."""
    torch, dist, mt, harness = ctx["torch"], ctx["dist"], ctx["mt"], ctx["harness"]
    rank, world, local_rank = ctx["rank"], ctx["world"], ctx["local_rank"]
    peaks, peaks_kind = ctx["peaks"], ctx["peaks_kind"]
    steps = args.steps if args.steps is not None else DEFAULT_STEPS[cfg]

    over = {"n_tenants": args.tenants} if args.tenants else {}
    if args.shortcuts and cfg == 4:
        over["shortcuts"] = (1, 3)      # conv layers 1 and 3 close two-layer residual blocks (identity shortcuts)
    models = synth.make_models(cfg, **over)
    batches = [synth.make_requests(cfg, models, n=args.requests, salt=1000 * rank + b) for b in range(N_INPUT_BUFFERS)]
    wl = synth.Workload(synth.CONFIG_NAMES[cfg], cfg, models, batches[0][0], batches[0][1])
    n, out_elems = wl.n, wl.out_elems

    mt.mt_shutdown()
    mt.mt_init(local_rank, max(64, len(models)), n)
    harness.register_models(models)
    dev_in = [harness.bf16_bits_to_device(x) for _, x in batches]
    dev_ids = [torch.from_numpy(i).cuda() for i, _ in batches]
    dev_out = torch.empty((n, out_elems), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()

    def step(i):
        b = i % N_INPUT_BUFFERS
        mt.mt_infer(dev_in[b], dev_ids[b], n, dev_out, stream)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    st = mt.mt_get_async_status()
    if st != (0, -1):
        raise SystemExit("device status after warm-up: %r" % (st,))

    # ---- timed region: device-resident inputs, CUDA events on the launching stream, executor events inside
    sampler = ClockSampler(gpu_selector(local_rank))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if not args.profile:
        sampler.start()
        time.sleep(0.05)
    blocks = []                         # (ms, executor kernel times, wall start, wall end)
    launches = 0
    total_ms = 0.0
    max_blocks = 1 if (world > 1 or args.profile) else MAX_BLOCKS
    for b in range(max_blocks):
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        mt.mt_set_kernel_timing(3)      # events around the layer executors (the dominant kernel) on every 4th step
        w0 = time.time()
        before = mt.mt_debug_launch_count()
        e0.record(stream)
        for i in range(steps):
            step(i)
        mt.mt_set_kernel_timing(0)      # closes the last group of executor launches: its stop event goes in here
        e1.record(stream)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        w1 = time.time()
        if b == 0:
            launches = mt.mt_debug_launch_count() - before      # kernels the library enqueued in the timed region
        ms = e0.elapsed_time(e1)
        blocks.append((ms, mt.mt_get_kernel_times(), w0, w1))
        total_ms += ms
        if total_ms >= SUSTAIN_MS:
            break
    sampler.stop()
    local_ms = blocks[0][0]

    # per-kernel breakdown of every launch of the path: a short separate pass (its events perturb small batches)
    mt.mt_set_kernel_timing(1)
    bd_steps = max(3, min(steps, 50))
    for i in range(bd_steps):
        step(i)
    torch.cuda.synchronize()
    mt.mt_set_kernel_timing(0)
    breakdown = mt.mt_get_kernel_times()
    units, ms = aggregate(n * steps, local_ms, world)

    # Workload 4's batch is bucketed inside its conv launch, so the timed conv kernel contains that sort.  For the conv
    # layers alone: the same steps once more with the bucketing as a launch of its own (right after the blocks above,
    # i.e. in the power-capped regime).
    alone = None
    if cfg == 4 and world == 1 and not args.profile:
        mt.mt_debug_set_option("conv_self_bucket", 0)
        for i in range(10):
            step(i)
        torch.cuda.synchronize()
        mt.mt_set_kernel_timing(3)
        e0.record(stream)
        for i in range(steps):
            step(i)
        mt.mt_set_kernel_timing(0)
        e1.record(stream)
        torch.cuda.synchronize()
        alone = (e0.elapsed_time(e1) / steps, mt.mt_get_kernel_times())
        mt.mt_debug_set_option("conv_self_bucket", 1)

    if args.profile:
        mt.mt_shutdown()
        return {"profile_run": True, "ms_per_step": ms / steps, "kernels": {nm: t / max(c, 1) for nm, t, c in breakdown}}

    # launch floor: a chain of empty kernels launched like the kernels of the path
    floor_us = None
    if world == 1:
        mt.mt_debug_empty_launches(200, stream)
        torch.cuda.synchronize()
        e0.record(stream)
        mt.mt_debug_empty_launches(2000, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        floor_us = e0.elapsed_time(e1) / 2000 * 1e3

    # ---- end to end: host buffers in, host buffers out, through the public entry points.  Every step copies its
    # inputs and ids from pinned host memory and its outputs back.  Primary figure: mt_infer_host_async on two
    # alternating streams (a batch's copies overlap its neighbours' kernels); beside it the synchronous
    # mt_infer_host, which returns only when the outputs have landed.
    e2e_steps = args.e2e_steps or max(4, min(steps, 50))
    h_in = [torch.from_numpy(x.view(np.int16)).pin_memory() for _, x in batches]
    h_ids = [torch.from_numpy(i).pin_memory() for i, _ in batches]
    h_outs = [torch.empty((n, out_elems), dtype=torch.float32).pin_memory() for _ in range(2)]
    h_out = h_outs[0]
    for i in range(3):
        mt.mt_infer_host(h_in[i % N_INPUT_BUFFERS], h_ids[i % N_INPUT_BUFFERS], n, h_out, stream)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0.record(stream)
    for i in range(e2e_steps):
        b = i % N_INPUT_BUFFERS
        mt.mt_infer_host(h_in[b], h_ids[b], n, h_out, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    sync_units, sync_ms = aggregate(n * e2e_steps, e0.elapsed_time(e1), world)
    two = [torch.cuda.Stream(), torch.cuda.Stream()]
    for i in range(4):
        mt.mt_infer_host_async(h_in[i % N_INPUT_BUFFERS], h_ids[i % N_INPUT_BUFFERS], n, h_outs[i % 2], two[i % 2])
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0.record(two[0])
    for i in range(e2e_steps):
        b = i % N_INPUT_BUFFERS
        mt.mt_infer_host_async(h_in[b], h_ids[b], n, h_outs[i % 2], two[i % 2])
    two[0].wait_stream(two[1])
    e1.record(two[0])
    torch.cuda.synchronize()
    e2e_units, e2e_ms = aggregate(n * e2e_steps, e0.elapsed_time(e1), world)
    checksum = float(h_out.double().abs().sum())
    if not np.isfinite(checksum):
        raise SystemExit("non-finite outputs")
    st = mt.mt_get_async_status()
    if st != (0, -1):
        raise SystemExit("device status after the timed region: %r" % (st,))
    mt.mt_shutdown()
    del dev_in, dev_ids, dev_out, h_in, h_ids, h_outs
    torch.cuda.empty_cache()
    if rank != 0:
        return None

    per_kernel = {name: {"ms_per_step": t / bd_steps, "launches_per_step": c / bd_steps} for name, t, c in breakdown}
    lps = {nm: c / bd_steps for nm, t, c in breakdown}
    dom = "grouped_conv3x3" if cfg == 4 else ("fused_mlp" if "fused_mlp" in lps else "grouped_gemm")

    def dom_ms(kernel_times):
        # per step = per-launch average x launches per step (the executors are timed on every fourth step)
        for nm, t, c in kernel_times:
            if nm == dom:
                return t / max(c, 1) * lps.get(nm, 1.0)
        return 0.0

    block_ms = [b[0] / steps for b in blocks]
    block_clk = [sampler.summary(b[2], b[3]) for b in blocks]
    block_dom = [dom_ms(b[1]) for b in blocks]
    long_first = blocks[0][0] >= 1000.0
    roof = dominant_roofline(wl, block_dom[0], peaks, peaks_kind, cfg, long_first)
    roof["kernel"] = dom
    roof["kernel_timing"] = "CUDA events around each run of the executor's launches, every 4th step of the timed region"
    line = result_line(units, ms, steps, n_gpus=world, steps=steps, warmup=args.warmup, scaling="weak",
                       vs_baseline=None, dtype="bf16", data="synthetic")
    line["config"] = {"workload": synth.CONFIG_NAMES[cfg], "requests_per_step_per_gpu": n, "tenants": len(models),
                      "reduced": bool(args.tenants or args.requests), "residual_blocks": bool(args.shortcuts and cfg == 4),
                      "l2": "weights streamed per step exceed the 126 MB L2 only for c2/c3/c5; inputs rotate over "
                            "%d device buffers" % N_INPUT_BUFFERS,
                      "parallelism": "replicas x%d (each GPU hosts all tenants, own batch)" % world}
    flops = synth.workload_flops(wl.models, wl.model_ids)
    bytes_all = synth.workload_bytes(wl.models, wl.model_ids)
    line["tflops"] = flops * steps * world / (ms * 1e-3) / 1e12

    def whole_pass(ms_per_step, long_run):
        tc = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) if long_run else peaks["bf16_tflops"]
        t_roof = max(flops / (tc * 1e12), bytes_all / (peaks["hbm_gbs"] * 1e9))
        return {"roofline_ms": t_roof * 1e3, "measured_ms": ms_per_step, "frac": t_roof * 1e3 / ms_per_step,
                "peaks": "of " + peaks_kind + (", tensor peak sustained" if long_run else ", tensor peak burst"),
                "flops_per_step": int(flops), "algorithmic_bytes_per_step": int(bytes_all)}

    line["whole_pass_roofline"] = whole_pass(line["ms_per_step"], long_first)
    line["roofline"] = roof
    if alone is not None:
        r2 = dominant_roofline(wl, dom_ms(alone[1]), peaks, peaks_kind, cfg, True)
        line["conv_layers_alone"] = {
            "note": "the same steps with the bucketing as a launch of its own (conv_self_bucket = 0), measured after the "
                    "repeated blocks (power-capped regime): the conv launch then holds the conv layers only",
            "ms_per_step": alone[0], "kernel_ms_per_step": r2["kernel_ms_per_step"], "achieved": r2["achieved"],
            "unit": r2["unit"], "frac_of_burst_peak": r2.get("frac_of_burst_peak"),
            "frac_of_sustained_peak": r2.get("frac_of_sustained_peak")}
    if len(blocks) > 1 or blocks[0][0] >= SUSTAIN_MS:
        # the later half of the blocks: the GPU has been busy for at least a second by then
        tail = list(range(len(blocks) // 2, len(blocks)))
        tail_ms = median([block_ms[i] for i in tail])
        tail_dom = median([block_dom[i] for i in tail])
        tail_clk = sampler.summary(blocks[tail[0]][2], blocks[tail[-1]][3])
        first_clk = block_clk[0]
        sus = {"blocks": len(blocks), "steps_per_block": steps, "device_seconds": total_ms * 1e-3,
               "ms_per_step": {"min": min(block_ms), "median": median(block_ms), "max": max(block_ms),
                               "first": block_ms[0], "last": block_ms[-1], "later_half_median": tail_ms},
               "value_later_half": n * world / (tail_ms * 1e-3),
               "sm_mhz": {"first_block": first_clk["sm_mhz"], "later_half": tail_clk["sm_mhz"]},
               "ms_x_mhz": {"first_block": (block_ms[0] * first_clk["sm_mhz"]) if first_clk["sm_mhz"] else None,
                            "later_half": (tail_ms * tail_clk["sm_mhz"]) if tail_clk["sm_mhz"] else None},
               "reasons_later_half": tail_clk["reasons"],
               "roofline_later_half": dominant_roofline(wl, tail_dom, peaks, peaks_kind, cfg, True),
               "whole_pass_roofline_later_half": whole_pass(tail_ms, True)}
        for k in ("traffic", "traffic_source", "algorithmic_bytes_per_step", "flops_per_step"):
            sus["roofline_later_half"].pop(k, None)
        line["sustained"] = sus
    line["kernels"] = per_kernel
    line["gpu_launches"] = int(launches)
    if floor_us is not None:
        line["launch_floor_us"] = floor_us
        line["launch_floor"] = ("one link of a chain of 2000 empty kernels launched like the kernels of the path "
                                "(programmatic dependent launch); this step has %d launches" % round(launches / steps))
    line["e2e"] = dict(result_line(e2e_units, e2e_ms, e2e_steps), steps=e2e_steps,
                       h2d_bytes_per_step=int(n * wl.in_elems * 2 + n * 4), d2h_bytes_per_step=int(n * out_elems * 4))
    line["e2e"]["call"] = "mt_infer_host_async, two streams in turn"
    line["e2e"]["synchronous_call"] = {"value": sync_units / (sync_ms * 1e-3), "unit": UNIT, "ms_per_step": sync_ms / e2e_steps,
                                       "call": "mt_infer_host"}
    for k in ("metric", "higher_is_better"):
        line["e2e"].pop(k, None)
    clocks = sampler.summary()
    clocks["timed_block"] = block_clk[0]
    clocks["period_ms"] = sampler.period_ms
    line["clocks"] = clocks
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = time_oracle(wl, cfg)
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=None, choices=[1, 2, 3, 4, 5],
                    help="only this workload (default: workload 2 as the headline and all five under per_config)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="headline workload only")
    ap.add_argument("--tenants", type=int, default=None, help="reduced case: number of tenants (profiling captures)")
    ap.add_argument("--requests", type=int, default=None, help="reduced case: requests per batch")
    ap.add_argument("--profile", action="store_true", help="timed loop only (no e2e, CPU baseline or clock sampler)")
    ap.add_argument("--shortcuts", action="store_true", help="workload 4 as two residual blocks: conv layers 1 and 3 add "
                    "the input of the layer before them (a variant, not the headline)")
    ap.add_argument("--cache-sweep", action="store_true", help="weight-residency leg: workload 2 behind a device cache "
                    "of 40-100 %% of its weights (prints its own JSON line)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank, world, local_rank = env_int("RANK", 0), env_int("WORLD_SIZE", 1), env_int("LOCAL_RANK", 0)
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_1901_06887_b200 import binding as mt, harness

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation")
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks, peaks_kind = load_peaks()
    ctx = dict(torch=torch, dist=dist, mt=mt, harness=harness, rank=rank, world=world, local_rank=local_rank,
               peaks=peaks, peaks_kind=peaks_kind)

    if args.cache_sweep:
        if rank == 0:
            run_cache_sweep(args, ctx)
        return
    head_cfg = args.config or HEADLINE_CONFIG
    line = measure_config(head_cfg, args, ctx)
    reduced = bool(args.tenants or args.requests or args.profile or args.shortcuts)
    if args.config is None and world == 1 and not reduced and not args.no_per_config and line is not None:
        # the same measurements for all five workloads; --steps applies to the headline only
        per = {"c%d" % head_cfg: {k: v for k, v in line.items() if k not in ("metric", "unit", "higher_is_better", "n_gpus",
                                                                              "scaling", "vs_baseline", "data")}}
        sub = argparse.Namespace(**vars(args))
        sub.steps = None
        sub.e2e_steps = None
        for cfg in (1, 3, 4, 5):
            r = measure_config(cfg, sub, ctx)
            per["c%d" % cfg] = {k: v for k, v in r.items() if k not in ("metric", "unit", "higher_is_better", "n_gpus",
                                                                         "scaling", "vs_baseline", "data")}
        line["per_config"] = {k: per[k] for k in sorted(per)}
    if rank == 0 and line is not None:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
