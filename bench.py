#!/usr/bin/env python
"""Benchmark of the mixed-tenant inference hot path.

One "step" = one mt_infer call: bucketing, one grouped launch per layer (the last one returns the rows to arrival order), over one synthetic
mixed batch.  Default workload: 64 tenants x MLP 1024-4096-4096-1024, 4096 requests, Zipf(1.1).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank hosts all tenants and runs its
own batch (requests of different batches are independent; no collective on the data path): weak scaling.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
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
DEFAULT_STEPS = {1: 20000, 2: 1500, 3: 2500, 4: 1500, 5: 50}
ORACLE_SAMPLE = {1: 64, 2: 2048, 3: 16384, 4: 24, 5: 96}      # requests of the batch the CPU baseline times
N_INPUT_BUFFERS = 3
# DRAM traffic of the dominant kernel from the ncu captures summarised under profiles/ (see there):
#   config 2: measured on a reduced case, traffic / algorithmic bytes = 0.995, scaled to the full launch;
#   config 4: measured at full size, bytes per step (four conv launches).  None = not captured.
TRAFFIC_RATIO = {2: 0.995}
TRAFFIC_BYTES = {4: 608.5e6}


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


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs (read-only queries)."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0])); mx.append(float(parts[1]))
                except ValueError:
                    continue
                for nm, v in zip(names, parts[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def gemm_roofline(wl, kernel_ms_per_launch_sum, peaks, peaks_kind, config):
    """Roofline of the dominant kernel (the grouped layer executor), all its launches of one step together:
    algorithmic bytes (weights + bias of tenants with requests once, activations in, activations out) and
    flops of those layers, against the measured HBM and bf16 peaks; the larger time bounds it."""
    per_layer_bytes = synth.workload_bytes(wl.models, wl.model_ids, per_layer=True)
    kinds = [l.kind for l in wl.models[0]]
    dom_kind = synth.CONV3X3 if synth.CONV3X3 in kinds else synth.DENSE
    counts = np.bincount(wl.model_ids, minlength=len(wl.models))
    byts = sum(b for b, k in zip(per_layer_bytes, kinds) if k == dom_kind)
    flops = sum(int(c) * sum(synth.layer_flops(l) for l in m if l.kind == dom_kind) for c, m in zip(counts, wl.models))
    # tensor peak: the kernel is timed inside a seconds-long loop (power cap active), so the sustained cuBLAS
    # figure is the matching denominator; the burst figure is reported beside it
    tc_peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    t_hbm = byts / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (tc_peak * 1e12)
    sec = kernel_ms_per_launch_sum * 1e-3
    if t_hbm >= t_tc:
        ach = byts / sec / 1e9 if sec > 0 else 0.0
        roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"]}
    else:
        ach = flops / sec / 1e12 if sec > 0 else 0.0
        roof = {"bound": "tensor", "achieved": ach, "peak": tc_peak, "unit": "TFLOP/s", "frac": ach / tc_peak,
                "peak_kind": "sustained (kernel timed inside a long loop)", "burst_peak": peaks["bf16_tflops"],
                "frac_of_burst_peak": ach / peaks["bf16_tflops"]}
    traffic = None
    if config in TRAFFIC_RATIO:
        traffic = int(TRAFFIC_RATIO[config] * byts)
    elif config in TRAFFIC_BYTES:
        traffic = int(TRAFFIC_BYTES[config])
    roof.update(traffic=traffic, peak_source="of " + peaks_kind, kernel="grouped_conv3x3" if dom_kind == synth.CONV3X3 else "grouped_gemm",
                algorithmic_bytes_per_step=int(byts), flops_per_step=int(flops), kernel_ms_per_step=kernel_ms_per_launch_sum)
    return roof


def time_oracle(wl, config, n_sample=None, repeats=1):
    import oracle
    oracle.build()
    n_s = min(wl.n, n_sample or ORACLE_SAMPLE[config])
    ids, x = wl.model_ids[:n_s], wl.inputs[:n_s]
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle.forward(wl.models, ids, x)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return {"value": n_s / best, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
            "sample": "first %d of %d requests of the batch, all tenants resident, wall clock %.2f s" % (n_s, wl.n, best)}


def run_reference(args, rank, world):
    """The reference arm: the fp64 CPU oracle as it stands, on the host cores, rank 0 only."""
    if rank != 0:
        return
    wl = synth.make_workload(args.config)
    n_s = min(wl.n, max(1, ORACLE_SAMPLE[args.config] // 4))
    import oracle
    oracle.build()
    ids, x = wl.model_ids[:n_s], wl.inputs[:n_s]
    for _ in range(min(args.warmup, 1)):
        oracle.forward(wl.models, ids, x)
    steps = min(args.steps, 8)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.forward(wl.models, ids, x)
    ms = (time.perf_counter() - t0) * 1e3
    line = result_line(n_s * steps, ms, steps, n_gpus=args.gpus, steps=steps, warmup=min(args.warmup, 1), scaling="weak",
                       vs_baseline=None, dtype="f64", data="synthetic", impl="reference",
                       config={"workload": synth.CONFIG_NAMES[args.config],
                               "sample": "each step = first %d of %d requests" % (n_s, wl.n)})
    line["cpu_baseline"] = {"value": line["value"], "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
                            "sample": "first %d of %d requests per step, %d steps" % (n_s, wl.n, steps)}
    line["e2e"] = {"value": line["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tenants", type=int, default=None, help="reduced case: number of tenants (profiling captures)")
    ap.add_argument("--requests", type=int, default=None, help="reduced case: requests per batch")
    ap.add_argument("--profile", action="store_true", help="timed loop only (no e2e, CPU baseline or clock sampler)")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = DEFAULT_STEPS[args.config]
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

    cfg = args.config
    over = {"n_tenants": args.tenants} if args.tenants else {}
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

    # ---- timed region: device-resident inputs, CUDA events on the launching stream, per-kernel events inside
    sampler = ClockSampler(local_rank)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    mt.mt_set_kernel_timing(3)          # events around the layer executors (the dominant kernel) on every 4th step
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    if not args.profile:
        sampler.start()
    launches_before = mt.mt_debug_launch_count()
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    mt.mt_set_kernel_timing(0)          # closes the last group of executor launches: its stop event goes in here
    e1.record(stream)
    torch.cuda.synchronize()
    launches = mt.mt_debug_launch_count() - launches_before      # kernels the library enqueued in the timed region
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    local_ms = e0.elapsed_time(e1)
    kernel_times = mt.mt_get_kernel_times()
    # per-kernel breakdown of every launch of the path: a short separate pass (its events perturb small batches)
    mt.mt_set_kernel_timing(1)
    bd_steps = max(3, min(args.steps, 50))
    for i in range(bd_steps):
        step(i)
    torch.cuda.synchronize()
    mt.mt_set_kernel_timing(0)
    breakdown = mt.mt_get_kernel_times()
    units, ms = aggregate(n * args.steps, local_ms, world)

    if args.profile:
        if rank == 0:
            print(json.dumps({"profile_run": True, "ms_per_step": ms / args.steps,
                              "kernels": {nm: t / max(c, 1) for nm, t, c in breakdown}}), flush=True)
        mt.mt_shutdown()
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- end to end: host buffers in, host buffers out, through the public entry points.  Every step copies its
    # inputs and ids from pinned host memory and its outputs back.  Primary figure: mt_infer_host_async on two
    # alternating streams (a batch's copies overlap its neighbours' kernels); beside it the synchronous
    # mt_infer_host, which returns only when the outputs have landed.
    e2e_steps = args.e2e_steps or max(4, min(args.steps, 50))
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

    if rank == 0:
        peaks, peaks_kind = load_peaks()
        per_kernel = {name: {"ms_per_step": t / bd_steps, "launches_per_step": c / bd_steps} for name, t, c in breakdown}
        # per step = per-launch average x launches per step (the executors are timed on every fourth step)
        lps = {nm: c / bd_steps for nm, t, c in breakdown}
        timed = dict((nm, t / max(c, 1) * lps.get(nm, 1.0)) for nm, t, c in kernel_times)
        dom = "grouped_conv3x3" if cfg == 4 else ("fused_mlp" if "fused_mlp" in timed else "grouped_gemm")
        dom_ms = timed.get(dom, 0.0)
        roof = gemm_roofline(wl, dom_ms, peaks, peaks_kind, cfg)
        roof["kernel"] = dom
        roof["kernel_timing"] = "CUDA events around each run of the executor's launches, every 4th step of the timed region"
        flops = synth.workload_flops(wl.models, wl.model_ids)
        bytes_all = synth.workload_bytes(wl.models, wl.model_ids)
        t_roof = max(flops / (peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * 1e12),
                     bytes_all / (peaks["hbm_gbs"] * 1e9))
        line = result_line(units, ms, args.steps, n_gpus=world, steps=args.steps, warmup=args.warmup, scaling="weak",
                           vs_baseline=None, dtype="bf16", data="synthetic")
        line["config"] = {"workload": synth.CONFIG_NAMES[cfg], "requests_per_step_per_gpu": n, "tenants": len(models),
                          "reduced": bool(args.tenants or args.requests),
                          "l2": "weights streamed per step exceed the 126 MB L2 only for c2/c3/c5; inputs rotate over "
                                "%d device buffers" % N_INPUT_BUFFERS,
                          "parallelism": "replicas x%d (each GPU hosts all tenants, own batch)" % world}
        line["tflops"] = flops * args.steps * world / (ms * 1e-3) / 1e12
        line["whole_pass_roofline"] = {"roofline_ms": t_roof * 1e3, "measured_ms": line["ms_per_step"],
                                       "frac": t_roof * 1e3 / line["ms_per_step"], "peaks": "of " + peaks_kind,
                                       "flops_per_step": int(flops), "algorithmic_bytes_per_step": int(bytes_all)}
        line["roofline"] = roof
        line["kernels"] = per_kernel
        line["gpu_launches"] = int(launches)
        line["e2e"] = dict(result_line(e2e_units, e2e_ms, e2e_steps), steps=e2e_steps,
                           h2d_bytes_per_step=int(n * wl.in_elems * 2 + n * 4), d2h_bytes_per_step=int(n * out_elems * 4))
        line["e2e"]["call"] = "mt_infer_host_async, two streams in turn"
        line["e2e"]["synchronous_call"] = {"value": sync_units / (sync_ms * 1e-3), "unit": UNIT, "ms_per_step": sync_ms / e2e_steps,
                                           "call": "mt_infer_host"}
        for k in ("metric", "higher_is_better"):
            line["e2e"].pop(k, None)
        line["clocks"] = clocks
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = time_oracle(wl, cfg)
        print(json.dumps(line), flush=True)
    mt.mt_shutdown()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
