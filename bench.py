#!/usr/bin/env python
"""Benchmark of the ZipLine barrier-selection search.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--workload c4] [--objective range|sum]

A step is one pass of the whole hot path (prologue, sweep, finalize) over one batch of synthetic
input.  The default workload is the n=1024, R=1024, B=64 configuration (512 MiB of int64
timestamps per step, larger than L2).  One JSON line is printed by rank 0.

With N > 1 (launched through torch.distributed.run) every rank runs the same-sized batch on its
own GPU with its own instance seeds: the batch dimension shards, there is no data-path
collective, and ``value`` is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import zl_inputs  # noqa: E402

METRIC = "ZipLine timestamps/sec (selections/sec in config) at 1 B200; achieved HBM GB/s vs peak"
CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def recorded_traffic(key):
    """DRAM bytes per launch from the committed ncu capture, or None once the kernel sources have changed since."""
    import hashlib
    try:
        rec = {}
        with open(os.path.join(ROOT, "profiles", "k_filter_c4_traffic.txt")) as f:
            for line in f:
                if line.strip() and not line.startswith("#"):
                    k, v = line.split()
                    rec[k] = v
        hsh = hashlib.sha256()
        for name in ("zipline.cu", "zl_device.cuh"):
            with open(os.path.join(ROOT, "paper_2001_01347_b200", "csrc", name), "rb") as f:
                hsh.update(f.read())
        return int(rec[key]) if rec.get("source_sha256") == hsh.hexdigest() and key in rec else None
    except Exception:
        return None


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi in the background while the timed region runs."""

    def __init__(self, device_index: int):
        self.idx, self.proc, self.path = device_index, None, f"/tmp/zl_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.idx}", f"--query-gpu={CLOCK_QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        for line in open(self.path):
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [x for x in sm if x >= 0.5 * max(sm)] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_sample(ts: np.ndarray, objective: int, max_instances: int, budget_s: float):
    """Time the oracle's sweep on up to max_instances instances, one thread per host core."""
    from concurrent.futures import ThreadPoolExecutor

    import oracle
    cores = os.cpu_count() or 1
    B = min(ts.shape[0], max_instances)
    t_one = time.perf_counter()
    oracle.sweep_window(ts[0], objective)                       # also sizes the sample
    t_one = time.perf_counter() - t_one
    B = max(1, min(B, int(budget_s * cores / max(t_one, 1e-6))))
    threads = min(cores, B)
    t0 = time.perf_counter()
    with ThreadPoolExecutor(threads) as ex:
        list(ex.map(lambda b: oracle.sweep_window(ts[b], objective), range(B)))
    dt = time.perf_counter() - t0
    return B, threads, dt


def run_reference(args, w, objective):
    """The oracle, as it stands, on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    ts = zl_inputs.generate(w, B=min(w.B, 16))
    per_step = []
    used = (0, 0)
    for s in range(args.warmup + args.steps):
        B, threads, dt = oracle_sample(ts, objective, max_instances=16, budget_s=4.0)
        used = (B, threads)
        if s >= args.warmup:
            per_step.append(dt / B)                             # seconds per instance
    sec_inst = statistics.mean(per_step)
    value = w.n * w.R / sec_inst
    sample = f"{used[0]} of {w.B} instances of {w.name} per step, sweep_window, {used[1]} threads"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "timestamps/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec_inst * w.B * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
            "data": "synthetic", "config": workload_config(w, objective, args.gpus),
            "cpu_baseline": {"value": value, "unit": "timestamps/s", "cores": used[1], "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "timestamps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def workload_config(w, objective, gpus):
    return {"workload": f"{w.name}: n={w.n} workers, R={w.R} lookahead, B={w.B} instances per GPU per step",
            "n": w.n, "R": w.R, "B": w.B, "objective": "range" if objective == 0 else "sum",
            "input_bytes_per_step_per_gpu": w.timestamps * 8, "l2": "inputs larger than L2 (no flush needed)"
            if w.timestamps * 8 > 200e6 else "inputs rotate over copies larger than L2",
            "parallelism": f"batch sharded over {gpus} GPU(s), no collective"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="zipline", choices=["zipline", "reference"])
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--objective", default="range", choices=["range", "sum"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--opt", action="append", default=[], help="library option key=value")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "zipline" else args.warmup
    w = zl_inputs.CONFIGS[args.workload]
    objective = 0 if args.objective == "range" else 1

    if args.impl == "reference":
        run_reference(args, w, objective)
        return

    import torch
    import torch.distributed as dist

    import paper_2001_01347_b200 as zl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the ZipLine kernels have no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # ---- inputs: this rank's shard of the global batch (instances rank*B .. rank*B+B-1)
    ts_np = zl_inputs.generate(w, first_instance=rank * w.B)
    copies = max(1, int(np.ceil(300e6 / ts_np.nbytes)))        # rotate when one batch would fit in L2
    d_ts = [torch.from_numpy(ts_np).to(dev)]
    for c in range(1, copies):
        d_ts.append(d_ts[0].clone())
    h_pinned = torch.from_numpy(ts_np).pin_memory()
    nts = w.timestamps

    def make_handle(flags):
        h = zl.ZipLine(w.n, w.R, w.B, objective, local, flags)
        for kv in args.opt:
            k, v = kv.split("=")
            h.set_option(k, int(v))
        return h

    def timed(h, steps, warmup, host=False, profile=False):
        sel = None

        def step(i):
            nonlocal sel
            sel = h.select_batched_host(h_pinned, sel) if host else h.select_batched(d_ts[i % copies], sel)

        for i in range(warmup):
            step(i)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if profile:
            h.profile_begin(steps)
        t0 = time.perf_counter()
        e0.record()
        for i in range(steps):
            step(i)
        e1.record()
        torch.cuda.synchronize()
        wall_ms = (time.perf_counter() - t0) * 1e3
        ms = wall_ms if host else e0.elapsed_time(e1)          # the host path runs on the library's own stream
        prof = None
        if profile:
            prof = h.profile_read()
            h.profile_end()
        if world > 1:
            t = torch.tensor([ms], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
            dist.barrier()
        return ms, prof, sel

    sampler = ClockSampler(local)
    h = make_handle(0)
    sampler.start()
    ms, _, sel = timed(h, args.steps, args.warmup)                       # the headline: no per-stage events in the stream
    psteps = max(3, min(args.steps, 50))
    _, prof, _ = timed(h, psteps, 3, profile=True)                       # per-stage CUDA events (they serialise the stages)
    status_ok = bool((sel.status == 0).all().item())
    launches = h.launches_per_call * args.steps
    ms_step = ms / args.steps
    value = world * nts / (ms_step * 1e-3)

    # the same search when every timestamp is examined (no early stop)
    hf = make_handle(zl.ZL_FLAG_FULL_SWEEP)
    steps_f = max(3, args.steps // 2)
    ms_f, _, _ = timed(hf, steps_f, 3)
    _, prof_f, _ = timed(hf, psteps, 3, profile=True)
    hf.destroy()
    clocks = sampler.stop()

    # what the memory system delivers for the bytes of the filter pass: a kernel that only loads them (a warp per row, the
    # row prefixes the early stop needs, then whole rows), with the L2 flushed before each launch and as run back to back
    probe = None
    if rank == 0 and h.route == 1:
        lmin_row = ts_np[:, :, -1].min(axis=1)
        cnt = (ts_np <= lmin_row[:, None, None]).sum(axis=2).astype(np.int64)
        pref = np.minimum(w.R, (cnt + 8 + 7) // 8 * 8).astype(np.int32).reshape(-1)     # as the filter pass requests them
        d_pref = torch.from_numpy(pref).to(dev)
        d_full = torch.full_like(d_pref, w.R)
        sink = torch.zeros(1, dtype=torch.int64, device=dev)
        flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

        def probe_us(counts, cold, reps=10):
            tot = 0.0
            for i in range(reps + 2):
                if cold:
                    flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                zl.zl_probe_read_batched(d_ts[i % copies], counts, sink)
                b.record()
                torch.cuda.synchronize()
                if i >= 2:
                    tot += a.elapsed_time(b)
            return tot / reps * 1e3
        probe = {"prefix_bytes": int(pref.astype(np.int64).sum()) * 8,
                 "prefix_us_cold_l2": probe_us(d_pref, True), "prefix_us": probe_us(d_pref, False),
                 "full_bytes": nts * 8, "full_us_cold_l2": probe_us(d_full, True), "full_us": probe_us(d_full, False),
                 "what": "load-only kernel on the bytes of the filter pass (row prefixes up to the first exhausted row, "
                         "then whole rows); cold = 256 MB written before each launch"}
        del flush

    # end to end: host buffers in, host results out, through the C ABI
    e2e_steps = max(3, min(args.steps, 10))
    ms_e, _, _ = timed(h, e2e_steps, 3, host=True)
    e2e_value = world * nts / (ms_e / e2e_steps * 1e-3)
    h_route = h.route
    h.destroy()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (the sweep), algorithmic bytes = 8 per timestamp it must examine
    peak, peak_kind = measured_peak_gbs()
    lmin = ts_np[:, :, -1].min(axis=1)
    route = h_route                                  # 0 segment sweep only, 1 RANGE filter route, 2 bucket route
    examined = int((ts_np <= lmin[:, None, None]).sum()) if route == 1 else nts
    def dominant(pr):
        if route == 1:
            names = ("k_prologue", "k_filter", "k_tail+k_tilemax+k_cellscan+k_refine+k_buckets+k_sweep", "k_finalize")
        elif route == 2:
            names = ("k_prologue", "k_sum_plan+k_sum_index", "k_sum_buckets+k_sweep", "k_finalize")
        else:
            names = ("k_prologue", "-", "k_sweep", "k_finalize")
        stages = dict(zip(names, (pr["ms_prologue"], pr["ms_filter"], pr["ms_sweep"], pr["ms_finalize"])))
        name = max(stages, key=stages.get)
        return name, stages[name] / pr["calls"]

    dom, sweep_ms = dominant(prof)
    ach = examined * 8 / (sweep_ms * 1e-3) / 1e9
    dom_f, sweep_ms_f = dominant(prof_f)
    ach_f = nts * 8 / (sweep_ms_f * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dom, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                "peak_kind": f"{peak_kind} copy bandwidth",
                "traffic": recorded_traffic(f"{w.name}_{args.objective}_default_{dom}"),
                "bytes_per_launch": examined * 8, "ms_per_launch": sweep_ms,
                "bytes_model": "8 B per timestamp not after the first exhausted row (the search stops there)"
                if route == 1 else "8 B per timestamp"}
    full = {"value": nts / (ms_f / steps_f * 1e-3), "unit": "timestamps/s", "ms_per_step": ms_f / steps_f,
            "roofline": {"bound": "hbm", "kernel": dom_f, "achieved": ach_f, "peak": peak, "unit": "GB/s",
                         "frac": ach_f / peak, "bytes_per_launch": nts * 8, "ms_per_launch": sweep_ms_f,
                         "traffic": recorded_traffic(f"{w.name}_{args.objective}_full_{dom_f}")}}

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        Bs, threads, dt = oracle_sample(ts_np, objective, max_instances=w.B, budget_s=20.0)
        cpu = {"value": Bs * w.n * w.R / dt, "unit": "timestamps/s", "cores": threads, "kind": "oracle",
               "sample": f"{Bs} of {w.B} instances of {w.name}, sweep_window (sort + one pass), {dt:.1f} s wall"}

    cfg = workload_config(w, objective, world)
    cfg.update({"selections_per_s": world * w.B / (ms_step * 1e-3), "early_stop": route == 1,
                "route": {0: "segment sweep", 1: "filter", 2: "buckets"}[route],
                "examined_fraction": examined / nts, "segments_per_instance": None,
                "kernel_ms": {k[3:]: prof[k] / prof["calls"] for k in ("ms_prologue", "ms_filter", "ms_sweep", "ms_finalize")},
                "kernel_ms_full_sweep": {k[3:]: prof_f[k] / prof_f["calls"]
                                         for k in ("ms_prologue", "ms_filter", "ms_sweep", "ms_finalize")},
                "all_status_ok": status_ok, "options": args.opt})
    line = {"metric": METRIC, "value": value, "unit": "timestamps/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int64", "data": "synthetic", "config": cfg, "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "timestamps/s", "h2d_bytes_per_step": nts * 8,
                    "d2h_bytes_per_step": w.B * (4 * w.n + 20), "ms_per_step": ms_e / e2e_steps},
            "gpu_launches": launches, "roofline": roofline, "full_sweep": full, "cpu_baseline": cpu,
            "load_only_probe": probe}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
