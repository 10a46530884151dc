#!/usr/bin/env python
"""Benchmark of the ZipLine barrier-selection search.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--workload c4] [--objective range|sum]

A step is one pass of the whole hot path (one ``zl_select_batched`` call) over one batch of synthetic
input.  The default workload is the n=1024, R=1024, B=64 configuration (512 MiB of int64 timestamps per
step).  Each of the K timed steps is measured with its own pair of CUDA events around ``inner`` consecutive
calls (so that the timed region lasts at least 0.1 s whatever K is) and reported as time per call; the
inputs rotate over as many copies as it takes for the bytes a call examines, times the copies, to exceed
the L2 several times over.  One JSON line is printed by rank 0.

With N > 1 (launched through torch.distributed.run) every rank runs the same-sized batch on its
own GPU with its own instance seeds: the batch dimension shards, there is no data-path
collective, and ``value`` is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import glob
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

METRIC = "ZipLine timestamps/sec (selections/sec in result) at 1 B200; achieved HBM GB/s vs peak"
NOMINAL_GBS = 8000.0                   # the HBM3e figure the target is quoted against
MIN_TIMED_MS = 100.0
CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def recorded_traffic(key):
    """DRAM bytes per launch from the committed ncu capture, or None once the kernel sources have changed since."""
    import hashlib
    try:
        rec = {}
        with open(os.path.join(ROOT, "profiles", "traffic.txt")) as f:
            for line in f:
                if line.strip() and not line.startswith("#"):
                    k, v = line.split()
                    rec[k] = v
        # the sources that make up the recorded kernel (k_filter): its file and the device headers it includes
        hsh = hashlib.sha256()
        csrc = os.path.join(ROOT, "paper_2001_01347_b200", "csrc")
        for name in ("filter.cu", "zl_batch.cuh", "zl_device.cuh", "zl_guard.cuh", "zl_types.cuh"):
            with open(os.path.join(csrc, name), "rb") as f:
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


def oracle_sample(ts: np.ndarray, objective: int, instances: int):
    """Time the oracle's sweep on the first `instances` instances, one thread per host core."""
    from concurrent.futures import ThreadPoolExecutor

    import oracle
    cores = os.cpu_count() or 1
    threads = min(cores, instances)
    t0 = time.perf_counter()
    with ThreadPoolExecutor(threads) as ex:
        list(ex.map(lambda b: oracle.sweep_window(ts[b], objective), range(instances)))
    return threads, time.perf_counter() - t0


def oracle_sample_size(ts: np.ndarray, objective: int, budget_s: float) -> int:
    """How many instances of the batch the oracle gets through in about budget_s seconds on the host cores."""
    import oracle
    t = time.perf_counter()
    oracle.sweep_window(ts[0], objective)
    t = max(time.perf_counter() - t, 1e-6)
    return max(1, min(ts.shape[0], int(budget_s * (os.cpu_count() or 1) / t)))


def workload_config(w, objective, gpus):
    return {"workload": f"{w.name}: n={w.n} workers, R={w.R} lookahead, B={w.B} instances per GPU per step",
            "n": w.n, "R": w.R, "B": w.B, "objective": "range" if objective == 0 else "sum",
            "input_bytes_per_step_per_gpu": w.timestamps * 8,
            "l2": "inputs rotate over copies so that the bytes one call examines x copies exceed 300 MB (more than twice the L2)",
            "parallelism": f"batch sharded over {gpus} GPU(s), no collective"}


def run_reference(args, w, objective):
    """The oracle, as it stands, on the host cores (rank 0 only): every step sweeps the same bounded sample of the batch."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    ts = zl_inputs.generate(w)
    total = max(1, args.steps + args.warmup)
    inst = oracle_sample_size(ts, objective, budget_s=min(8.0, 120.0 / total))
    per_step, threads = [], 1
    for s in range(args.warmup + args.steps):
        threads, dt = oracle_sample(ts, objective, inst)
        if s >= args.warmup:
            per_step.append(dt)
    sec = statistics.median(per_step)
    value = inst * w.n * w.R / sec
    sample = f"the first {inst} of {w.B} instances of {w.name} per step, sweep_window (sort + one pass), {threads} threads"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "timestamps/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
            "data": "synthetic", "config": workload_config(w, objective, args.gpus),
            "timing": {"ms_per_step_median": sec * 1e3, "ms_per_step_min": min(per_step) * 1e3, "ms_per_step_max": max(per_step) * 1e3,
                       "what": "one step = the oracle on the sample named in cpu_baseline.sample (not extrapolated to the batch)"},
            "cpu_baseline": {"value": value, "unit": "timestamps/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "timestamps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


STAGES = {  # names of what runs between the library's stage events, by route
    1: ("k_range_head", "k_filter", "k_tail", "k_range_rest"),     # large shapes: the last stage is one kernel per phase
    2: ("k_prologue", "k_sum_plan+k_sum_index", "k_sum_buckets+k_sweep", "k_finalize"),
    0: ("k_prologue", "-", "k_sweep", "k_finalize"),
    3: ("k_small", "-", "-", "-"),
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="zipline", choices=["zipline", "reference"])
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--objective", default="range", choices=["range", "sum"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-probe", action="store_true")
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
    nts = w.timestamps
    lmin_inst = ts_np[:, :, -1].min(axis=1)
    examined_early = int((ts_np <= lmin_inst[:, None, None]).sum())      # timestamps not after the first exhausted row

    def make_handle(flags):
        h = zl.ZipLine(w.n, w.R, w.B, objective, local, flags)
        for kv in args.opt:
            k, v = kv.split("=")
            h.set_option(k, int(v))
        return h

    h = make_handle(0)
    route = h.route                                  # 0 segment sweep only, 1 RANGE filter route, 2 bucket route
    examined = examined_early if route == 1 else nts
    copies = max(1, min(16, int(np.ceil(300e6 / (examined * 8)))))
    d_ts = [torch.from_numpy(ts_np).to(dev)]
    for c in range(1, copies):
        d_ts.append(d_ts[0].clone())
    h_pinned = torch.from_numpy(ts_np).pin_memory()

    def timed(h, steps, warmup, host=False, profile=False, inner=None):
        """Per-step times (ms per call) of `steps` samples of `inner` calls each; inner is sized from the warm-up."""
        sel = None
        k = 0

        def call():
            nonlocal sel, k
            sel = h.select_batched_host(h_pinned, sel) if host else h.select_batched(d_ts[k % copies], sel)
            k += 1

        for _ in range(warmup):
            call()
        torch.cuda.synchronize()
        if inner is None:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(8):
                call()
            b.record()
            torch.cuda.synchronize()
            est_ms = a.elapsed_time(b) / 8
            inner = 1 if host else max(1, int(np.ceil(1.3 * MIN_TIMED_MS / (steps * est_ms))))
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()
        if profile:
            h.profile_begin(steps * inner)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        t0 = time.perf_counter()
        for a, b in ev:
            a.record()
            for _ in range(inner):
                call()
            b.record()
        torch.cuda.synchronize()
        wall_ms = (time.perf_counter() - t0) * 1e3
        if host:                                                  # the host path runs on the library's own stream
            per = [wall_ms / steps] * steps
            total = wall_ms
        else:
            per = [a.elapsed_time(b) / inner for a, b in ev]
            total = ev[0][0].elapsed_time(ev[-1][1])
        prof = None
        if profile:
            prof = h.profile_read()
            h.profile_end()
        if world > 1:
            t = torch.tensor([total], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            total = float(t.item())
            dist.barrier()
        return {"per": per, "total_ms": total, "inner": inner, "calls": steps * inner, "prof": prof, "sel": sel}

    def spread(t):
        return {"inner_repeats": t["inner"], "samples": len(t["per"]), "timed_region_ms": t["total_ms"],
                "ms_per_step_median": statistics.median(t["per"]), "ms_per_step_min": min(t["per"]), "ms_per_step_max": max(t["per"])}

    sampler = ClockSampler(local)
    sampler.start()
    t_main = timed(h, args.steps, args.warmup)                           # the headline: no per-stage events in the stream
    t_prof = timed(h, max(3, min(args.steps, 20)), 3, profile=True, inner=max(1, t_main["inner"] // 4))   # stage events serialise the stages
    status_ok = bool((t_main["sel"].status == 0).all().item())
    launches = h.launches_per_call * t_main["calls"]
    ms_step = t_main["total_ms"] / t_main["calls"]
    value = world * nts / (ms_step * 1e-3)

    # the same search when every timestamp is examined (no early stop)
    hf = make_handle(zl.ZL_FLAG_FULL_SWEEP)
    t_full = timed(hf, max(3, args.steps // 2), 3)
    t_fprof = timed(hf, max(3, min(args.steps, 20)), 3, profile=True, inner=max(1, t_full["inner"] // 4))
    hf.destroy()
    clocks = sampler.stop()
    ms_full = t_full["total_ms"] / t_full["calls"]

    # what the memory system delivers for the bytes of the filter pass: a kernel that only loads them (a warp per row, the
    # row prefixes the early stop needs, then whole rows), over the same rotating copies
    probe = None
    if rank == 0 and route == 1 and not args.no_probe:
        cnt = (ts_np <= lmin_inst[:, None, None]).sum(axis=2).astype(np.int64)
        pref = np.minimum(w.R, (cnt + 8 + 7) // 8 * 8).astype(np.int32).reshape(-1)     # as the filter pass requests them
        d_pref = torch.from_numpy(pref).to(dev)
        d_full = torch.full_like(d_pref, w.R)
        sink = torch.zeros(1, dtype=torch.int64, device=dev)

        def probe_us(counts, reps=10, inner=8):
            best = []
            k = 0
            for i in range(reps + 2):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for _ in range(inner):
                    zl.zl_probe_read_batched(d_ts[k % copies], counts, sink)
                    k += 1
                b.record()
                torch.cuda.synchronize()
                if i >= 2:
                    best.append(a.elapsed_time(b) / inner * 1e3)
            return statistics.median(best)
        probe = {"prefix_bytes": int(pref.astype(np.int64).sum()) * 8, "prefix_us": probe_us(d_pref),
                 "full_bytes": nts * 8, "full_us": probe_us(d_full),
                 "what": "load-only kernel on the bytes of the filter pass (row prefixes up to the first exhausted row, "
                         "then whole rows), a warp per row, back to back over the rotating input copies"}

    # end to end: host buffers in, host results out, through the C ABI
    e2e_steps = max(3, min(args.steps, 10))
    t_e2e = timed(h, e2e_steps, 3, host=True)
    ms_e2e = t_e2e["total_ms"] / t_e2e["calls"]
    e2e_value = world * nts / (ms_e2e * 1e-3)
    h.destroy()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel: algorithmic bytes = 8 per timestamp it must examine
    peak, peak_kind = measured_peak_gbs()
    names = STAGES[route]

    def dominant(pr):
        stages = {}
        for nm, v in zip(names, (pr["ms_prologue"], pr["ms_filter"], pr["ms_sweep"], pr["ms_finalize"])):
            if nm != "-":
                stages[nm] = v
        name = max(stages, key=stages.get)
        return name, stages[name] / pr["calls"], {k: v / pr["calls"] for k, v in stages.items()}

    def fractions(nbytes, ms):
        gbs = nbytes / (ms * 1e-3) / 1e9
        return {"GB/s": gbs, "frac_of_measured": gbs / peak, "frac_of_nominal_8000": gbs / NOMINAL_GBS}

    dom, dom_ms, stage_ms = dominant(t_prof["prof"])
    ach = examined * 8 / (dom_ms * 1e-3) / 1e9
    dom_f, dom_ms_f, stage_ms_f = dominant(t_fprof["prof"])
    ach_f = nts * 8 / (dom_ms_f * 1e-3) / 1e9
    model = ("8 B per timestamp not after the first exhausted row (the search stops there)" if route == 1 else "8 B per timestamp")
    roofline = {"bound": "hbm", "kernel": dom, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                "peak_kind": f"{peak_kind} copy bandwidth", "frac_of_nominal_8000": ach / NOMINAL_GBS,
                "traffic": recorded_traffic(f"{w.name}_{args.objective}_default_{dom}"),
                "bytes_per_launch": examined * 8, "ms_per_launch": dom_ms, "bytes_model": model,
                "whole_call": {"examined_bytes": fractions(examined * 8, ms_step), "all_input_bytes": fractions(nts * 8, ms_step),
                               "what": "the same bytes divided by ms_per_step (every kernel of the call, launch gaps included)"}}
    full = {"value": world * nts / (ms_full * 1e-3), "unit": "timestamps/s", "ms_per_step": ms_full, "timing": spread(t_full),
            "what": "ZL_FLAG_FULL_SWEEP: every timestamp is examined, so timestamps/s and bytes/s count the same elements",
            "roofline": {"bound": "hbm", "kernel": dom_f, "achieved": ach_f, "peak": peak, "unit": "GB/s",
                         "frac": ach_f / peak, "frac_of_nominal_8000": ach_f / NOMINAL_GBS, "bytes_per_launch": nts * 8,
                         "ms_per_launch": dom_ms_f, "traffic": recorded_traffic(f"{w.name}_{args.objective}_full_{dom_f}"),
                         "whole_call": {"all_input_bytes": fractions(nts * 8, ms_full)}},
            "kernel_ms": stage_ms_f}

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        inst = oracle_sample_size(ts_np, objective, budget_s=20.0)
        threads, dt = oracle_sample(ts_np, objective, inst)
        cpu = {"value": inst * w.n * w.R / dt, "unit": "timestamps/s", "cores": threads, "kind": "oracle",
               "sample": f"the first {inst} of {w.B} instances of {w.name}, sweep_window (sort + one pass), {dt:.1f} s wall"}

    result = {"selections_per_s": world * w.B / (ms_step * 1e-3), "early_stop": route == 1,
              "route": {0: "segment sweep", 1: "filter", 2: "buckets", 3: "one launch"}[route],
              "examined_fraction": examined / nts, "input_copies": copies,
              "value_counts": "all n*R*B timestamps of the batch per call (nominal: the early stop examines examined_fraction of them; "
                              "full_sweep.value counts examined timestamps only)",
              "kernel_ms": stage_ms, "all_status_ok": status_ok, "options": args.opt}
    line = {"metric": METRIC, "value": value, "unit": "timestamps/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int64", "data": "synthetic", "config": workload_config(w, objective, world),
            "timing": spread(t_main), "result": result, "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "timestamps/s", "h2d_bytes_per_step": nts * 8,
                    "d2h_bytes_per_step": w.B * (4 * w.n + 20), "ms_per_step": ms_e2e},
            "gpu_launches": launches, "roofline": roofline, "full_sweep": full, "cpu_baseline": cpu,
            "load_only_probe": probe}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
