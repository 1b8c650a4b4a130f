#!/usr/bin/env python
"""Benchmark of the AdaScale gain-ratio step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one whole iteration (reduce + scalar part + update) over one batch of synthetic
gradients.  The metric is the algorithmic bytes of a step, P * (S * b_g + 24), divided by its
duration.  Rank 0 prints one JSON line.  With N > 1 every rank runs an independent replica on
its own GPU (the method has no cross-GPU exchange); the value is the sum over ranks divided
by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "adascale_step gradient GB/s and % of B200 HBM peak; step latency (us)"
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the reduce kernel, from the ncu
# captures summarised under profiles/ (same kernel build); None where no capture exists
NCU_TRAFFIC_BYTES = {"resnet18": 382.5e6, "resnet50": 852.9e6}
NCU_TRAFFIC_BYTES_FUSED = {"resnet18": 512.0e6}
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 * 1024 * 1024


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="resnet18")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="two-kernel", choices=["two-kernel", "fused"],
                    help="fused: lagged gain estimate, one kernel per step, P*(S*b_g+16) bytes")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def algorithmic_bytes(wl):
    bg = 2 if wl.grad_dtype == "bf16" else 4
    reduce_b = wl.P * (wl.S * bg + 4)   # S rows read, mean gradient written
    update_b = wl.P * 20                # gbar, w, v read; w, v written
    return reduce_b, update_b


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi sampling of SM clock and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def dist_setup(n):
    import torch
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return world, rank, local


def max_over_ranks(value, world, device=None):
    """Slowest rank's value (collective used for timing only, never on the data path)."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(local_ms, step_bytes, world, device=None):
    """(slowest rank's ms per step, GB/s summed over the replicas at that pace)."""
    ms = max_over_ranks(local_ms, world, device)
    return ms, world * step_bytes / (ms * 1e-3) / 1e9


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def oracle_rows(grads):
    return [[g.detach().cpu().contiguous().view(-1) for g in row] for row in grads]


def as_oracle_array(t):
    import numpy as np
    import torch
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def time_oracle(wl, grads_cpu, w_cpu, v_cpu, budget_s, max_steps, fraction=1.0):
    """Times the CPU oracle as it stands on (a column slice of) the workload."""
    import numpy as np
    import oracle
    cores = os.cpu_count() or 1
    orc = oracle.Oracle(wl.S, momentum=wl.momentum, weight_decay=wl.weight_decay, nthreads=cores)
    lr = oracle.make_lr(wl.lr.get("kind", "const"), eta0=wl.lr.get("eta0", 0.1), d=wl.lr.get("d", 1.0),
                        T_S1=wl.lr.get("T_S1", 1.0), milestones=wl.lr.get("milestones", ()))
    cut = [max(1, int(n * fraction)) if n else 0 for n in wl.numels]
    rows = [[as_oracle_array(g[:c]) for g, c in zip(row, cut)] for row in grads_cpu]
    w64 = [t[:c].numpy().astype(np.float64) for t, c in zip(w_cpu, cut)]
    v64 = [t[:c].numpy().astype(np.float64) for t, c in zip(v_cpu, cut)]
    bg = 2 if wl.grad_dtype == "bf16" else 4
    bytes_per_step = sum(cut) * (wl.S * bg + 24)
    times = []
    t_start = time.perf_counter()
    while len(times) < max_steps and (time.perf_counter() - t_start < budget_s or not times):
        t0 = time.perf_counter()
        orc.step(rows, w64, v64, lr)
        times.append(time.perf_counter() - t0)
    return times, bytes_per_step, cores


def run_reference(args, wl):
    """The CPU oracle on the host cores, rank 0 only."""
    import torch
    from paper_2007_05105_b200 import synthetic
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = args.steps if args.steps is not None else 5
    warmup = args.warmup if args.warmup is not None else 1
    src = synthetic.GradientSource(wl, device="cpu")
    grads = src.fill(0)
    wflat, vflat = src.init_params()
    w, v = src.views(wflat), src.views(vflat)
    # calibrate on 1/16 of the columns, then pick the slice that keeps the run to ~2 minutes
    t_cal, _, cores = time_oracle(wl, grads, w, v, budget_s=0.0, max_steps=1, fraction=1.0 / 16)
    est_full = t_cal[0] * 16
    fraction = 1.0
    while fraction > 1.0 / 1024 and est_full * fraction * (steps + warmup) > 120.0:
        fraction /= 2
    time_oracle(wl, grads, w, v, budget_s=1e9, max_steps=warmup, fraction=fraction)
    times, bytes_per_step, cores = time_oracle(wl, grads, w, v, budget_s=1e9, max_steps=steps, fraction=fraction)
    total = sum(times)
    value = bytes_per_step * len(times) / total / 1e9
    sample = "columns [0, %g * numel) of every tensor, all %d rows, %d steps" % (fraction, wl.S, len(times))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": len(times), "warmup": warmup, "ms_per_step": 1e3 * total / len(times) / fraction,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "P": wl.P, "tensors": len(wl.shapes), "S": wl.S, "grad_dtype": wl.grad_dtype,
                   "sample_fraction": fraction, "note": "ms_per_step is scaled to the whole workload"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, wl):
    import torch
    from paper_2007_05105_b200 import binding as B
    from paper_2007_05105_b200 import synthetic

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    world, rank, local = dist_setup(args.gpus)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    reduce_b, update_b = algorithmic_bytes(wl)
    fused = args.mode == "fused"
    if fused:  # S rows, w and v read, w and v written; the mean gradient never leaves the registers
        reduce_b, update_b = wl.P * (wl.S * (2 if wl.grad_dtype == "bf16" else 4) + 16), 0
    step_b = reduce_b + update_b
    est_ms = step_b / 6.0e9  # at ~6 TB/s
    steps = args.steps if args.steps is not None else max(20, min(2000, int(3000.0 / max(est_ms, 1e-3))))
    warmup = args.warmup if args.warmup is not None else max(3, min(20, steps // 10))

    src = synthetic.GradientSource(wl, device=dev)
    grads = src.fill(0)
    wflat, vflat = src.init_params()
    w, v = src.views(wflat), src.views(vflat)
    ada = B.AdaScale(src.numels, wl.S, wl.grad_dtype, momentum=wl.momentum, weight_decay=wl.weight_decay, device=local,
                     flags=(B.FLAG_LAGGED | B.FLAG_FUSED) if fused else 0)
    sched = B.make_schedule(wl.lr.get("kind", "const"), eta0=wl.lr.get("eta0", 0.1), d=wl.lr.get("d", 1.0),
                            T_S1=wl.lr.get("T_S1", 1.0), milestones=wl.lr.get("milestones", ()))
    gp, wp, vp = B.pointer_array(grads), B.pointer_array(w), B.pointer_array(v)
    stream = torch.cuda.current_stream(dev)
    sh = stream.cuda_stream  # passed explicitly: no per-call stream lookup on the host
    working_set = wl.P * ((2 if wl.grad_dtype == "bf16" else 4) * wl.S + 12)
    flush = None
    if working_set <= 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)

    def one_step():
        if flush is not None:
            flush.zero_()
        ada.step(gp, wp, vp, sched, sh)

    for _ in range(warmup):
        one_step()
    torch.cuda.synchronize(dev)

    # ---- whole-step timing: K steps, events on the launching stream
    sampler = ClockSampler(local)
    barrier(world)
    torch.cuda.synchronize(dev)
    if rank == 0:
        sampler.start()
    launches0 = ada.launch_count
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            ada.step(gp, wp, vp, sched, sh)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        local_ms = e0.elapsed_time(e1) / steps
    else:
        # working set near L2 size: flush between steps and time each step on its own
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in evs:
            flush.zero_()
            a.record(stream)
            ada.step(gp, wp, vp, sched, sh)
            b.record(stream)
        torch.cuda.synchronize(dev)
        local_ms = sum(a.elapsed_time(b) for a, b in evs) / steps
    launches = ada.launch_count - launches0
    barrier(world)
    torch.cuda.synchronize(dev)
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step, value = whole_job_value(local_ms, step_b, world, dev)

    # ---- per-kernel timing (separate pass: events between the two launches of a step)
    ksteps = min(steps, 200)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(ksteps)]
    for a, b, c in ev:
        if flush is not None:
            flush.zero_()
        a.record(stream)
        if fused:
            ada.step(gp, wp, vp, sched, sh)
            b.record(stream)
        else:
            ada.reduce(gp, sched, sh)
            b.record(stream)
            ada.update(wp, vp, sh)
        c.record(stream)
    torch.cuda.synchronize(dev)
    t_reduce = sum(a.elapsed_time(b) for a, b, c in ev) / ksteps
    t_update = sum(b.elapsed_time(c) for a, b, c in ev) / ksteps
    # the same kernels launched back to back on their own (no neighbour's dirty lines to write back)
    iso = {}
    if not fused:
        for name, call in (("reduce", lambda: ada.reduce(gp, sched, sh)), ("update", lambda: ada.update(wp, vp, sh))):
            i0, i1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(3):
                call()
            i0.record(stream)
            for _ in range(ksteps):
                call()
            i1.record(stream)
            torch.cuda.synchronize(dev)
            iso[name + "_us"] = i0.elapsed_time(i1) / ksteps * 1e3
    # small working sets: also the warm figure (no L2 flush, steps back to back)
    warm_ms = None
    if flush is not None:
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0.record(stream)
        for _ in range(steps):
            ada.step(gp, wp, vp, sched, sh)
        w1.record(stream)
        torch.cuda.synchronize(dev)
        warm_ms = w0.elapsed_time(w1) / steps
    peak, peak_kind = measured_peak()
    reduce_gbs = reduce_b / (t_reduce * 1e-3) / 1e9
    update_gbs = update_b / (t_update * 1e-3) / 1e9 if not fused else 0.0

    # ---- bandwidth ceilings of this GPU with the library's own trivial kernels
    ceilings = {}
    if rank == 0:
        nbytes = 1 << 30
        a = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        b = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        a.zero_(), b.zero_()
        for kind, name, moved in ((0, "read", nbytes), (1, "copy", 2 * nbytes), (2, "rmw", 3 * nbytes)):
            for _ in range(3):
                B.stream_probe(kind, a, b, nbytes, device=local)
            p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            p0.record(stream)
            for _ in range(10):
                B.stream_probe(kind, a, b, nbytes, device=local)
            p1.record(stream)
            torch.cuda.synchronize(dev)
            ceilings[name + "_gbs"] = moved * 10 / (p0.elapsed_time(p1) * 1e-3) / 1e9
        del a, b

    # ---- end to end: gradients start in pinned host memory, statistics come back
    e2e = None
    if not args.no_e2e:
        bg = 2 if wl.grad_dtype == "bf16" else 4
        h2d = wl.P * wl.S * bg
        host_rows = [torch.empty(src.flat_len, dtype=src.rows[0].dtype).pin_memory() for _ in range(wl.S)]
        for hr, dr in zip(host_rows, src.rows):
            hr.copy_(dr)
        hp = B.pointer_array([src.views(hr) for hr in host_rows])
        esteps = max(3, min(steps, int(20e9 / max(h2d, 1))))
        for _ in range(2):
            ada.step_host(hp, wp, vp, sched)
        barrier(world)
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        for _ in range(esteps):
            ada.step_host(hp, wp, vp, sched)   # returns after the device finished and the stats arrived
        torch.cuda.synchronize(dev)
        e_ms = (time.perf_counter() - t0) * 1e3 / esteps
        e_ms = max_over_ranks(e_ms, world, dev)
        e2e = {"value": world * step_b / (e_ms * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": 112, "ms_per_step": e_ms, "steps": esteps,
               "api": "adascale_step_host (pinned host gradients -> device staging -> step -> stats to host)"}
        del host_rows

    # ---- the CPU oracle on this machine's cores, rank 0, one GPU only
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        grads_cpu = oracle_rows(grads)
        w_cpu = [t.detach().cpu() for t in w]
        v_cpu = [t.detach().cpu() for t in v]
        t_cal, _, cores = time_oracle(wl, grads_cpu, w_cpu, v_cpu, budget_s=0.0, max_steps=1, fraction=1.0 / 16)
        fraction = 1.0
        while fraction > 1.0 / 1024 and t_cal[0] * 16 * fraction > 10.0:
            fraction /= 2
        times, bps, cores = time_oracle(wl, grads_cpu, w_cpu, v_cpu, budget_s=15.0, max_steps=50, fraction=fraction)
        cpu = {"value": bps * len(times) / sum(times) / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
               "sample": "columns [0, %g * numel) of every tensor, all %d rows, %d steps of the fp64 oracle "
                         "with OpenMP over columns" % (fraction, wl.S, len(times)),
               "s_per_step_scaled": sum(times) / len(times) / fraction}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_per_step, "step_latency_us": ms_per_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "pct_of_nominal_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
            "pct_of_measured_copy": 100.0 * value / world / peak,
            "config": {"workload": wl.name, "P": wl.P, "tensors": len(wl.shapes), "S": wl.S,
                       "grad_dtype": wl.grad_dtype, "bytes_per_step": step_b, "mode": args.mode,
                       "cache": ("L2 flushed between steps (working set %d MB)" % (working_set >> 20)) if flush is not None
                       else ("inputs larger than L2 (working set %d MB)" % (working_set >> 20)),
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "roofline": {"bound": "hbm", "kernel": "k_reduce (fused)" if fused else "k_reduce", "achieved": reduce_gbs, "peak": peak, "unit": "GB/s",
                         "frac": reduce_gbs / peak, "peak_kind": peak_kind + " copy bandwidth", "traffic": NCU_TRAFFIC_BYTES_FUSED.get(wl.name) if fused else NCU_TRAFFIC_BYTES.get(wl.name),
                         "bytes_per_launch": reduce_b, "us_per_launch": t_reduce * 1e3,
                         "timing": "events around each launch inside the step sequence (reduce, update, reduce, ...)",
                         "back_to_back_alone": iso,
                         "update_kernel": None if fused else
                         {"kernel": "k_update", "achieved": update_gbs, "frac": update_gbs / peak,
                          "bytes_per_launch": update_b, "us_per_launch": t_update * 1e3}},
            "warm_l2": None if warm_ms is None else {"ms_per_step": warm_ms, "value": step_b / (warm_ms * 1e-3) / 1e9,
                                                     "note": "no L2 flush, steps back to back"},
            "ceilings": ceilings, "clocks": clocks, "e2e": e2e, "cpu_baseline": cpu, "gpu_launches": launches,
        }
        print(json.dumps(line), flush=True)
    ada.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    args = parse_args()
    from paper_2007_05105_b200 import synthetic
    wl = synthetic.workload(args.workload)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
