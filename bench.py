#!/usr/bin/env python
"""Benchmark of the AdaScale gain-ratio step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
                    [--mode two-kernel|fused|sharded]

A step is one whole iteration (reduce + scalar part + update) over one batch of synthetic
gradients.  The metric is the algorithmic bytes of a step, P * (S * b_g + 24), divided by its
duration.  Rank 0 prints one JSON line.

The headline workload is the largest one (decoder_24l).  W warm-up steps are followed by R
blocks of exactly K steps, each block between two CUDA events on the launching stream; R is
chosen so that about half a second of GPU work is timed whatever K is, and the line reports
the median block.  The same line carries, under "workloads", the step time, the rate and the
per-kernel figures of all five workloads measured in the same run.

With N > 1 every rank runs an independent replica on its own GPU (weak scaling; the value is
the sum over ranks at the slowest rank's pace), or, with --mode sharded, its slice of the
columns with one all-reduce of 16 bytes per step (strong scaling).  Started without a
launcher (no WORLD_SIZE in the environment), --gpus N starts its N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "adascale_step gradient GB/s and % of B200 HBM peak; step latency (us)"
HEADLINE = "decoder_24l"
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the reduce kernel, from the ncu
# captures summarised under profiles/ (None where no capture of the current kernel exists).
# decoder_24l is too large to capture; its figure is the capture of a narrower decoder of the
# same structure scaled by the number of parameters.
NCU_TRAFFIC_BYTES = {"decoder_24l": 4.578e9 * 354823168 / 68212736, "decoder_4l": 4.578e9, "resnet50": 850.8e6}
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 * 1024 * 1024
TIMED_SECONDS = 0.5      # GPU work timed per workload, whatever --steps says
MAX_REPEATS = 2000
ORACLE_SAMPLE_BYTES = 2 << 30   # gradient bytes of the oracle's timed sample, at most


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="two-kernel", choices=["two-kernel", "fused", "sharded"],
                    help="fused: lagged gain estimate, one kernel per step, P*(S*b_g+16) bytes; "
                         "sharded: columns split over the ranks, 16-byte all-reduce per step")
    ap.add_argument("--grads-ready", action="store_true",
                    help="ADASCALE_FLAG_GRADS_READY: rows may be streamed before the previous kernel has drained")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the four other workloads")
    return ap.parse_args(argv)


def grad_bytes(wl):
    return 2 if wl.grad_dtype == "bf16" else 4


def algorithmic_bytes(wl, fused=False):
    bg = grad_bytes(wl)
    if fused:  # S rows, w and v read, w and v written; the mean gradient never leaves the registers
        return wl.P * (wl.S * bg + 16), 0
    reduce_b = wl.P * (wl.S * bg + 4)   # S rows read, mean gradient written
    update_b = wl.P * 20                # gbar, w, v read; w, v written
    return reduce_b, update_b


def working_set(wl):
    return wl.P * (grad_bytes(wl) * wl.S + 12)


def config_of(wl, mode, world):
    """The same dictionary in both arms: what is measured, not how."""
    fused = mode == "fused"
    rb, ub = algorithmic_bytes(wl, fused)
    ws = working_set(wl)
    return {"workload": wl.name, "P": wl.P, "tensors": len(wl.shapes), "S": wl.S, "grad_dtype": wl.grad_dtype,
            "bytes_per_step": rb + ub, "mode": mode,
            "cache": ("L2 flushed between steps (working set %d MB)" % (ws >> 20)) if ws <= 2 * L2_BYTES
            else ("inputs larger than L2 (working set %d MB)" % (ws >> 20)),
            "parallelism": "single GPU" if world <= 1 else
            ("columns sharded over %d GPUs, 16-byte all-reduce per step" % world if mode == "sharded"
             else "replicas only")}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi sampling of SM clock and throttle reasons while a timed region runs (read only)."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index, period_ms=50):
        self.index = index
        self.period_ms = period_ms
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", str(self.period_ms)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            time.sleep(0.3)   # let the first sample arrive before the timed region starts
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.1)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        rows, reasons = [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                rows.append((float(parts[0]), float(parts[1]), float(parts[2])))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # "under load" = samples drawing more than half way between idle and the largest draw seen
        pmax, pmin = max(r[2] for r in rows), min(r[2] for r in rows)
        loaded = [r for r in rows if r[2] >= pmin + 0.5 * (pmax - pmin)] or rows
        return {"sm_mhz": statistics.median(r[0] for r in loaded), "sm_mhz_min": min(r[0] for r in loaded),
                "sm_max_mhz": max(r[1] for r in rows), "power_w_max": pmax, "samples": len(rows),
                "samples_under_load": len(loaded), "reasons": sorted(reasons)}


# ------------------------------------------------------------------ ranks


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(cmd, n, extra_env=None):
    """Starts `cmd` n times, one process per rank (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_* set), and
    waits for all of them.  Returns the largest exit code.  The children inherit stdout."""
    port = free_port()
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.update(extra_env or {})
        procs.append(subprocess.Popen(cmd, env=env))
    return max(p.wait() for p in procs)


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


# ------------------------------------------------------------------ the oracle as a CPU baseline


def as_oracle_array(t):
    import numpy as np
    import torch
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def oracle_inputs(wl, grads, w, v, fraction):
    """Host copies of columns [0, fraction * numel) of every tensor (all rows)."""
    import numpy as np
    cut = [max(1, int(n * fraction)) if n else 0 for n in wl.numels]
    rows = [[as_oracle_array(g[:c].detach().cpu().contiguous().view(-1)) for g, c in zip(row, cut)] for row in grads]
    w64 = [t[:c].detach().cpu().numpy().astype(np.float64) for t, c in zip(w, cut)]
    v64 = [t[:c].detach().cpu().numpy().astype(np.float64) for t, c in zip(v, cut)]
    return rows, w64, v64, sum(cut)


def time_oracle(wl, rows, w64, v64, columns, budget_s, max_steps):
    """Times the CPU oracle as it stands on the given columns."""
    import oracle
    cores = os.cpu_count() or 1
    orc = oracle.Oracle(wl.S, momentum=wl.momentum, weight_decay=wl.weight_decay, nthreads=cores)
    lr = oracle.make_lr(wl.lr.get("kind", "const"), eta0=wl.lr.get("eta0", 0.1), d=wl.lr.get("d", 1.0),
                        T_S1=wl.lr.get("T_S1", 1.0), milestones=wl.lr.get("milestones", ()))
    bytes_per_step = columns * (wl.S * grad_bytes(wl) + 24)
    times = []
    t_start = time.perf_counter()
    while len(times) < max_steps and (time.perf_counter() - t_start < budget_s or not times):
        t0 = time.perf_counter()
        orc.step(rows, w64, v64, lr)
        times.append(time.perf_counter() - t0)
    return times, bytes_per_step, cores


def oracle_baseline(wl, grads, w, v, total_budget_s, steps_wanted):
    """Calibrates on 1/64 of the columns, then times a slice that fits the budget."""
    rows, w64, v64, cols = oracle_inputs(wl, grads, w, v, 1.0 / 64)
    t_cal, _, _ = time_oracle(wl, rows, w64, v64, cols, 0.0, 1)
    t_cal, _, _ = time_oracle(wl, rows, w64, v64, cols, 0.0, 1)     # second call: threads are up
    est_full = t_cal[0] * 64
    fraction = 1.0
    grad_total = wl.P * wl.S * grad_bytes(wl)
    while fraction > 1.0 / 1024 and (est_full * fraction * max(steps_wanted, 3) > total_budget_s
                                     or grad_total * fraction > ORACLE_SAMPLE_BYTES):
        fraction /= 2
    if fraction != 1.0 / 64:
        rows, w64, v64, cols = oracle_inputs(wl, grads, w, v, fraction)
    return rows, w64, v64, cols, fraction


def run_reference(args, wl):
    """The CPU oracle on the host cores, rank 0 only."""
    from paper_2007_05105_b200 import synthetic
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = args.steps if args.steps is not None else 5
    warmup = args.warmup if args.warmup is not None else 1
    # generate only as many columns as the slice needs: the workload's first tensors' shapes, cut
    src_wl = wl
    src = synthetic.GradientSource(src_wl, device="cpu") if wl.P * wl.S * grad_bytes(wl) <= (4 << 30) else None
    if src is None:
        # too large to generate whole on the host: a workload of the same structure cut to 1/32 of every tensor
        src_wl = synthetic.workload(wl.name)
        src_wl.shapes = [(max(1, n // 32),) for n in wl.numels]
        src = synthetic.GradientSource(src_wl, device="cpu")
        scale_cols = 1.0 / 32
    else:
        scale_cols = 1.0
    grads = src.fill(0)
    wflat, vflat = src.init_params()
    w, v = src.views(wflat), src.views(vflat)
    rows, w64, v64, cols, fraction = oracle_baseline(src_wl, grads, w, v, 100.0, steps + warmup)
    time_oracle(src_wl, rows, w64, v64, cols, 1e9, warmup)
    times, bytes_per_step, cores = time_oracle(src_wl, rows, w64, v64, cols, 1e9, steps)
    total = sum(times)
    value = bytes_per_step * len(times) / total / 1e9
    frac_of_workload = cols / wl.P
    sample = ("the first %d of %d columns (%.4g of every tensor), all %d rows, %d steps of the fp64 oracle with "
              "OpenMP over columns" % (cols, wl.P, fraction * scale_cols, wl.S, len(times)))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": len(times), "warmup": warmup, "ms_per_step": 1e3 * total / len(times) / frac_of_workload,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(wl, args.mode, 1 if args.mode != "sharded" else args.gpus),
        "note": "ms_per_step is scaled from the sample to the whole workload",
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ GPU measurements


def _events(torch, n):
    return [torch.cuda.Event(enable_timing=True) for _ in range(n)]


class Job:
    """One workload resident on the device: gradients, parameters, context, pointer arrays."""

    def __init__(self, wl, dev, local, mode, grads_ready):
        import torch
        from paper_2007_05105_b200 import binding as B
        from paper_2007_05105_b200 import synthetic
        self.torch, self.B = torch, B
        self.wl, self.dev, self.mode = wl, dev, mode
        self.fused = mode == "fused"
        self.src = synthetic.GradientSource(wl, device=dev)
        self.grads = self.src.fill(0)
        wflat, vflat = self.src.init_params()
        self.w, self.v = self.src.views(wflat), self.src.views(vflat)
        flags = (B.FLAG_LAGGED | B.FLAG_FUSED) if self.fused else 0
        if grads_ready:
            flags |= B.FLAG_GRADS_READY
        self.ada = B.AdaScale(self.src.numels, wl.S, wl.grad_dtype, momentum=wl.momentum,
                              weight_decay=wl.weight_decay, device=local, flags=flags)
        self.sched = B.make_schedule(wl.lr.get("kind", "const"), eta0=wl.lr.get("eta0", 0.1), d=wl.lr.get("d", 1.0),
                                     T_S1=wl.lr.get("T_S1", 1.0), milestones=wl.lr.get("milestones", ()))
        self.gp, self.wp, self.vp = B.pointer_array(self.grads), B.pointer_array(self.w), B.pointer_array(self.v)
        self.stream = torch.cuda.current_stream(dev)
        self.sh = self.stream.cuda_stream  # passed explicitly: no per-call stream lookup on the host
        self.flush = None
        if working_set(wl) <= 2 * L2_BYTES:
            self.flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)
        self.sharded = None
        if mode == "sharded":
            from paper_2007_05105_b200 import sharded
            self.sums = torch.zeros(2, dtype=torch.float64, device=dev)
            self.sharded = sharded.ShardedAdaScale(self.ada, self.sums)

    def step(self):
        if self.sharded is not None:
            self.sharded.step(self.gp, self.wp, self.vp, self.sched, self.sh)
        else:
            self.ada.step(self.gp, self.wp, self.vp, self.sched, self.sh)

    def close(self):
        self.ada.close()


def time_blocks(job, steps, warmup):
    """`warmup` steps and one untimed block, then R blocks of exactly `steps` steps, R chosen from the
    untimed block so that about TIMED_SECONDS of GPU work are timed.  Returns (ms per step of every
    block, kernels launched inside the timed blocks).

    Large working sets: one event pair around each block of back-to-back steps.  Working sets
    within twice the L2 size: the L2 is flushed before every step and each step is timed on
    its own (the flush is outside the events)."""
    torch = job.torch

    def block():
        if job.flush is None:
            e0, e1 = _events(torch, 2)
            e0.record(job.stream)
            for _ in range(steps):
                job.step()
            e1.record(job.stream)
            return [(e0, e1)]
        evs = [_events(torch, 2) for _ in range(steps)]
        for a, b in evs:
            job.flush.zero_()
            a.record(job.stream)
            job.step()
            b.record(job.stream)
        return evs

    def block_ms(evs):
        return sum(a.elapsed_time(b) for a, b in evs) / steps

    for _ in range(warmup):
        if job.flush is not None:
            job.flush.zero_()
        job.step()
    cal = block()
    torch.cuda.synchronize(job.dev)
    repeats = int(-(-TIMED_SECONDS * 1e3 // max(block_ms(cal) * steps, 1e-6)))
    repeats = max(3, min(MAX_REPEATS, repeats))
    launches0 = job.ada.launch_count
    pending, per_block = [], []
    for i in range(repeats):
        pending.append(block())
        if len(pending) >= 64 or i == repeats - 1:   # bound the number of live events
            torch.cuda.synchronize(job.dev)
            per_block.extend(block_ms(evs) for evs in pending)
            pending = []
    return per_block, job.ada.launch_count - launches0


def time_kernels(job, n):
    """Per-kernel times: events between the two launches of a step, inside the step sequence."""
    torch, ada = job.torch, job.ada
    ev = [_events(torch, 3) for _ in range(n)]
    for a, b, c in ev:
        if job.flush is not None:
            job.flush.zero_()
        a.record(job.stream)
        if job.fused:
            ada.step(job.gp, job.wp, job.vp, job.sched, job.sh)
            b.record(job.stream)
        else:
            ada.reduce(job.gp, job.sched, job.sh)
            b.record(job.stream)
            ada.update(job.wp, job.vp, job.sh)
        c.record(job.stream)
    torch.cuda.synchronize(job.dev)
    t_reduce = statistics.median(a.elapsed_time(b) for a, b, c in ev)
    t_update = statistics.median(b.elapsed_time(c) for a, b, c in ev)
    iso = {}
    if not job.fused:  # the same kernels back to back on their own (no neighbour's dirty lines to write back)
        for name, call in (("reduce", lambda: ada.reduce(job.gp, job.sched, job.sh)),
                           ("update", lambda: ada.update(job.wp, job.vp, job.sh))):
            i0, i1 = _events(torch, 2)
            for _ in range(3):
                call()
            i0.record(job.stream)
            for _ in range(n):
                call()
            i1.record(job.stream)
            torch.cuda.synchronize(job.dev)
            iso[name + "_us"] = i0.elapsed_time(i1) / n * 1e3
    return t_reduce, t_update, iso


def probe_rate(torch, B, dev, local, kind, nbytes, reps=10):
    """The library's trivial streaming kernels over `nbytes` per array: kind 0 read, 1 copy, 2 a += b."""
    nbytes = max(1 << 20, (int(nbytes) // 16) * 16)
    a = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    b = a if kind == 0 else torch.empty(nbytes, dtype=torch.uint8, device=dev)
    a.zero_()
    b.zero_()
    moved = (1, 2, 3)[kind] * nbytes
    stream = torch.cuda.current_stream(dev)
    for _ in range(3):
        B.stream_probe(kind, a, b, nbytes, device=local)
    p0, p1 = _events(torch, 2)
    p0.record(stream)
    for _ in range(reps):
        B.stream_probe(kind, a, b, nbytes, device=local)
    p1.record(stream)
    torch.cuda.synchronize(dev)
    del a, b
    return moved * reps / (p0.elapsed_time(p1) * 1e-3) / 1e9


def choose_counts(args):
    steps = args.steps if args.steps is not None else 20
    warmup = max(3, args.warmup if args.warmup is not None else 5)
    return steps, warmup


def measure(args, wl, dev, local, world, rank, peak, headline):
    """Step and per-kernel timings of one workload.  The extras of the headline run are added by the caller."""
    import torch
    mode = args.mode if headline else "two-kernel"
    job = Job(wl, dev, local, mode, args.grads_ready)
    fused = job.fused
    reduce_b, update_b = algorithmic_bytes(wl, fused)
    step_b = reduce_b + update_b
    steps, warmup = choose_counts(args)

    sampler = ClockSampler(local)
    barrier(world)
    torch.cuda.synchronize(dev)
    if rank == 0:
        sampler.start()
    blocks, launches = time_blocks(job, steps, warmup)
    repeats = len(blocks)
    barrier(world)
    torch.cuda.synchronize(dev)
    clocks = sampler.stop() if rank == 0 else None
    local_ms = statistics.median(blocks)
    ms_per_step, value = whole_job_value(local_ms, step_b, world if mode != "sharded" else 1, dev)

    res = {"job": job, "steps": steps, "warmup": warmup, "repeats": repeats, "ms_per_step": ms_per_step,
           "value": value, "blocks_ms_per_step": {"min": min(blocks), "median": local_ms, "max": max(blocks)},
           "timed_gpu_seconds": sum(blocks) * steps * 1e-3, "clocks": clocks,
           "gpu_launches": launches, "gpu_launches_per_block": launches // repeats,
           "step_b": step_b, "reduce_b": reduce_b, "update_b": update_b}
    if mode != "sharded":
        t_reduce, t_update, iso = time_kernels(job, max(10, min(200, steps * min(repeats, 5))))
        res.update({"t_reduce_ms": t_reduce, "t_update_ms": t_update, "iso": iso})
        if job.flush is not None:  # small working sets: also the warm figure (no L2 flush, steps back to back)
            w0, w1 = _events(torch, 2)
            w0.record(job.stream)
            for _ in range(200):
                job.ada.step(job.gp, job.wp, job.vp, job.sched, job.sh)
            w1.record(job.stream)
            torch.cuda.synchronize(dev)
            res["warm_ms"] = w0.elapsed_time(w1) / 200
    return res


def kernel_report(res, peak, probes):
    """Per-kernel roofline figures.  `frac` divides algorithmic bytes per launch by the launch time and by the
    measured copy rate; the probe fractions use the library's own read / read-modify-write kernels at the
    same byte count in the same process.  A fraction above 1 means that part of the algorithmic bytes
    (the mean gradient) was served from L2 and never crossed the HBM interface."""
    out = {}
    gb = res["reduce_b"] / (res["t_reduce_ms"] * 1e-3) / 1e9
    out["k_reduce"] = {"achieved": gb, "frac": gb / peak, "bytes_per_launch": res["reduce_b"],
                       "us_per_launch": res["t_reduce_ms"] * 1e3,
                       "us_alone": res["iso"].get("reduce_us")}
    if probes and probes.get("read_gbs"):
        out["k_reduce"]["frac_of_read_probe"] = gb / probes["read_gbs"]
    if gb / peak > 1.0:
        out["k_reduce"]["note"] = ("above the copy rate: the kernel's traffic is 94-97 % reads, which HBM serves faster "
                                   "than a copy's 1:1 mix; frac_of_read_probe is the like-for-like ceiling")
    if res["update_b"]:
        ub = res["update_b"] / (res["t_update_ms"] * 1e-3) / 1e9
        out["k_update"] = {"achieved": ub, "frac": ub / peak, "bytes_per_launch": res["update_b"],
                           "us_per_launch": res["t_update_ms"] * 1e3, "us_alone": res["iso"].get("update_us")}
        if probes and probes.get("rmw_gbs"):
            out["k_update"]["frac_of_rmw_probe"] = ub / probes["rmw_gbs"]
        if ub / peak > 1.0:
            out["k_update"]["note"] = "above the copy rate: most of the mean gradient is read from L2"
    return out


def sharded_check(job, world, rank):
    """One step from a fresh state: the scalars every rank holds against the oracle's scalar part on the
    gathered per-rank sums, and this rank's mean gradient of its first columns against the oracle."""
    import numpy as np
    import torch
    import torch.distributed as dist
    import oracle
    B, wl = job.B, job.wl
    ada = B.AdaScale(job.src.numels, wl.S, wl.grad_dtype, momentum=wl.momentum, weight_decay=wl.weight_decay,
                     device=job.dev.index)
    sums = torch.zeros(2, dtype=torch.float64, device=job.dev)
    ada.reduce_sums(job.gp, sums, job.sh)
    mine = sums.clone()
    if world > 1:
        gathered = [torch.zeros_like(mine) for _ in range(world)]
        dist.all_gather(gathered, mine)
        dist.all_reduce(sums, op=dist.ReduceOp.SUM)
    else:
        gathered = [mine]
    w = [t.clone() for t in job.w]
    v = [t.clone() for t in job.v]
    ada.apply_sums(sums, job.sched, w, v, job.sh)
    st = ada.get_gain_tau(True)
    # this rank's columns: mean gradient of the first tensor (at most 2^20 columns) against the oracle
    n0 = min(job.src.numels[0], 1 << 20)
    rows = [as_oracle_array(row[0][:n0].detach().cpu().contiguous()) for row in job.grads]
    ogbar, _, _, _ = oracle.grad_stats(rows, True, os.cpu_count() or 1)
    gbar = ada.mean_grad_tensors()[0][:n0].cpu().numpy().astype(np.float64)
    scale = np.max(np.abs(np.stack([r.astype(np.float32) if r.dtype != np.uint16 else
                                    (r.astype(np.uint32) << 16).view(np.float32) for r in rows])), axis=0)
    ok_gbar = bool((np.abs(gbar - ogbar) <= 3e-7 * max(1.0, 0.15 * wl.S ** 0.5) * scale + 1e-45).all())
    D = sum(float(g[0]) for g in gathered)
    N = sum(float(g[1]) for g in gathered)
    orc = oracle.Oracle(wl.S, momentum=wl.momentum, weight_decay=wl.weight_decay)
    lr = oracle.make_lr(wl.lr.get("kind", "const"), eta0=wl.lr.get("eta0", 0.1), d=wl.lr.get("d", 1.0),
                        T_S1=wl.lr.get("T_S1", 1.0), milestones=wl.lr.get("milestones", ()))
    ost = orc.scalar(lr, D=D, N=N, Q=0.0)
    ok = ok_gbar and all(abs(getattr(st, k) - ost[k]) <= 1e-12 * abs(ost[k]) for k in ("r", "tau", "eta"))
    ada.close()
    flag = torch.tensor([1.0 if ok else 0.0], dtype=torch.float64, device=job.dev)
    if world > 1:
        dist.all_reduce(flag, op=dist.ReduceOp.MIN)
    return {"ok": bool(flag.item() == 1.0), "r": st.r, "tau": st.tau, "eta": st.eta, "oracle_r": ost["r"],
            "what": "one step from a fresh state: r, tau, eta of every rank against the oracle's scalar part on the "
                    "gathered per-rank sums (1e-12), mean gradient of each rank's first columns against the oracle"}


def run_ours(args):
    import torch
    from paper_2007_05105_b200 import binding as B
    from paper_2007_05105_b200 import synthetic

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    if args.mode == "sharded":
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", str(free_port()))
    world, rank, local = dist_setup(args.gpus)
    if local >= torch.cuda.device_count():
        raise SystemExit("rank %d needs GPU %d, this machine has %d" % (rank, local, torch.cuda.device_count()))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peak, peak_kind = measured_peak()
    fused = args.mode == "fused"

    wl_full = synthetic.workload(args.workload)
    wl = wl_full
    if args.mode == "sharded":
        import torch.distributed as dist
        from paper_2007_05105_b200 import sharded
        if not dist.is_initialized():   # one rank: the exchange still goes through NCCL
            dist.init_process_group(backend="nccl", rank=0, world_size=1)
        pieces = sharded.split_columns(wl_full.numels, rank, world)
        wl = synthetic.workload(args.workload, seed=wl_full.seed + 101 * rank)
        wl.shapes = [(n,) for _, _, n in pieces]

    res = measure(args, wl, dev, local, world, rank, peak, headline=True)
    job = res["job"]
    check = None
    if args.mode == "sharded":
        check = sharded_check(job, world, rank)
        # the whole job: all ranks' bytes at the slowest rank's pace
        total_b = sum(algorithmic_bytes(wl_full))
        res["ms_per_step"] = max_over_ranks(res["ms_per_step"], world, dev)
        res["value"] = total_b / (res["ms_per_step"] * 1e-3) / 1e9
        res["step_b"] = total_b

    # ---- end to end: gradients start in pinned host memory, statistics come back
    e2e = None
    if not args.no_e2e and args.mode != "sharded":
        h2d = wl.P * wl.S * grad_bytes(wl)
        host_rows = [torch.empty(job.src.flat_len, dtype=job.src.rows[0].dtype).pin_memory() for _ in range(wl.S)]
        for hr, dr in zip(host_rows, job.src.rows):
            hr.copy_(dr)
        hp = B.pointer_array([job.src.views(hr) for hr in host_rows])
        esteps = max(3, min(res["steps"], int(10e9 / max(h2d, 1))))
        for _ in range(2):
            job.ada.step_host(hp, job.wp, job.vp, job.sched)
        barrier(world)
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        for _ in range(esteps):
            job.ada.step_host(hp, job.wp, job.vp, job.sched)   # returns after the device finished and the stats arrived
        torch.cuda.synchronize(dev)
        e_ms = (time.perf_counter() - t0) * 1e3 / esteps
        e_ms = max_over_ranks(e_ms, world, dev)
        e2e = {"value": world * res["step_b"] / (e_ms * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": 112, "ms_per_step": e_ms, "steps": esteps,
               "api": "adascale_step_host (pinned host gradients -> device staging -> step -> stats to host)"}
        del host_rows, hp

    # ---- the CPU oracle on this machine's cores, rank 0, one GPU only
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and args.mode != "sharded":
        rows, w64, v64, cols, fraction = oracle_baseline(wl, job.grads, job.w, job.v, 12.0, 3)
        times, bps, cores = time_oracle(wl, rows, w64, v64, cols, 12.0, 50)
        cpu = {"value": bps * len(times) / sum(times) / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
               "sample": "columns [0, %g * numel) of every tensor (%d columns), all %d rows, %d steps of the fp64 "
                         "oracle with OpenMP over columns" % (fraction, cols, wl.S, len(times)),
               "s_per_step_scaled": sum(times) / len(times) * wl.P / cols}
        del rows, w64, v64

    job.close()
    del job
    res.pop("job")
    torch.cuda.empty_cache()

    # ---- bandwidth ceilings of this GPU: the library's own trivial kernels at the kernels' byte counts
    probes = None
    if rank == 0 and args.mode != "sharded":
        probes = {"read_gbs": probe_rate(torch, B, dev, local, 0, res["reduce_b"]),
                  "read_bytes": res["reduce_b"]}
        if res["update_b"]:
            probes["rmw_gbs"] = probe_rate(torch, B, dev, local, 2, res["update_b"] / 3)
            probes["copy_gbs"] = probe_rate(torch, B, dev, local, 1, res["update_b"] / 2)
            probes["rmw_copy_bytes"] = res["update_b"]
        probes["note"] = ("the library's trivial streaming kernels in this process: read = one pass over as many bytes "
                          "as a reduce launch moves; rmw (a[i] += b[i]: two reads, one write) and copy move as many "
                          "bytes as an update launch")

    # ---- all five workloads in the same run (rank 0 of a single-GPU run)
    workloads = None
    if world == 1 and not args.no_sweep and args.mode == "two-kernel":
        workloads = {}
        sweep_sampler = ClockSampler(local, period_ms=100)
        sweep_sampler.start()
        for name in synthetic.WORKLOAD_NAMES:
            if name == wl.name:
                r = res
                pr = probes
            else:
                r = measure(args, synthetic.workload(name), dev, local, 1, 0, peak, headline=False)
                r.pop("job").close()
                torch.cuda.empty_cache()
                pr = {"read_gbs": probe_rate(torch, B, dev, local, 0, r["reduce_b"], reps=20),
                      "rmw_gbs": probe_rate(torch, B, dev, local, 2, r["update_b"] / 3, reps=20)}
            entry = {"step_us": r["ms_per_step"] * 1e3, "gbs": r["value"],
                     "pct_of_measured_copy": 100.0 * r["value"] / peak,
                     "pct_of_nominal_8TBs": 100.0 * r["value"] / NOMINAL_HBM_GBS,
                     "bytes_per_step": r["step_b"], "steps": r["steps"], "repeats": r["repeats"],
                     "timed_gpu_seconds": r["timed_gpu_seconds"],
                     "kernels": kernel_report(r, peak, pr),
                     "probes_at_kernel_bytes": {k: v for k, v in (pr or {}).items() if k.endswith("_gbs")},
                     "sm_mhz": (r["clocks"] or {}).get("sm_mhz"), "reasons": (r["clocks"] or {}).get("reasons")}
            if "warm_ms" in r:
                entry["warm_l2_step_us"] = r["warm_ms"] * 1e3
                entry["cache"] = "L2 flushed before every step; warm_l2_step_us: back to back without the flush"
            workloads[name] = entry
        res["sweep_clocks"] = sweep_sampler.stop()

    if rank == 0:
        kernels = kernel_report(res, peak, probes) if args.mode != "sharded" else {}
        kr = kernels.get("k_reduce", {})
        line = {
            "metric": METRIC, "value": res["value"], "unit": "GB/s", "n_gpus": world, "steps": res["steps"],
            "warmup": res["warmup"], "repeats": res["repeats"], "ms_per_step": res["ms_per_step"],
            "step_latency_us": res["ms_per_step"] * 1e3, "higher_is_better": True,
            "scaling": "strong" if args.mode == "sharded" else "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "pct_of_nominal_8TBs": 100.0 * res["value"] / world / NOMINAL_HBM_GBS,
            "pct_of_measured_copy": 100.0 * res["value"] / world / peak,
            "timing": "median of %d blocks of %d back-to-back steps, CUDA events on the launching stream; "
                      "%.2f s of GPU work timed" % (res["repeats"], res["steps"], res["timed_gpu_seconds"]),
            "blocks_ms_per_step": res["blocks_ms_per_step"],
            "config": dict(config_of(wl_full, args.mode, world)),
            "grads_ready_flag": bool(args.grads_ready),
            "roofline": None if not kr else {
                "bound": "hbm", "kernel": "k_reduce (fused)" if fused else "k_reduce", "achieved": kr["achieved"],
                "peak": peak, "unit": "GB/s", "frac": kr["frac"], "peak_kind": peak_kind + " copy bandwidth",
                "traffic": NCU_TRAFFIC_BYTES.get(wl.name + ("_fused" if fused else "")),
                "bytes_per_launch": kr["bytes_per_launch"], "us_per_launch": kr["us_per_launch"],
                "timing": "median over events around each launch inside the step sequence (reduce, update, reduce, ...)",
                "frac_of_read_probe": kr.get("frac_of_read_probe"), "us_alone": kr.get("us_alone"), "note": kr.get("note"),
                "update_kernel": kernels.get("k_update")},
            "ceilings": probes, "workloads": workloads, "clocks": res["clocks"],
            "sweep_clocks": res.get("sweep_clocks"), "e2e": e2e, "cpu_baseline": cpu,
            "gpu_launches": res["gpu_launches"], "gpu_launches_per_block": res["gpu_launches_per_block"],
        }
        if check is not None:
            line["sharded_check"] = check
        print(json.dumps(line), flush=True)
    if torch.distributed.is_available() and torch.distributed.is_initialized():
        torch.distributed.destroy_process_group()
    if check is not None and not check["ok"]:
        raise SystemExit("sharded step disagrees with the oracle")


def main():
    args = parse_args()
    from paper_2007_05105_b200 import synthetic
    if args.impl == "reference":
        run_reference(args, synthetic.workload(args.workload))
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher: start the ranks here, one process per GPU; rank 0 prints the line
        sys.exit(spawn_ranks([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], args.gpus))
    run_ours(args)


if __name__ == "__main__":
    main()
