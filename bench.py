#!/usr/bin/env python
"""Benchmark of the isomorphic neighbourhood all-to-all on one B200 (or N independent
replicas, one per GPU).

A step is one `Iso_Start` of the whole schedule on the workload (default: all-to-all on a
32x32x32 torus, Moore neighbourhood of radius 1, 64-byte fp32 blocks).  The headline value
is the effective bandwidth over the bytes the message-combining schedule actually moves
(read + written), device timed with CUDA events; the same line carries the payload rate,
the one-pass direct kernel for comparison, the roofline fraction, the end-to-end rate with
host buffers and the CPU oracle timed on the host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--sweep]
    python bench.py --impl reference ...      # times the CPU oracle instead
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "neighbor-alltoall effective GB/s (device-timed) and % of B200 HBM peak, combining vs direct"
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes (read + written) per launch of the dominant kernel, from the ncu capture
# summarised under profiles/ (iso_gather_rows_wide on cfg2_alltoall); only valid for that kernel build
# and workload, so it is reported for the default workload and schedule only.
TRAFFIC_BYTES_PER_LAUNCH = {"cfg2_alltoall": 44.56e6}
FALLBACK_HBM_GBS = 6650.0
L2_FLUSH_BYTES = 512 << 20


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while running."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        rows = [r for t, r in self.rows if t0 <= t <= t1 + 0.2] or [r for _, r in self.rows]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower() == "active":
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def tukey_median(xs):
    """Median after removing outliers beyond 3 x IQR (the paper's protocol, Section IV)."""
    xs = sorted(xs)
    if len(xs) < 4:
        return statistics.median(xs)
    q1, q3 = np.percentile(xs, [25, 75])
    lo, hi = q1 - 3 * (q3 - q1), q3 + 3 * (q3 - q1)
    kept = [x for x in xs if lo <= x <= hi]
    return statistics.median(kept or xs)


def init_distributed(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        import torch
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist_mod.init_process_group(backend=backend, rank=rank, world_size=world)
        dist = dist_mod
    return rank, world, local, dist


def max_over_ranks(dist, value: float, device) -> float:
    """The slowest rank's time: what a multi-rank run reports."""
    if dist is None:
        return value
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ------------------------------------------------------------------------ reference arm
def oracle_run(w, send):
    """One pass of the CPU oracle over the whole workload (only the CPU-baseline leg and the
    reference arm call this)."""
    import oracle
    from paper_1606_07676_b200 import workloads as wl
    lens, sd, rd, ss, rs = wl.layout(w)
    if w.collective == "alltoall":
        return oracle.alltoall(w.dims, w.offsets, w.block_bytes, send)
    if w.collective == "allgather":
        return oracle.allgather(w.dims, w.offsets, w.block_bytes, send)
    return oracle.alltoallv(w.dims, w.offsets, lens, sd, rd, ss, rs, send)


def run_reference(args):
    """Times the CPU oracle, as it stands, on the same workload and metric."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_1606_07676_b200 import workloads as wl

    w = wl.config(args.workload)
    lens, sd, rd, ss, rs = wl.layout(w)
    send = wl.send_buffer_np(w, ss)
    bytes_min = 2 * w.P * int(lens.sum())
    for _ in range(max(1, args.warmup)):
        oracle_run(w, send)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_run(w, send)
    dt = (time.perf_counter() - t0) / args.steps
    value = bytes_min / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": args.workload, "P": w.P, "s": w.s, "note": "CPU oracle (direct definition), "
                   "one host thread, whole workload per step; bytes = one read + one write of every block"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle",
                         "sample": "the whole workload, %d steps" % args.steps},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------ our arm
class Bound:
    """A workload bound to device buffers through the C-ABI binding."""

    def __init__(self, torch, iso, wl, name, seed=None):
        self.torch, self.iso = torch, iso
        self.w = wl.config(name) if seed is None else wl.config(name, seed)
        w = self.w
        self.lens, self.sd, self.rd, self.ss, self.rs = wl.layout(w)
        self.send = wl.payload_torch(w.kind, w.seed, 0, w.P * self.ss, "cuda")
        self.recv = torch.empty(w.P * self.rs, dtype=torch.uint8, device="cuda")
        self.comm = iso.Iso_neighborhood_create(w.dims, w.offsets)
        if w.collective == "alltoall":
            self.req = iso.Iso_neighbor_alltoall_init(self.send, w.block_bytes, 1, self.recv, w.block_bytes, 1, self.comm)
        elif w.collective == "allgather":
            self.req = iso.Iso_neighbor_allgather_init(self.send, w.block_bytes, 1, self.recv, w.block_bytes, 1, self.comm)
        else:
            self.req = iso.Iso_neighbor_alltoallv_init(self.send, self.lens, self.sd, 1, self.recv, self.lens, self.rd, 1, self.comm)

    bulk_threshold = None
    single_launch = False
    slabs = None      # None: the library's choice
    chains = None
    graph = None
    tune = False      # let the library time its execution variants and keep the fastest
    pipeline = None   # slabs of the pipelined one-launch execution (None: off)

    def set(self, alg, fusion, execution=None):
        """Selects the schedule; `execution` (slabs, chains, graph) copies another instance's
        tuned choice instead of tuning again."""
        iso = self.iso
        iso.Iso_request_set_single_launch(self.req, Bound.single_launch)
        iso.Iso_request_set_algorithm(self.req, alg, fusion)
        if Bound.bulk_threshold is not None:
            iso.Iso_request_set_bulk_threshold(self.req, Bound.bulk_threshold)
        ex = execution or {"slabs": Bound.slabs, "chains": Bound.chains, "graph": Bound.graph}
        iso.Iso_request_set_slabs(self.req, ex["slabs"] if ex["slabs"] is not None else 0)
        iso.Iso_request_set_chains(self.req, ex["chains"] if ex["chains"] is not None else 1)
        iso.Iso_request_set_graph(self.req, bool(ex["graph"]))
        iso.Iso_request_set_pipeline(self.req, Bound.pipeline or 0)
        stream = self.torch.cuda.current_stream()
        if Bound.tune and execution is None and not Bound.single_launch:
            iso.Iso_request_tune(self.req, stream, cold=True)   # the timed steps rotate over instances: cold caches
        iso.Iso_Start(self.req, stream)    # materialise outside the timed region
        iso.Iso_wait(self.req)
        return iso.Iso_request_get_stats(self.req)

    def execution(self):
        return self.iso.Iso_request_get_execution(self.req)

    def close(self):
        self.iso.Iso_request_free(self.req)
        self.iso.Iso_comm_free(self.comm)


class Flush:
    """Empties the L2 of anything useful: overwrites a buffer larger than the cache, then reads
    a second one so that the cache is left full of clean, unrelated lines (a cache full of
    dirty lines would charge their write-back to whatever runs next)."""

    def __init__(self, torch):
        self.a = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device="cuda")
        self.b = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device="cuda")
        self.sink = torch.zeros(1, dtype=torch.int64, device="cuda")

    def __call__(self):
        self.a.add_(1)
        self.sink += self.b.sum()


def time_steps(torch, fn, steps, warmup, flush):
    """Per-step device times (ms) of `fn(k)`: one CUDA event pair per step on the current
    stream, the L2 flushed between steps outside the timed spans."""
    for k in range(warmup):
        if flush is not None:
            flush()
        fn(k)
    torch.cuda.synchronize()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    for k in range(steps):
        if flush is not None:
            flush()
        starts[k].record()
        fn(k)
        ends[k].record()
    torch.cuda.synchronize()
    return [s.elapsed_time(e) for s, e in zip(starts, ends)]


def time_run(torch, fn, steps, warmup):
    """Device time (ms) per step of `steps` back-to-back calls fn(0..steps-1), one CUDA event
    pair around the whole run on the current stream."""
    for k in range(warmup):
        fn(k)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for k in range(steps):
        fn(k)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / steps


class Replicas:
    """Independent instances of one workload (different seeds, own buffers and requests),
    enough of them that a round-robin over the instances touches far more memory than the
    L2 holds before an instance comes round again."""

    def __init__(self, torch, iso, wl, name, min_bytes=4 * 126 * (1 << 20), max_replicas=16):
        first = Bound(torch, iso, wl, name)
        st = iso.Iso_request_get_stats(first.req)
        foot = st["P"] * (st["send_stride"] + st["recv_stride"] + st["inter_stride"])
        n = max(1, min(max_replicas, -(-min_bytes // max(1, foot))))
        self.items = [first] + [Bound(torch, iso, wl, name, seed=first.w.seed + 1000 * k) for k in range(1, n)]
        self.footprint = foot
        self.iso, self.torch = iso, torch

    def set(self, alg, fusion):
        st = self.items[0].set(alg, fusion)
        ex = self.items[0].execution() if Bound.tune else None
        for b in self.items[1:]:
            b.set(alg, fusion, ex)
        return st

    def execution(self):
        return self.items[0].execution()

    def start(self, k):
        b = self.items[k % len(self.items)]
        self.iso.Iso_Start(b.req, self.torch.cuda.current_stream())

    def close(self):
        for b in self.items:
            b.close()


def end_to_end(torch, iso, b, moved, minimum, args, dist, world):
    """The same step through Iso_Start_host: pinned host buffers in and out, copies inside the
    timed region; with several ranks the slowest one counts and the rate is the aggregate."""
    hs = torch.empty(b.w.P * b.ss, dtype=torch.uint8).pin_memory()
    hs.copy_(b.send.cpu())
    hr = torch.empty(b.w.P * b.rs, dtype=torch.uint8).pin_memory()
    stream = torch.cuda.current_stream()

    def start_host(k):
        iso.Iso_Start_host(b.req, hs, hr, stream)

    e2e_steps = max(3, min(args.steps, 20))
    if dist is not None:
        dist.barrier()
    me = time_run(torch, start_host, e2e_steps, 3)
    me = max_over_ranks(dist, me, "cuda")
    return {"value": world * moved / (me * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": me,
            "h2d_bytes_per_step": world * int(hs.numel()), "d2h_bytes_per_step": world * int(hr.numel()),
            "payload_gbs": world * minimum / (me * 1e-3) / 1e9}


def cpu_baseline(w, seconds=10.0):
    """The oracle, as it stands, on this host: repeated runs of the whole workload for a
    bounded time; returns GB/s over one read + one write of every delivered block."""
    from paper_1606_07676_b200 import workloads as wl
    lens, sd, rd, ss, rs = wl.layout(w)
    send = wl.send_buffer_np(w, ss)
    bytes_min = 2 * w.P * int(lens.sum())
    oracle_run(w, send)
    times = []
    t_end = time.perf_counter() + seconds
    while len(times) < 3 or (time.perf_counter() < t_end and len(times) < 50):
        t0 = time.perf_counter()
        oracle_run(w, send)
        times.append(time.perf_counter() - t0)
    dt = statistics.median(times)
    out = {"value": bytes_min / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
           "sample": "the whole workload (%d processes x %d blocks), median of %d runs" % (w.P, w.s, len(times)),
           "ms": dt * 1e3}
    # The same oracle over all host cores: the destination ranks are cut into one contiguous
    # range per thread (the C call releases the interpreter lock); regular collectives only.
    cores = len(os.sched_getaffinity(0))
    if cores > 1 and w.collective in ("alltoall", "allgather"):
        import oracle
        from concurrent.futures import ThreadPoolExecutor
        fn = oracle.alltoall if w.collective == "alltoall" else oracle.allgather
        cuts = [w.P * k // cores for k in range(cores + 1)]
        with ThreadPoolExecutor(cores) as pool:
            def whole():
                list(pool.map(lambda k: fn(w.dims, w.offsets, w.block_bytes, send, cuts[k], cuts[k + 1]),
                              range(cores)))
            whole()
            par = []
            t_end = time.perf_counter() + seconds / 2
            while len(par) < 3 or (time.perf_counter() < t_end and len(par) < 50):
                t0 = time.perf_counter()
                whole()
                par.append(time.perf_counter() - t0)
        pdt = statistics.median(par)
        out["all_cores"] = {"value": bytes_min / pdt / 1e9, "unit": "GB/s", "cores": cores, "ms": pdt * 1e3,
                            "sample": "same workload, one contiguous rank range per thread, median of %d runs"
                                      % len(par)}
    return out


def run_ours(args):
    import torch
    rank, world, local, dist = init_distributed(args.gpus)
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    from paper_1606_07676_b200 import binding as iso
    from paper_1606_07676_b200 import workloads as wl
    iso.load_library()

    peak, peak_kind = measured_peak()
    Bound.bulk_threshold = args.bulk_threshold
    Bound.single_launch = args.single_launch
    Bound.slabs, Bound.chains, Bound.graph, Bound.tune = args.slabs, args.chains, args.graph, args.tune
    Bound.pipeline = args.pipeline
    reps = Replicas(torch, iso, wl, args.workload)
    b = reps.items[0]

    # ---- headline: message-combining schedule, one launch per dimension ----------------
    st = reps.set(iso.ISO_ALG_COMBINING, args.fusion)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local) if rank == 0 else None
    t0 = time.time()
    ms = time_run(torch, reps.start, args.steps, args.warmup)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t1 = time.time()
    clocks = None
    if sampler is not None and (world > 1 or args.headline_only):
        clocks = sampler.stop(t0, t1)
        sampler = None
    ms = max_over_ranks(dist, ms, "cuda")
    moved, minimum = st["bytes_moved"], st["bytes_min"]
    value = world * moved / (ms * 1e-3) / 1e9
    per_gpu = moved / (ms * 1e-3) / 1e9

    detail = {"combining": {"fusion_level": args.fusion, "rounds": st["rounds"], "launches": st["launches"],
                            "execution": dict(reps.execution(), tuned=bool(args.tune)),
                            "bytes_moved": moved, "bytes_min": minimum, "ms": ms, "gbs_moved": per_gpu,
                            "gbs_payload": minimum / (ms * 1e-3) / 1e9, "replicas": len(reps.items),
                            "footprint_bytes_per_replica": reps.footprint}}

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": args.workload, "collective": b.w.collective, "dims": list(b.w.dims), "s": b.w.s,
                   "P": b.w.P, "block_bytes": b.w.block_bytes or None,
                   "schedule": "combining (Section V), fusion level %d" % args.fusion,
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": "inputs larger than L2: steps rotate over %d independent instances of the workload "
                         "(%.0f MB each, %.0f MB in all), timed back to back between one event pair"
                         % (len(reps.items), reps.footprint / 1e6, reps.footprint * len(reps.items) / 1e6),
                   "bytes": "value = bytes read + written by the schedule / device time"},
        "gpu_launches": iso.Iso_request_get_stats(b.req)["launches"] * args.steps,
        "frac_of_nominal_8TBs": per_gpu / NOMINAL_HBM_GBS,
        "frac_of_measured": per_gpu / peak,
        # the same time over the minimum one-read-one-write payload instead of the bytes moved
        "payload": {"gbs": world * minimum / (ms * 1e-3) / 1e9,
                    "frac_of_measured": minimum / (ms * 1e-3) / 1e9 / peak,
                    "frac_of_nominal_8TBs": minimum / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
    }

    if rank == 0 and world == 1 and args.headline_only:
        line["e2e"] = None
        line["roofline"] = {"bound": "hbm", "achieved": per_gpu, "peak": peak, "unit": "GB/s",
                            "frac": per_gpu / peak, "traffic": args.traffic, "peak_kind": "%s copy bandwidth" % peak_kind}
    elif rank == 0 and world == 1:
        flush = Flush(torch)
        one = lambda k: reps.start(0)
        # the same schedule on ONE instance: per-step events with an L2 flush in between
        # (includes the event and launch latency of a lone step), and back to back (warm)
        cold = time_steps(torch, one, min(args.steps, 50), 3, flush)
        detail["combining"]["ms_single_flushed_median"] = tukey_median(cold)
        detail["combining"]["ms_single_warm"] = time_run(torch, one, args.steps, 3)
        # per-round launches (the paper's schedule, one launch per round) and the direct kernel
        for key, alg, fusion in (("combining_per_round", iso.ISO_ALG_COMBINING, 0), ("direct", iso.ISO_ALG_DIRECT, 1)):
            s2 = reps.set(alg, fusion)
            m2 = time_run(torch, reps.start, args.steps, args.warmup)
            detail[key] = {"launches": s2["launches"], "bytes_moved": s2["bytes_moved"], "ms": m2,
                           "gbs_moved": s2["bytes_moved"] / (m2 * 1e-3) / 1e9,
                           "gbs_payload": s2["bytes_min"] / (m2 * 1e-3) / 1e9,
                           "frac_of_peak_moved": s2["bytes_moved"] / (m2 * 1e-3) / 1e9 / peak}
        st = reps.set(iso.ISO_ALG_COMBINING, args.fusion)
        # clocks were sampled over all device-timed legs above (the headline leg alone
        # lasts only steps x 40 microseconds)
        clocks = sampler.stop(t0, time.time())
        sampler = None

        line["e2e"] = end_to_end(torch, iso, b, moved, minimum, args, dist, world)

        # ---- roofline of the dominant kernel ------------------------------------------
        launches = max(1, st["launches"])
        kernel = "iso_gather_bulk" if st["bulk_bytes"] * 2 > moved else "iso_gather_rows_wide<16,12>"
        line["roofline"] = {
            "bound": "hbm", "kernel": kernel, "achieved": per_gpu, "peak": peak, "unit": "GB/s",
            "frac": per_gpu / peak, "peak_kind": "%s copy bandwidth" % peak_kind,
            "bytes_per_launch": moved // launches, "avg_launch_ms": ms / launches,
            "traffic": args.traffic if args.traffic is not None else (
                TRAFFIC_BYTES_PER_LAUNCH.get(args.workload) if args.fusion == 1 and not args.single_launch
                and args.bulk_threshold is None else None),
            "traffic_note": "DRAM read+write bytes per launch (ncu, caches flushed before each launch); "
                            "writes still held in L2 when the kernel ends are not in it",
            "note": "achieved = bytes read+written per launch / (step time / launches per step); "
                    "launch gaps are inside the step time",
        }
        line["cpu_baseline"] = cpu_baseline(b.w, args.cpu_seconds)
    elif world > 1:
        # every rank runs its replica through the host-buffer entry point; slowest rank counts
        e2e = end_to_end(torch, iso, b, moved, minimum, args, dist, world)
        line["e2e"] = e2e
        line["roofline"] = {"bound": "hbm", "achieved": per_gpu, "peak": peak, "unit": "GB/s",
                            "frac": per_gpu / peak, "traffic": None, "peak_kind": "%s copy bandwidth" % peak_kind}

    reps.close()
    del reps, b
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and args.sweep and not args.headline_only:
        detail["sweep"] = sweep(torch, iso, wl, peak, args)
    line["clocks"] = clocks
    line["detail"] = detail
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def sweep(torch, iso, wl, peak, args):
    """Every named workload, combining (one launch per dimension, and per round) and direct:
    the results table.  Same protocol as the headline (rotation over instances, back to back)."""
    out = {}
    for name in (wl.PAPER_NAMES if args.sweep == "paper" else wl.CONFIG_NAMES):
        reps = Replicas(torch, iso, wl, name)
        row = {}
        for key, alg, fusion in (("combining", iso.ISO_ALG_COMBINING, 1), ("combining_per_round", iso.ISO_ALG_COMBINING, 0),
                                 ("direct", iso.ISO_ALG_DIRECT, 1), ("combining_tuned", iso.ISO_ALG_COMBINING, 1)):
            # the last row: the same schedule after Iso_request_tune has timed slabs x chains x
            # graph replay (cold caches) and kept the fastest plan
            was = Bound.tune
            Bound.tune = was or key == "combining_tuned"
            st = reps.set(alg, fusion)
            Bound.tune = was
            steps = 40 if st["bytes_moved"] < (4 << 30) else 6
            ms = time_run(torch, reps.start, steps, 4)
            row[key] = {"rounds": st["rounds"], "launches": st["launches"], "execution": reps.execution(),
                        "bytes_moved": st["bytes_moved"],
                        "bytes_min": st["bytes_min"], "bulk_bytes": st["bulk_bytes"], "ms": ms,
                        "replicas": len(reps.items),
                        "gbs_moved": st["bytes_moved"] / ms / 1e6, "gbs_payload": st["bytes_min"] / ms / 1e6,
                        "frac_moved_of_peak": st["bytes_moved"] / ms / 1e6 / peak,
                        "frac_moved_of_8TBs": st["bytes_moved"] / ms / 1e6 / NOMINAL_HBM_GBS}
        out[name] = row
        reps.close()
        del reps
        torch.cuda.empty_cache()
    return out


def run_init_times(args):
    """Host-side set-up times on the grid of the paper's Table II (Moore neighbourhoods, d = 2..5,
    r = 1..3, 480 processes): neighbourhood creation and all-to-all init (schedule computation and
    lowering; no device is touched).  Median of 400 calls, milliseconds."""
    from paper_1606_07676_b200 import binding as iso
    from paper_1606_07676_b200 import workloads as wl
    dims_for = {2: (24, 20), 3: (10, 8, 6), 4: (6, 5, 4, 4), 5: (5, 4, 4, 3, 2)}
    out = {}
    for d, dims in dims_for.items():
        for r_ in (1, 2, 3):
            offs = wl.moore(d, r_)
            t_create, t_init = [], []
            for _ in range(args.steps if args.steps < 1000 else 400):
                t0 = time.perf_counter()
                comm = iso.Iso_neighborhood_create(dims, offs)
                t1 = time.perf_counter()
                req = iso.Iso_neighbor_alltoall_init(None, 1, 4, None, 1, 4, comm)
                t2 = time.perf_counter()
                iso.Iso_request_free(req)
                iso.Iso_comm_free(comm)
                t_create.append((t1 - t0) * 1e3)
                t_init.append((t2 - t1) * 1e3)
            out["d%d_r%d" % (d, r_)] = {"s": int(len(offs)), "create_ms": statistics.median(t_create),
                                        "alltoall_init_ms": statistics.median(t_init)}
    print(json.dumps({"init_times": out, "unit": "ms", "note": "host only, median of repeated calls"}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2_alltoall")
    ap.add_argument("--fusion", type=int, default=1)
    ap.add_argument("--sweep", nargs="?", const="configs", default=None, choices=["configs", "paper"],
                    help="also time every named workload (configs: the five configurations; "
                         "paper: the paper's larger neighbourhoods)")
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--headline-only", action="store_true",
                    help="time the headline schedule only (short runs under a profiler)")
    ap.add_argument("--single-launch", action="store_true",
                    help="run all phases in one cooperative launch instead of one launch per phase")
    ap.add_argument("--bulk-threshold", type=int, default=None,
                    help="override the size from which parts go to the bulk-copy kernel (0: never)")
    ap.add_argument("--slabs", type=int, default=None, help="slabs of dimension 0 (default: the library's choice)")
    ap.add_argument("--chains", type=int, default=None, help="slabs that run side by side")
    ap.add_argument("--pipeline", type=int, default=None,
                    help="pipelined one-launch execution over this many slabs (Iso_request_set_pipeline)")
    ap.add_argument("--graph", action="store_true", help="replay the launches from a captured graph")
    ap.add_argument("--tune", action="store_true",
                    help="call Iso_request_tune before timing: the library times its execution variants "
                         "(slabs, chains, graph replay) and keeps the fastest")
    ap.add_argument("--traffic", type=float, default=None,
                    help="DRAM bytes per launch of the dominant kernel from an ncu capture, if one is current")
    ap.add_argument("--init-times", action="store_true",
                    help="print host-side set-up times on the grid of the paper's Table II and exit")
    args = ap.parse_args()
    if args.init_times:
        return run_init_times(args)
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
