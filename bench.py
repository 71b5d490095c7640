#!/usr/bin/env python
"""Benchmark of the isomorphic neighbourhood all-to-all on one B200 (or N independent
replicas, one per GPU).

A step is one `Iso_Start` of the whole schedule on the workload (default: the largest of the
configurations, all-to-all on a 256x256 torus, Moore neighbourhood of radius 2, 4 KB blocks:
6.4 GB per buffer).  The headline value is the effective bandwidth over the bytes the
message-combining schedule moves (read + written), device timed with CUDA events over
repeated runs of K steps; the same line carries the payload rate, the roofline fraction of
the dominant kernel with its DRAM traffic, the end-to-end rate with host buffers, the CPU
oracle timed on the host cores, and a table (`detail.configs`) with every configuration
under the combining, the direct and the hop-by-hop schedule, each checked against the
oracle on sampled ranks after it was timed.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--sweep paper]
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
FALLBACK_HBM_GBS = 6650.0
L2_FLUSH_BYTES = 512 << 20
L2_BYTES = 126 << 20
HEADLINE = "cfg3_m4096"
# ncu counters of the dominant kernels (DRAM bytes per launch), each stamped with a hash of
# the kernel sources it was taken on; an entry whose stamp is not the present sources' is
# ignored (traffic: null)
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.txt")
KERNEL_SOURCES = ("iso_kernels.cuh", "iso_api.cu", "iso_schedule.cpp", "iso_internal.h")


def sources_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_1606_07676_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, schedule: str):
    """DRAM bytes per step of `workload` under `schedule` from the tracked ncu summary, as
    {"bytes_per_step", "launches", "mode", "scaled_from"}, or None when there is no entry or
    the kernels have changed since it was captured."""
    try:
        lines = open(TRAFFIC_FILE).read().splitlines()
    except OSError:
        return None
    now = sources_hash()
    for ln in lines:
        f = ln.split()
        if len(f) < 7 or f[0].startswith("#"):
            continue
        if f[0] == workload and f[1] == schedule and f[6] == now:
            return {"bytes_per_step": float(f[3]), "launches": int(f[2]), "mode": f[4], "scaled_from": f[5]}
    return None


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


# ------------------------------------------------------------ what both arms agree on
def replica_count(w) -> int:
    """Independent instances of a workload that the timed steps rotate over, so that an
    instance's send and receive buffers have left the L2 before it comes round again."""
    from paper_1606_07676_b200 import workloads as wl
    lens, sd, rd, ss, rs = wl.layout(w)
    foot = max(1, w.P * (ss + rs))
    return max(1, min(16, -(-4 * L2_BYTES // foot)))


def config_dict(w, fusion: int, n_gpus: int) -> dict:
    """The `config` object of the JSON line; the same in both arms."""
    from paper_1606_07676_b200 import workloads as wl
    lens, sd, rd, ss, rs = wl.layout(w)
    foot = w.P * (ss + rs)
    n = replica_count(w)
    if n == 1:
        l2 = "inputs larger than L2: %.0f MB of send and receive buffers per step" % (foot / 1e6)
    else:
        l2 = ("inputs larger than L2: steps rotate over %d independent instances of the workload "
              "(%.1f MB of send and receive buffers each)" % (n, foot / 1e6))
    return {"workload": w.name, "collective": w.collective, "dims": list(w.dims), "s": w.s, "P": w.P,
            "block_bytes": w.block_bytes or None,
            "schedule": "combining (Section V), fusion level %d" % fusion,
            "parallelism": "replicas only" if n_gpus > 1 else "single GPU",
            "l2": l2,
            "bytes": "value = bytes the message-combining schedule reads + writes (2 x P x sum_i m_i x hops_i) / time, "
                     "the same byte count in both arms; payload = one read + one write of every delivered block"}


# ------------------------------------------------------------------------ the CPU oracle
class OracleSample:
    """A bounded sample of a workload for the CPU oracle: the receive buffers of the ranks of
    the first planes of dimension 0 (the whole workload when that is small).  The host send
    buffer is reserved in full, but only the planes those ranks read from are generated, so a
    6 GB workload costs a few hundred MB of host memory.  Only the CPU-baseline leg and the
    reference arm use this."""

    def __init__(self, w, max_out_bytes=192 << 20, whole_below=512 << 20):
        from paper_1606_07676_b200 import workloads as wl
        self.w = w
        self.lens, self.sd, self.rd, self.ss, self.rs = wl.layout(w)
        P, p0 = w.P, w.dims[0]
        plane = P // p0
        planes = max(1, min(p0, max_out_bytes // max(1, plane * self.rs)))
        if planes >= p0 or P * self.ss <= whole_below:
            self.r0, self.r1 = 0, P
            self.send = wl.send_buffer_np(w, self.ss)
            self.what = "the whole workload (%d processes x %d blocks)" % (P, w.s)
        else:
            self.r0, self.r1 = 0, planes * plane
            need = sorted({(x - int(c0)) % p0 for x in range(planes) for c0 in list(w.offsets[:, 0]) + [0]})
            self.send = np.empty((P, self.ss), dtype=np.uint8)
            for x in need:
                self.send[x * plane:(x + 1) * plane] = wl.payload_np(
                    w.kind, w.seed, 0, x * plane * self.ss, plane * self.ss).reshape(plane, self.ss)
            self.what = ("the receive buffers of %d of %d processes (planes 0..%d of dimension 0; %d source planes "
                         "generated)" % (self.r1, P, planes - 1, len(need)))
        self.ranks = self.r1 - self.r0
        self.bytes_min = 2 * self.ranks * int(self.lens.sum())

    def nominal_moved(self) -> int:
        """Bytes the message-combining schedule moves for the sampled ranks, by the paper's
        count (Section V: a block hops once per non-zero coordinate)."""
        from oracle import counters
        w = self.w
        if w.collective == "allgather":
            zeros = sum(1 for v in counters.residues(w.offsets, w.dims) if not any(v))
            parts = counters.allgather_direct_volume(w.offsets, w.d, w.dims) + zeros
            return 2 * self.ranks * w.block_bytes * parts
        hops = counters.direct_hops(w.offsets, w.d, w.dims)
        return 2 * self.ranks * sum(int(n) * max(h, 1) for n, h in zip(self.lens, hops))

    def run(self, lo=None, hi=None):
        import oracle
        w = self.w
        lo = self.r0 if lo is None else lo
        hi = self.r1 if hi is None else hi
        if w.collective == "alltoall":
            return oracle.alltoall(w.dims, w.offsets, w.block_bytes, self.send, lo, hi)
        if w.collective == "allgather":
            return oracle.allgather(w.dims, w.offsets, w.block_bytes, self.send, lo, hi)
        return oracle.alltoallv(w.dims, w.offsets, self.lens, self.sd, self.rd, self.ss, self.rs, self.send, lo, hi)


def cpu_baseline(w, seconds=10.0):
    """The oracle, as it stands, on this host: repeated passes over a bounded sample of the
    workload; GB/s over one read + one write of every delivered block."""
    sample = OracleSample(w)
    sample.run()
    times = []
    t_end = time.perf_counter() + seconds
    while len(times) < 3 or (time.perf_counter() < t_end and len(times) < 50):
        t0 = time.perf_counter()
        sample.run()
        times.append(time.perf_counter() - t0)
    dt = statistics.median(times)
    out = {"value": sample.bytes_min / dt / 1e9, "unit": "GB/s (payload: one read + one write of every delivered block)",
           "cores": 1, "kind": "oracle", "sample": "%s, median of %d passes" % (sample.what, len(times)),
           "ms_per_pass": dt * 1e3, "ms_whole_workload_extrapolated": dt * 1e3 * w.P / sample.ranks}
    # The same oracle over all host cores: the sampled ranks are cut into one contiguous range
    # per thread (the C call releases the interpreter lock).
    cores = len(os.sched_getaffinity(0))
    if cores > 1:
        from concurrent.futures import ThreadPoolExecutor
        cuts = [sample.r0 + sample.ranks * k // cores for k in range(cores + 1)]
        with ThreadPoolExecutor(cores) as pool:
            def whole():
                list(pool.map(lambda k: sample.run(cuts[k], cuts[k + 1]), range(cores)))
            whole()
            par = []
            t_end = time.perf_counter() + seconds / 2
            while len(par) < 3 or (time.perf_counter() < t_end and len(par) < 50):
                t0 = time.perf_counter()
                whole()
                par.append(time.perf_counter() - t0)
        pdt = statistics.median(par)
        out["all_cores"] = {"value": sample.bytes_min / pdt / 1e9, "unit": "GB/s", "cores": cores, "ms_per_pass": pdt * 1e3,
                            "sample": "same sample, one contiguous rank range per thread, median of %d passes" % len(par)}
    return out


def run_reference(args):
    """Times the CPU oracle, as it stands, on a bounded sample of the same workload, in the
    same unit and over the same byte count as the GPU arm."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_1606_07676_b200 import workloads as wl

    w = wl.config(args.workload)
    sample = OracleSample(w)
    for _ in range(max(1, args.warmup)):
        sample.run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        sample.run()
    dt = (time.perf_counter() - t0) / args.steps
    value = sample.nominal_moved() / dt / 1e9
    what = "%s per step, %d steps, one host thread" % (sample.what, args.steps)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": config_dict(w, args.fusion, args.gpus),
        "payload": {"gbs": sample.bytes_min / dt / 1e9},
        "ms_whole_workload_extrapolated": dt * 1e3 * w.P / sample.ranks,
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": what},
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
    pair around the whole run on the current stream (the stream the kernels are launched on)."""
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


def time_repeats(torch, fn, steps, warmup, dist=None, min_total_ms=500.0, max_repeats=400):
    """Runs of exactly `steps` back-to-back steps, each between a synchronisation (and a
    barrier over the ranks) and one CUDA event pair, repeated until at least `min_total_ms`
    of device time has been timed.  Returns the per-step times (ms) of the runs; with several
    ranks every entry is the slowest rank's."""
    first = max_over_ranks(dist, time_run(torch, fn, steps, warmup), "cuda")      # calibration, not reported
    repeats = int(max(1, min(max_repeats, -(-min_total_ms // max(first * steps, 1e-6)))))
    out = []
    for _ in range(repeats):
        if dist is not None:
            dist.barrier()
        out.append(max_over_ranks(dist, time_run(torch, fn, steps, 0), "cuda"))
    return out


def spread(times):
    return {"ms": statistics.median(times), "ms_min": min(times), "ms_max": max(times), "repeats": len(times)}


class Replicas:
    """Independent instances of one workload (different seeds, own buffers and requests),
    enough of them that a round-robin over the instances touches far more memory than the
    L2 holds before an instance comes round again."""

    def __init__(self, torch, iso, wl, name):
        first = Bound(torch, iso, wl, name)
        st = iso.Iso_request_get_stats(first.req)
        n = replica_count(first.w)
        self.items = [first] + [Bound(torch, iso, wl, name, seed=first.w.seed + 1000 * k) for k in range(1, n)]
        self.footprint = st["P"] * (st["send_stride"] + st["recv_stride"])
        self.iso, self.torch = iso, torch
        self.k = 0

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


def parity_check(torch, b, n_random=40):
    """The receive buffers of sampled ranks of instance `b`, as its last start left them,
    against the CPU oracle: the oracle names the source process of every block and the
    block's bytes are regenerated on the host.  Outside every timed region."""
    import oracle
    from paper_1606_07676_b200 import workloads as wl
    w = b.w
    torch.cuda.synchronize()
    P, last = w.P, w.dims[-1]
    plane = P // w.dims[0]
    rng = np.random.default_rng(2016)
    ranks = sorted({0, 1, last - 1, last % P, plane - 1, plane % P, P - plane, P - last, P - 1,
                    *rng.integers(0, P, n_random).tolist()})
    for r in ranks:
        got = b.recv[r * b.rs:(r + 1) * b.rs].cpu().numpy()
        for i in range(w.s):
            n = int(b.lens[i])
            q = oracle.source_rank(w.dims, r, w.offsets[i])
            want = wl.payload_np(w.kind, w.seed, 0, q * b.ss + int(b.sd[i]), n)
            if not np.array_equal(got[int(b.rd[i]):int(b.rd[i]) + n], want):
                return False
    return True


def end_to_end(torch, iso, b, moved, minimum, steps, dist, world):
    """The same step through Iso_Start_host: pinned host buffers in and out, copies inside the
    timed region; with several ranks the slowest one counts and the rate is the aggregate."""
    hs = torch.empty(b.w.P * b.ss, dtype=torch.uint8, pin_memory=True)
    hs.copy_(b.send)
    hr = torch.empty(b.w.P * b.rs, dtype=torch.uint8, pin_memory=True)
    stream = torch.cuda.current_stream()

    def start_host(k):
        iso.Iso_Start_host(b.req, hs, hr, stream)

    if dist is not None:
        dist.barrier()
    me = time_run(torch, start_host, steps, 2)
    me = max_over_ranks(dist, me, "cuda")
    # the result that travelled back, against the device's own receive buffers
    same = bool(torch.equal(hr, b.recv.cpu()))
    try:
        link = iso.Iso_request_get_host_transfer_ms(b.req)    # of the last step: first copy begins .. last copy ends
    except iso.IsoError:
        link = None
    del hs, hr
    return {"link_busy": link,"value": world * moved / (me * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": me, "steps": steps,
            "h2d_bytes_per_step": world * int(b.w.P * b.ss), "d2h_bytes_per_step": world * int(b.w.P * b.rs),
            "payload_gbs": world * minimum / (me * 1e-3) / 1e9,
            "link_gbs_per_direction": b.w.P * b.ss / (me * 1e-3) / 1e9,
            "host_result_equals_device_result": same}


SCHEDULES = (("combining", "ISO_ALG_COMBINING", 1), ("direct", "ISO_ALG_DIRECT", 1), ("torus", "ISO_ALG_TORUS", 1),
             ("combining_2", "ISO_ALG_COMBINING", 2))   # two dimensions per phase (from three dimensions on)


def skipped(key, w):
    """Schedules a workload does not have: Algorithm 1 is an all-to-all schedule; with two
    dimensions per phase a torus of fewer than three dimensions has the direct schedule."""
    return (key == "torus" and w.collective == "allgather") or (key == "combining_2" and len(w.dims) < 3)


def row(st, times, peak, ok):
    ms = statistics.median(times)
    moved, minimum = st["bytes_moved"], st["bytes_min"]
    return dict(spread(times), rounds=st["rounds"], launches=st["launches"], bytes_moved=moved, bytes_min=minimum,
                gbs_moved=moved / ms / 1e6, gbs_payload=minimum / ms / 1e6,
                frac_of_measured=moved / ms / 1e6 / peak, frac_of_nominal_8TBs=moved / ms / 1e6 / NOMINAL_HBM_GBS,
                payload_frac_of_measured=minimum / ms / 1e6 / peak, parity_checked=ok)


def steps_for(est_ms, floor_steps):
    """Steps per timed run of a table row: at least `floor_steps`, and enough that a run
    lasts about 20 ms."""
    return int(max(floor_steps, min(20000, -(-20.0 // max(est_ms, 1e-4)))))


def config_table(torch, iso, wl, peak, args, names, have=None):
    """Every configuration under the combining schedule (one launch per dimension), the
    one-pass direct schedule, the hop-by-hop schedule of Algorithm 1 and the combining schedule
    with two dimensions per phase, each timed as
    repeated runs until `--detail-ms` of device time and then checked against the oracle.
    `have` holds rows measured elsewhere (the headline workload)."""
    out = dict(have or {})
    for name in names:
        if name in out:
            continue
        reps = Replicas(torch, iso, wl, name)
        rows = {}
        for key, alg_name, fusion in SCHEDULES:
            if skipped(key, reps.items[0].w):
                rows[key] = None
                continue
            st = reps.set(getattr(iso, alg_name), fusion)
            est = time_run(torch, reps.start, 8, 3)
            k = steps_for(est, args.steps)
            times = time_repeats(torch, reps.start, k, 0, None, args.detail_ms)
            ok = all(parity_check(torch, b, 12) for b in reps.items[:2])
            rows[key] = dict(row(st, times, peak, ok), steps_per_run=k, replicas=len(reps.items),
                             execution=reps.execution())
        out[name] = rows
        reps.close()
        del reps
        torch.cuda.empty_cache()
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
    alg = {"combining": iso.ISO_ALG_COMBINING, "direct": iso.ISO_ALG_DIRECT, "torus": iso.ISO_ALG_TORUS}[args.alg]

    # ---- headline: message-combining schedule, one launch per dimension ----------------
    st = reps.set(alg, args.fusion)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local) if rank == 0 else None
    t0 = time.time()
    if args.headline_only:
        times = [max_over_ranks(dist, time_run(torch, reps.start, args.steps, args.warmup), "cuda")]
    else:
        times = time_repeats(torch, reps.start, args.steps, args.warmup, dist, args.min_ms)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    ms = statistics.median(times)
    moved, minimum = st["bytes_moved"], st["bytes_min"]
    value = world * moved / (ms * 1e-3) / 1e9
    per_gpu = moved / (ms * 1e-3) / 1e9
    launches = iso.Iso_request_get_stats(b.req)["launches"]
    # the output of the timed request, as the last timed step left it, against the oracle
    parity = all(parity_check(torch, x) for x in reps.items[:2]) if not args.headline_only else None

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "ms_per_step_min": min(times), "ms_per_step_max": max(times),
        "repeats": len(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": config_dict(b.w, args.fusion, world),
        "gpu_launches": launches * args.steps * len(times),
        "parity_checked": parity,
        "frac_of_nominal_8TBs": per_gpu / NOMINAL_HBM_GBS,
        "frac_of_measured": per_gpu / peak,
        # the same time over the minimum one-read-one-write payload instead of the bytes moved
        "payload": {"gbs": world * minimum / (ms * 1e-3) / 1e9,
                    "frac_of_measured": minimum / (ms * 1e-3) / 1e9 / peak,
                    "frac_of_nominal_8TBs": minimum / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
    }
    if args.alg != "combining":
        line["config"]["schedule"] = args.alg

    # ---- roofline of the dominant kernel ----------------------------------------------
    kernel = "iso_gather_bulk" if st["bulk_bytes"] * 2 > moved else "iso_gather_rows_wide"
    rec = recorded_traffic(args.workload, args.alg) if (
        args.fusion == 1 and not args.single_launch and args.bulk_threshold is None and not args.tune
        and args.slabs is None and args.pipeline is None) else None
    roofline = {
        "bound": "hbm", "kernel": kernel, "achieved": per_gpu, "peak": peak, "unit": "GB/s",
        "frac": per_gpu / peak, "peak_kind": "%s copy bandwidth" % peak_kind,
        "frac_note": "rate over the bytes the schedule reads + writes; intermediate blocks that one phase "
                     "writes and the next reads may be served by L2, dram_frac counts device-memory bytes only",
        "launches_per_step": launches, "bytes_per_launch": moved // max(1, launches),
        "avg_launch_ms": ms / max(1, launches),
        "traffic": None, "dram_frac": None,
        "note": "achieved = bytes read+written per launch / (step time / launches per step), "
                "timed live with CUDA events on the launching stream; launch gaps are inside the step time",
    }
    if args.traffic is not None:
        roofline["traffic"] = args.traffic
        roofline["dram_frac"] = args.traffic * launches / (ms * 1e-3) / 1e9 / peak
    elif rec is not None:
        roofline["traffic"] = rec["bytes_per_step"] / max(1, launches)
        roofline["dram_frac"] = rec["bytes_per_step"] / (ms * 1e-3) / 1e9 / peak
        roofline["traffic_note"] = ("dram__bytes_read.sum + dram__bytes_write.sum per launch (ncu, %s; %s), from "
                                    "profiles/dram_traffic.txt, taken on the present kernel sources"
                                    % (rec["mode"].replace("_", " "), rec["scaled_from"].replace("_", " ")))
    else:
        roofline["traffic_note"] = "no ncu capture of the present kernel sources for this workload and schedule"
    line["roofline"] = roofline

    detail = {"headline": {"fusion_level": args.fusion, "rounds": st["rounds"], "launches": launches,
                           "execution": dict(reps.execution(), tuned=bool(args.tune)),
                           "bytes_moved": moved, "bytes_min": minimum, "replicas": len(reps.items),
                           "footprint_bytes_per_replica": reps.footprint}}
    clocks = None
    full = rank == 0 and world == 1 and not args.headline_only
    if full:
        # the headline workload under the other schedules, while its buffers are there
        have = {args.workload: {"combining": dict(row(st, times, peak, parity), steps_per_run=args.steps,
                                                  replicas=len(reps.items), execution=reps.execution())}}
        if args.alg == "combining" and not args.no_detail:
            for key, alg_name, fusion in SCHEDULES[1:]:
                if skipped(key, b.w):
                    have[args.workload][key] = None
                    continue
                s2 = reps.set(getattr(iso, alg_name), fusion)
                est = time_run(torch, reps.start, 3, 2)
                k = steps_for(est, min(args.steps, 20))
                t2 = time_repeats(torch, reps.start, k, 0, None, args.detail_ms)
                have[args.workload][key] = dict(row(s2, t2, peak, all(parity_check(torch, x, 12) for x in reps.items[:2])),
                                                steps_per_run=k, replicas=len(reps.items), execution=reps.execution())
            st = reps.set(alg, args.fusion)
        # the same request one start at a time, the L2 emptied before each (outside the timed span)
        flush = Flush(torch)
        cold = time_steps(torch, reps.start, max(10, min(args.steps, 50)), 3, flush)
        detail["headline"]["cold"] = {
            "ms": tukey_median(cold), "ms_min": min(cold), "ms_max": max(cold), "steps": len(cold),
            "gbs_moved": moved / (tukey_median(cold) * 1e-3) / 1e9,
            "note": "one CUDA event pair per Iso_Start, %d MB written and read between starts to empty the L2; "
                    "median after removing outliers beyond 3 x IQR" % (L2_FLUSH_BYTES >> 20)}
        del flush
        try:
            line["e2e"] = end_to_end(torch, iso, b, moved, minimum, max(3, min(args.steps, 5 if moved > (1 << 30) else 20)), dist, world)
        except RuntimeError as err:      # page-locking two host copies of the buffers failed
            line["e2e"] = None
            detail["e2e_error"] = str(err)[:200]
        reps.close()
        del reps, b
        torch.cuda.empty_cache()
        if not args.no_detail:
            detail["launch_floor_us"] = {
                "dependent_launches": iso.Iso_measure_launch_floor(torch.cuda.current_stream(), 4000, True),
                "plain_launches": iso.Iso_measure_launch_floor(torch.cuda.current_stream(), 4000, False),
                "note": "device time per launch of an empty kernel, back to back on one stream: a phase of a "
                        "schedule cannot be shorter; cfg1 and cfg3_m4 are bound by it"}
            names = wl.CONFIG_NAMES if args.workload == HEADLINE else ()
            detail["configs"] = config_table(torch, iso, wl, peak, args, names, have)
            for name in ("cfg1", "cfg3_m4"):
                for key, r_ in (detail["configs"].get(name) or {}).items():
                    if r_:
                        r_["launch_floor_ms"] = r_["launches"] * detail["launch_floor_us"]["dependent_launches"] * 1e-3
            # DRAM traffic of the configurations whose intermediate blocks stay in L2
            for name in ("cfg2_alltoall", "cfg3_m64", "cfg3_m512"):
                rec2 = recorded_traffic(name, "combining")
                r_ = (detail["configs"].get(name) or {}).get("combining")
                if rec2 and r_:
                    r_["dram_bytes_per_step"] = rec2["bytes_per_step"]
                    r_["dram_frac_of_measured"] = rec2["bytes_per_step"] / r_["ms"] / 1e6 / peak
                    r_["l2_served_share"] = 1.0 - rec2["bytes_per_step"] / r_["bytes_moved"]
            # end to end on the small configuration too (54.5 MB each way: latency of the pipeline shows)
            if "cfg2_alltoall" in detail["configs"] and args.workload != "cfg2_alltoall":
                small = Bound(torch, iso, wl, "cfg2_alltoall")
                s2 = small.set(iso.ISO_ALG_COMBINING, 1)
                detail["configs"]["cfg2_alltoall"]["combining"]["e2e"] = end_to_end(
                    torch, iso, small, s2["bytes_moved"], s2["bytes_min"], 20, None, 1)
                small.close()
                del small
        else:
            detail["configs"] = have
        clocks = sampler.stop(t0, time.time())
        sampler = None
        if args.sweep:
            detail["sweep"] = sweep(torch, iso, wl, peak, args)
        line["cpu_baseline"] = cpu_baseline(wl.config(args.workload), args.cpu_seconds)
    else:
        if sampler is not None:
            clocks = sampler.stop(t0, time.time())
            sampler = None
        if world > 1:
            # every rank runs its replica through the host-buffer entry point; slowest rank counts
            try:
                line["e2e"] = end_to_end(torch, iso, b, moved, minimum, 3, dist, world)
            except RuntimeError as err:
                line["e2e"] = None
                detail["e2e_error"] = str(err)[:200]
        else:
            line["e2e"] = None
        reps.close()
        del reps, b
        torch.cuda.empty_cache()
    line["clocks"] = clocks
    line["detail"] = detail
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def sweep(torch, iso, wl, peak, args):
    """The paper's larger neighbourhoods: combining (one launch per dimension, and per round),
    direct, and the combining schedule after Iso_request_tune.  Same protocol as the table of
    configurations (rotation over instances, back to back)."""
    out = {}
    for name in wl.PAPER_NAMES:
        reps = Replicas(torch, iso, wl, name)
        rows = {}
        for key, alg, fusion in (("combining", iso.ISO_ALG_COMBINING, 1), ("combining_per_round", iso.ISO_ALG_COMBINING, 0),
                                 ("direct", iso.ISO_ALG_DIRECT, 1), ("combining_tuned", iso.ISO_ALG_COMBINING, 1)):
            # the last row: the same schedule after Iso_request_tune has timed slabs x chains x
            # graph replay (cold caches) and kept the fastest plan
            was = Bound.tune
            Bound.tune = was or key == "combining_tuned"
            st = reps.set(alg, fusion)
            Bound.tune = was
            est = time_run(torch, reps.start, 8, 3)
            k = steps_for(est, 20)
            times = time_repeats(torch, reps.start, k, 0, None, args.detail_ms)
            rows[key] = dict(row(st, times, peak, all(parity_check(torch, b, 8) for b in reps.items[:1])),
                             steps_per_run=k, replicas=len(reps.items), execution=reps.execution(),
                             bulk_bytes=st["bulk_bytes"])
        out[name] = rows
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
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--alg", default="combining", choices=["combining", "direct", "torus"],
                    help="schedule of the headline run (the table always has all three)")
    ap.add_argument("--fusion", type=int, default=1)
    ap.add_argument("--min-ms", type=float, default=500.0,
                    help="the K-step run is repeated until this much device time has been timed")
    ap.add_argument("--detail-ms", type=float, default=500.0, help="the same for every row of the table")
    ap.add_argument("--sweep", nargs="?", const="paper", default=None, choices=["paper"],
                    help="also time the paper's larger neighbourhoods")
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--headline-only", action="store_true",
                    help="one K-step run of the headline schedule and nothing else (short runs under a profiler)")
    ap.add_argument("--no-detail", action="store_true", help="skip the table of configurations")
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
    ap.add_argument("--sources-hash", action="store_true",
                    help="print the stamp of the present kernel sources (for profiles/dram_traffic.txt) and exit")
    args = ap.parse_args()
    if args.sources_hash:
        print(sources_hash())
        return 0
    if args.init_times:
        return run_init_times(args)
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
