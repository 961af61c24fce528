#!/usr/bin/env python
"""Benchmark of the natural-compression hot path on B200.

Headline workload (c4, the largest configuration that fits one GPU): n = 16 workers, each an
fp32 gradient of d = 335,141,888 entries (Student-t(3) * 1e-4).  One step = one pass of the path
over that batch:
    nc_compress_batch   C_nat of the 16 vectors, one launch          (worker side)
    nc_aggregate        fixed-order fp32 sum of the 16 packed buffers (master side)
    nc_sum_fp32         the uncompressed 16-way sum of the same buffers (reference point)
`value` = n * d worker-entries per step / step time.  Inputs are 21.45 GB, far larger than the
126 MB L2, so nothing is flushed between steps.

The other four configurations run as legs of the same invocation (rank 0, N = 1) and are
reported per call under `kernels`:
    c1  d = 2^20, n = 4             nc_compress_batch, nc_aggregate (launch-bound, L2-resident)
    c2  ResNet-50 shape, n = 8      nc_compress_batch, nc_aggregate, nc_sum_fp32
    c3  same buffers, D_nat^{2,8}   nd_norms_batch, nd_round_batch, nd_compress_batch, nd_aggregate
    c5  d = 2^28, n = 8, keep 1 %   nd_sparse_compact_compress_batch, nd_sparse_compact_aggregate
Every leg is timed for at least --leg-seconds with an event after every call, while the SM clock
is sampled; each call is reported against the measured copy bandwidth and the nominal 8 TB/s.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (under torchrun) every rank runs an independent replica of the headline workload
("replicas only": the path has no exchange step on one node) and the value is the sum.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
import argparse
import importlib.util
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "compress + decode-accumulate throughput (worker-entries through the whole path)"
UNIT = "Gelem/s"
NOMINAL_HBM_GBPS = 8000.0
C4_N, C4_D = 16, 335_141_888
P_DITHER, S_DITHER = 2, 8
S_SPARSE = 4
SPARSE_CAP_FRACTION = 0.0125
CPU_SAMPLE_D = 1 << 22            # entries per worker of the oracle's bounded sample


def load_workloads():
    """The seeded input generators, loaded by file path: they hold none of the method's
    arithmetic, and the reference arm must be able to use them without the CUDA library."""
    spec = importlib.util.spec_from_file_location(
        "_natcomp_workloads", os.path.join(ROOT, "paper_1905_10988_b200", "workloads.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def ncu_traffic_per_entry(kernel):
    """DRAM bytes (read + written) per worker-entry that an ncu capture of `kernel` showed, from
    the table kept beside the profile summaries; None when the table has no such row."""
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")) as f:
            row = json.load(f)["kernels"][kernel]
        return float(row["dram_bytes_per_entry"]), row.get("capture")
    except Exception:
        return None, None


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while a timed region runs."""

    def __init__(self, index, period=0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples),
                "sm_mhz_min": min(self.samples) if self.samples else None}


def physical_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ---------------------------------------------------------------------------------------------
# headline workload


class HeadlineC4:
    """Device buffers of one replica of workload c4 and the C-ABI calls of a step."""

    GROUPS = ("nc_compress", "nc_aggregate", "sum_fp32")
    KERNEL_OF = {"nc_compress": "nc_compress_kernel", "nc_aggregate": "nc_aggregate_kernel",
                 "sum_fp32": "nc_sum_fp32_kernel"}
    LAUNCHES_PER_STEP = 3

    def __init__(self, nc, workloads, rank, device, n=C4_N, d=C4_D):
        from paper_1905_10988_b200 import timing
        self.nc, self.n, self.d = nc, n, d
        u8 = dict(dtype=torch.uint8, device=device)
        self.workers = timing.replica_worker_ids(rank, n)
        self.x = [workloads.config4_vector(w, d, device) for w in self.workers]
        self.exp = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
        self.sign = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
        self.out_nc = torch.empty(d, dtype=torch.float32, device=device)
        self.out_sum = torch.empty(d, dtype=torch.float32, device=device)
        self.outputs = (self.out_nc, self.out_sum)
        self.seed = 0

    def step(self, marks=None):
        nc, n, d = self.nc, self.n, self.d

        def mark(name):
            if marks is not None:
                ev = torch.cuda.Event(enable_timing=True)
                ev.record()
                marks.append((name, ev))

        mark("start")
        nc.nc_compress_batch(self.x, d, self.seed, self.workers, self.exp, self.sign, n)
        mark("nc_compress")
        nc.nc_aggregate(self.exp, self.sign, n, d, self.out_nc)
        mark("nc_aggregate")
        nc.nc_sum_fp32(self.x, n, d, self.out_sum)
        mark("sum_fp32")

    def algorithmic_bytes(self):
        n, d = self.n, self.d
        return {"nc_compress": n * d * (4 + 1.125), "nc_aggregate": d * (1.125 * n + 4),
                "sum_fp32": d * (4 * n + 4)}

    def units(self):
        return {"nc_compress": self.n * self.d, "nc_aggregate": self.d, "sum_fp32": self.d}


# ---------------------------------------------------------------------------------------------
# legs: the other configurations, one call after the other with an event after each


def time_sequence(calls, min_seconds, gpu_index, max_iters=20000):
    """Runs the sequence of (name, fn) repeatedly for at least `min_seconds` of device time, an
    event after every call, the SM clock sampled meanwhile.  Returns per call the list of
    device times in ms, and the clock record."""
    for _ in range(3):
        for _, fn in calls:
            fn()
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _, fn in calls:
        fn()
    e1.record()
    torch.cuda.synchronize()
    one = max(e0.elapsed_time(e1), 1e-3)
    iters = int(min(max_iters, max(20, min_seconds * 1e3 / one + 1)))
    sampler = ClockSampler(gpu_index)
    sampler.start()
    rows = []
    done = 0
    while done < iters:                       # in batches, so that events do not pile up
        batch = min(200, iters - done)
        evs = []
        for _ in range(batch):
            row = [torch.cuda.Event(enable_timing=True)]
            row[0].record()
            for _, fn in calls:
                fn()
                ev = torch.cuda.Event(enable_timing=True)
                ev.record()
                row.append(ev)
            evs.append(row)
        torch.cuda.synchronize()
        for row in evs:
            rows.append([a.elapsed_time(b) for a, b in zip(row[:-1], row[1:])])
        done += batch
    clocks = sampler.stop()
    per_call = {name: [r[i] for r in rows] for i, (name, _) in enumerate(calls)}
    return per_call, clocks, iters


def summarize_call(times_ms, nbytes, units, unit_name, peak, clocks, extra=None):
    mean = sum(times_ms) / len(times_ms)
    med = statistics.median(times_ms)
    out = {"ms": round(mean, 5), "ms_median": round(med, 5), "ms_best": round(min(times_ms), 5)}
    if nbytes:
        gbps = nbytes / mean / 1e6
        out.update({"algorithmic_GBps": round(gbps, 1),
                    "frac_of_measured_peak": round(gbps / peak, 4),
                    "frac_of_nominal_8TBps": round(gbps / NOMINAL_HBM_GBPS, 4)})
    if units:
        out[unit_name] = round(units / mean / 1e6, 1)
    if clocks.get("sm_mhz"):
        # time x clock: comparable across runs that settled at different SM clocks
        out["ms_x_sm_mhz"] = round(mean * clocks["sm_mhz"], 2)
    if extra:
        out.update(extra)
    return out


def leg_c1(nc, workloads, device, peak, seconds, gpu_index):
    n, d = 4, 1 << 20
    u8 = dict(dtype=torch.uint8, device=device)
    # two buffer sets used in turn; all of it (21 MB) stays L2-resident either way
    sets = []
    for k in range(2):
        xs = [workloads.config1_vector(w, d, device) for w in range(n)]
        es = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
        ss = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
        sets.append((xs, es, ss, torch.empty(d, dtype=torch.float32, device=device)))
    state = {"k": 0}
    workers = list(range(n))

    def compress():
        state["k"] ^= 1
        xs, es, ss, _ = sets[state["k"]]
        nc.nc_compress_batch(xs, d, 0, workers, es, ss, n)

    def aggregate():
        _, es, ss, out = sets[state["k"]]
        nc.nc_aggregate(es, ss, n, d, out)

    t, clocks, iters = time_sequence([("nc_compress_batch", compress), ("nc_aggregate", aggregate)],
                                     min(seconds, 0.3), gpu_index)
    note = {"note": "launch-bound and L2-resident (21 MB): the time is what counts, not the fraction"}
    # the same two calls replayed from a CUDA graph: what is left when the host's marshalling and
    # launch latency are out of the way
    graph = None
    try:
        gs = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(gs):
            with torch.cuda.graph(g, stream=gs, capture_error_mode="thread_local"):
                compress()
                aggregate()
        for _ in range(10):
            g.replay()
        torch.cuda.synchronize()
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        reps = 2000
        a.record()
        for _ in range(reps):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        graph = {"ms_per_compress_plus_aggregate": round(a.elapsed_time(b) / reps, 5), "replays": reps}
    except RuntimeError as exc:               # optional: report why it is missing
        graph = {"unavailable": str(exc).splitlines()[0][:160]}
    return {
        "workload": "c1: d=2^20, n=4, N(0,1e-3^2) + 1% zeros + 0.1% powers of two",
        "iterations": iters, "clocks": clocks, "graph_replay": graph,
        "nc_compress_batch": summarize_call(t["nc_compress_batch"], n * d * 5.125, n * d,
                                            "Gelem_per_s", peak, clocks, note),
        "nc_aggregate": summarize_call(t["nc_aggregate"], d * (1.125 * n + 4), d, "Gelem_per_s",
                                       peak, clocks, note),
    }


def leg_c2_c3(nc, workloads, device, peak, seconds, gpu_index):
    n = 8
    sizes = workloads.resnet50_tensor_sizes()
    off = workloads.offsets_from_sizes(sizes)
    d, B = off[-1], len(sizes)
    u8 = dict(dtype=torch.uint8, device=device)
    f32 = dict(dtype=torch.float32, device=device)
    xs = [workloads.config2_vector(w, device, sizes) for w in range(n)]
    workers = list(range(n))
    es = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
    ss = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
    out = torch.empty(d, **f32)
    out2 = torch.empty(d, **f32)
    t, clocks, iters = time_sequence([
        ("nc_compress_batch", lambda: nc.nc_compress_batch(xs, d, 0, workers, es, ss, n)),
        ("nc_aggregate", lambda: nc.nc_aggregate(es, ss, n, d, out)),
        ("nc_sum_fp32", lambda: nc.nc_sum_fp32(xs, n, d, out2)),
    ], seconds, gpu_index)
    c2 = {
        "workload": "c2: ResNet-50-shaped gradients, d=25,557,032 in 161 tensors, n=8",
        "iterations": iters, "clocks": clocks,
        "nc_compress_batch": summarize_call(t["nc_compress_batch"], n * d * 5.125, n * d,
                                            "Gelem_per_s", peak, clocks),
        "nc_aggregate": summarize_call(t["nc_aggregate"], d * (1.125 * n + 4), d, "Gelem_per_s",
                                       peak, clocks),
        "nc_sum_fp32": summarize_call(t["nc_sum_fp32"], d * (4 * n + 4), d, "Gelem_per_s", peak,
                                      clocks),
    }
    del es, ss
    # c3: D_nat^{2,8} on the same buffers; the norm pass and the rounding pass also on their own
    offd = torch.tensor(off, dtype=torch.int64, device=device)
    norms = [torch.empty(B, **f32) for _ in range(n)]
    levels = [torch.empty(nc.nd_level_bytes(d), **u8) for _ in range(n)]
    signs = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
    wsb = nc.nd_batch_workspace_bytes(d, B, n)
    ws = torch.empty(wsb, **u8)
    t, clocks, iters = time_sequence([
        ("nd_norms_batch", lambda: nc.nd_norms_batch(xs, d, offd, B, P_DITHER, norms, n, ws, wsb)),
        ("nd_round_batch", lambda: nc.nd_round_batch(xs, d, offd, B, S_DITHER, 0, workers, norms,
                                                     levels, signs, n)),
        ("nd_compress_batch", lambda: nc.nd_compress_batch(xs, d, offd, B, P_DITHER, S_DITHER, 0,
                                                           workers, norms, levels, signs, n, ws,
                                                           wsb)),
        ("nd_aggregate", lambda: nc.nd_aggregate(norms, levels, signs, n, d, offd, B, S_DITHER,
                                                 out)),
    ], seconds, gpu_index)
    two_reads = {"bytes_counted": "x once (4 + 0.625 B per entry); the call reads x twice from "
                                  "HBM where a bucket does not stay on chip"}
    c3 = {
        "workload": "c3: D_nat^{2,8} on the c2 buffers (161 buckets), n=8",
        "iterations": iters, "clocks": clocks,
        "nd_norms_batch": summarize_call(t["nd_norms_batch"], n * d * 4.0, n * d, "Gelem_per_s",
                                         peak, clocks),
        "nd_round_batch": summarize_call(t["nd_round_batch"], n * d * 4.625, n * d, "Gelem_per_s",
                                         peak, clocks),
        "nd_compress_batch": summarize_call(t["nd_compress_batch"], n * d * 4.625, n * d,
                                            "Gelem_per_s", peak, clocks, two_reads),
        "nd_aggregate": summarize_call(t["nd_aggregate"], d * (0.625 * n + 4), d, "Gelem_per_s",
                                       peak, clocks),
    }
    return c2, c3


def leg_c5(nc, workloads, device, peak, seconds, gpu_index, sm_count):
    n, d = 8, 1 << 28
    u8 = dict(dtype=torch.uint8, device=device)
    xs = [workloads.config5_vector(w, d, device) for w in range(n)]
    workers = list(range(n))
    cap = int(d * SPARSE_CAP_FRACTION)
    idx = [torch.empty(cap, dtype=torch.int32, device=device) for _ in range(n)]
    planes = [torch.empty(nc.nd_sparse_plane_bytes(cap, S_SPARSE), **u8) for _ in range(n)]
    count = [torch.zeros(1, dtype=torch.int32, device=device) for _ in range(n)]
    norm = [torch.zeros(1, dtype=torch.float32, device=device) for _ in range(n)]
    wsb = nc.nd_sparse_batch_workspace_bytes(d, cap, n)
    ws = torch.empty(wsb, **u8)
    out = torch.empty(d, dtype=torch.float32, device=device)
    t, clocks, iters = time_sequence([
        ("nd_sparse_compact_compress_batch", lambda: nc.nd_sparse_compact_compress_batch(
            xs, d, workloads.KEEP_1PCT_THRESHOLD, workloads.KEEP_1PCT_SCALE, nc.P_INF, S_SPARSE, 0,
            workers, idx, planes, count, norm, cap, n, ws, wsb)),
        ("nd_sparse_compact_aggregate", lambda: nc.nd_sparse_compact_aggregate(
            idx, planes, count, norm, n, S_SPARSE, d, cap, out)),
    ], seconds, gpu_index)
    listed = int(sum(int(c.cpu().numpy().view(np.uint32)[0]) for c in count))
    kept = 0.01 * d * n
    mhz = clocks.get("sm_mhz") or 1965
    # the selection draws one generator block (18 wide multiplies) per 4 coordinates; a
    # sub-partition issues one wide multiply per 4 cycles
    ceiling = sm_count * 4 * 32 * mhz * 1e6 / 4 / 4.5 / 1e9
    comp = summarize_call(t["nd_sparse_compact_compress_batch"],
                          kept * 32 + listed * 4.375, n * d, "Gcoord_per_s", peak, clocks,
                          {"bound": "alu", "generator_ceiling_Gcoord_per_s": round(ceiling, 1)})
    comp["frac_of_generator_ceiling"] = round(comp["Gcoord_per_s"] / ceiling, 4)
    return {
        "workload": "c5: d=2^28, n=8, N(0,1), keep 1% then D_nat^{inf,4}, index list + 3-bit codes",
        "iterations": iters, "clocks": clocks, "listed_entries": listed,
        "nd_sparse_compact_compress_batch": comp,
        "nd_sparse_compact_aggregate": summarize_call(
            t["nd_sparse_compact_aggregate"], 4.0 * d + listed * 4.375, d, "Gelem_per_s", peak,
            clocks),
    }


# ---------------------------------------------------------------------------------------------
# CPU oracle legs


def cpu_sample_inputs(workloads, d=CPU_SAMPLE_D, n=C4_N):
    return [workloads.config4_vector(w, d, "cpu").numpy() for w in range(n)]


def cpu_oracle_step(oracle, xs):
    """The headline step on the oracle, as it stands."""
    d = xs[0].size
    packed = [oracle.nc_compress(x, 0, w) for w, x in enumerate(xs)]
    oracle.nc_aggregate([p[0] for p in packed], [p[1] for p in packed], d)
    oracle.sum_fp32(xs)


def cpu_baseline(workloads):
    import oracle
    xs = cpu_sample_inputs(workloads)
    units = len(xs) * xs[0].size
    all_cores = oracle.max_threads()
    cpu_oracle_step(oracle, [x[:4096] for x in xs])          # first call builds / loads
    res = {}
    for label, threads in (("one_thread", 1), ("all_cores", all_cores)):
        oracle.set_threads(threads)
        t0 = time.perf_counter()
        cpu_oracle_step(oracle, xs)
        res[label] = {"value": units / (time.perf_counter() - t0) / 1e9, "cores": threads}
    oracle.set_threads(all_cores)
    sample = ("the headline step (C_nat of 16 workers, 16-way aggregate, 16-way fp32 sum) on the "
              "first %d entries' worth of each worker's c4 vector (%d worker-entries), OpenMP "
              "over entries" % (xs[0].size, units))
    return {"value": res["all_cores"]["value"], "unit": UNIT, "cores": all_cores, "kind": "oracle",
            "sample": sample, "one_thread": res["one_thread"]["value"]}


def run_reference(args, rank):
    if rank != 0:
        return
    import oracle
    workloads = load_workloads()
    xs = cpu_sample_inputs(workloads)
    units = len(xs) * xs[0].size
    cores = oracle.max_threads()
    cpu_oracle_step(oracle, [x[:4096] for x in xs])
    for _ in range(min(args.warmup, 3)):
        cpu_oracle_step(oracle, [x[:1 << 18] for x in xs])
    times = []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        cpu_oracle_step(oracle, xs)
        times.append(time.perf_counter() - t0)
    total = sum(times)
    value = units * len(times) / total / 1e9
    sample = ("every step = the headline step on the first %d entries of each of the 16 c4 "
              "vectors (%d worker-entries), all host cores" % (xs[0].size, units))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32+f32",
        "data": "synthetic",
        "config": {"workload": "c4: n=16 workers, d=335,141,888 fp32 entries each (bounded sample)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------


PROFILE_CASES = ("nc_compress", "nc_aggregate", "sum_fp32", "nd_norms", "nd_round", "nd_compress",
                 "nd_aggregate", "sparse_compress", "sparse_aggregate")


def run_profile_case(nc, workloads, args, device):
    """Profiling aid: one call alone on a small case (the ResNet-50 shape with --workers workers,
    larger than L2 from 2 workers on), timed with events; the command ncu captures."""
    n = args.workers
    sizes = workloads.resnet50_tensor_sizes()
    off = workloads.offsets_from_sizes(sizes)
    d, B = off[-1], len(sizes)
    u8 = dict(dtype=torch.uint8, device=device)
    f32 = dict(dtype=torch.float32, device=device)
    xs = [workloads.config2_vector(w, device, sizes) for w in range(n)]
    workers = list(range(n))
    es = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
    ss = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
    out = torch.empty(d, **f32)
    offd = torch.tensor(off, dtype=torch.int64, device=device)
    norms = [torch.empty(B, **f32) for _ in range(n)]
    levels = [torch.empty(nc.nd_level_bytes(d), **u8) for _ in range(n)]
    wsb = nc.nd_batch_workspace_bytes(d, B, n)
    ws = torch.empty(wsb, **u8)
    cap = int(d * SPARSE_CAP_FRACTION)
    idx = [torch.empty(cap, dtype=torch.int32, device=device) for _ in range(n)]
    planes = [torch.empty(nc.nd_sparse_plane_bytes(cap, S_SPARSE), **u8) for _ in range(n)]
    count = [torch.zeros(1, dtype=torch.int32, device=device) for _ in range(n)]
    norm = [torch.zeros(1, **f32) for _ in range(n)]
    swsb = nc.nd_sparse_batch_workspace_bytes(d, cap, n)
    sws = torch.empty(swsb, **u8)
    kept = 0.01 * d * n
    cases = {
        "nc_compress": (lambda: nc.nc_compress_batch(xs, d, 0, workers, es, ss, n), n * d * 5.125),
        "nc_aggregate": (lambda: nc.nc_aggregate(es, ss, n, d, out), d * (1.125 * n + 4)),
        "sum_fp32": (lambda: nc.nc_sum_fp32(xs, n, d, out), d * (4 * n + 4)),
        "nd_norms": (lambda: nc.nd_norms_batch(xs, d, offd, B, P_DITHER, norms, n, ws, wsb),
                     n * d * 4.0),
        "nd_round": (lambda: nc.nd_round_batch(xs, d, offd, B, S_DITHER, 0, workers, norms, levels,
                                               ss, n), n * d * 4.625),
        "nd_compress": (lambda: nc.nd_compress_batch(xs, d, offd, B, P_DITHER, S_DITHER, 0, workers,
                                                     norms, levels, ss, n, ws, wsb), n * d * 4.625),
        "nd_aggregate": (lambda: nc.nd_aggregate(norms, levels, ss, n, d, offd, B, S_DITHER, out),
                         d * (0.625 * n + 4)),
        "sparse_compress": (lambda: nc.nd_sparse_compact_compress_batch(
            xs, d, workloads.KEEP_1PCT_THRESHOLD, workloads.KEEP_1PCT_SCALE, nc.P_INF, S_SPARSE, 0,
            workers, idx, planes, count, norm, cap, n, sws, swsb), kept * 34.2),
        "sparse_aggregate": (lambda: nc.nd_sparse_compact_aggregate(
            idx, planes, count, norm, n, S_SPARSE, d, cap, out), 4.0 * d + kept * 2.2),
    }
    # what the master-side calls read must exist first
    for first in ("nc_compress", "nd_compress", "sparse_compress"):
        cases[first][0]()
    fn, nbytes = cases[args.profile]
    for _ in range(args.warmup):
        fn()
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    print(json.dumps({"profile": args.profile, "workers": n, "d": d, "ms": ms,
                      "algorithmic_GBps": nbytes / ms / 1e6}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-legs", action="store_true", help="skip the c1, c2, c3 and c5 legs")
    ap.add_argument("--leg-seconds", type=float, default=0.6,
                    help="device time spent on each leg (the SM clock is sampled every 20 ms)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--profile", default=None, choices=list(PROFILE_CASES),
                    help="profiling aid: time one call alone on the ResNet-50 shape")
    ap.add_argument("--workers", type=int, default=2,
                    help="number of simulated workers with --profile")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    import paper_1905_10988_b200 as nc
    from paper_1905_10988_b200 import timing, workloads

    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    gpu_index = physical_gpu_index(local_rank)
    sm_count = torch.cuda.get_device_properties(device).multi_processor_count
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    if args.profile:
        run_profile_case(nc, workloads, args, device)
        return

    peak, peak_kind = measured_hbm_peak()

    # ---- legs first (their buffers are freed before the headline buffers are made)
    legs = {}
    if rank == 0 and world == 1 and not args.no_legs:
        legs["c1"] = leg_c1(nc, workloads, device, peak, args.leg_seconds, gpu_index)
        torch.cuda.empty_cache()
        legs["c2"], legs["c3"] = leg_c2_c3(nc, workloads, device, peak, args.leg_seconds, gpu_index)
        torch.cuda.empty_cache()
        legs["c5"] = leg_c5(nc, workloads, device, peak, args.leg_seconds, gpu_index, sm_count)
        torch.cuda.empty_cache()

    # ---- headline: K timed steps of workload c4
    hp = HeadlineC4(nc, workloads, rank, device)
    for _ in range(args.warmup):
        hp.step()
    torch.cuda.synchronize()
    sampler = ClockSampler(gpu_index, period=0.005)    # >= 25 samples even for 20 steps
    marks_all = []
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    t_start = torch.cuda.Event(enable_timing=True)
    t_stop = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for _ in range(args.steps):
        marks = []
        hp.step(marks)       # an event after every call: 4 events per ~9 ms step
        marks_all.append(marks)
    t_stop.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    elapsed_ms = timing.max_over_ranks(t_start.elapsed_time(t_stop), dist, device)

    group_times = {g: [] for g in HeadlineC4.GROUPS}
    for marks in marks_all:
        for (_, a), (name, b) in zip(marks[:-1], marks[1:]):
            group_times[name].append(a.elapsed_time(b))
    units_per_step = hp.n * hp.d
    ms_per_step = elapsed_ms / args.steps
    value = world * units_per_step / (ms_per_step * 1e-3) / 1e9

    alg, units = hp.algorithmic_bytes(), hp.units()
    c4 = {"workload": "c4: n=16, d=335,141,888, 1e-4 * Student-t(3)", "iterations": args.steps,
          "clocks": clocks}
    for g, call in (("nc_compress", "nc_compress_batch"), ("nc_aggregate", "nc_aggregate"),
                    ("sum_fp32", "nc_sum_fp32")):
        c4[call] = summarize_call(group_times[g], alg[g], units[g], "Gelem_per_s", peak, clocks)
    legs["c4"] = c4

    # the dominant kernel of the timed step: the call group with the largest measured share
    mean_ms = {g: sum(v) / len(v) for g, v in group_times.items()}
    dom = max(mean_ms, key=mean_ms.get)
    dom_kernel = HeadlineC4.KERNEL_OF[dom]
    achieved = alg[dom] / (mean_ms[dom] * 1e-3) / 1e9
    per_entry, capture = ncu_traffic_per_entry(dom_kernel)
    roofline = {"bound": "hbm", "kernel": "%s (one launch per step, %d workers)" % (dom_kernel, hp.n),
                "share_of_step": round(mean_ms[dom] / ms_per_step, 4),
                "achieved": round(achieved, 1), "peak": peak, "peak_kind": peak_kind,
                "unit": "GB/s", "frac": round(achieved / peak, 4),
                "frac_of_nominal_8TBps": round(achieved / NOMINAL_HBM_GBPS, 4),
                "ms_mean": round(mean_ms[dom], 4),
                "ms_median": round(statistics.median(group_times[dom]), 4),
                "ms_best": round(min(group_times[dom]), 4),
                "algorithmic_bytes_per_launch": alg[dom],
                "traffic": (per_entry * units[dom]) if per_entry is not None else None,
                "traffic_source": capture}
    if dom == "nc_compress":
        # the second resource of this kernel: the generator needs 18 wide 32x32->64 multiplies
        # per 4 entries, and a sub-partition issues one per 4 cycles
        mhz = clocks.get("sm_mhz") or 1965
        gen_peak = sm_count * 4 * 32 * mhz * 1e6 / 4 / 4.5 / 1e9
        rate = units[dom] / mean_ms[dom] / 1e6
        roofline["generator_view"] = {"achieved_Gelem_per_s": round(rate, 1),
                                      "multiplier_pipe_peak_Gelem_per_s": round(gen_peak, 1),
                                      "at_sm_mhz": mhz, "frac": round(rate / gen_peak, 4)}

    # one roofline row per call of every leg
    rooflines = []
    for leg in ("c1", "c2", "c3", "c4", "c5"):
        for call, row in legs.get(leg, {}).items():
            if isinstance(row, dict) and "frac_of_measured_peak" in row:
                rooflines.append({"config": leg, "call": call, "ms": row["ms"],
                                  "achieved_GBps": row["algorithmic_GBps"],
                                  "frac": row["frac_of_measured_peak"],
                                  "frac_of_nominal_8TBps": row["frac_of_nominal_8TBps"],
                                  "bound": row.get("bound", "hbm")})

    # end to end: host buffers -> device -> whole step -> aggregates back on the host
    e2e = None
    if args.e2e_steps > 0:
        # several ranks share one host's memory: four distinct pinned vectors per rank then
        e2e = timing.e2e_host_steps(nc, hp, args.e2e_steps, 0 if world == 1 else 4)
        e2e_ms = timing.max_over_ranks(e2e["ms_per_step"], dist, device)
        e2e["value"] = world * units_per_step / (e2e_ms * 1e-3) / 1e9
        e2e["ms_per_step"] = e2e_ms
        e2e["unit"] = UNIT

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(workloads)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u32+f32", "data": "synthetic",
            "config": {"workload": "c4: C_nat at BERT-large scale, n=16 workers, d=335141888 fp32 "
                                   "entries each in 25 MiB buckets; nc_compress_batch + "
                                   "nc_aggregate + nc_sum_fp32 (uncompressed 16-way sum) per step",
                       "unit_definition": "worker-entries (n*d) through the step per second",
                       "l2": "inputs are 21.45 GB per replica, larger than the 126 MB L2; no flush",
                       "multi_gpu": "replicas only",
                       "legs": "c1, c2, c3 and c5 per call under `kernels`"},
            "clocks": clocks, "e2e": e2e,
            "gpu_launches": HeadlineC4.LAUNCHES_PER_STEP * args.steps,
            "roofline": roofline, "rooflines": rooflines, "cpu_baseline": cpu, "kernels": legs,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
