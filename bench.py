#!/usr/bin/env python
"""Benchmark of the natural-compression hot path on B200.

One step = one pass of the whole path over one batch of synthetic gradients, on the
ResNet-50-shaped workload (n = 8 workers, d = 25,557,032 fp32 entries in 161 buckets):
  C_nat  : nc_compress_batch (8 workers, one launch) + nc_aggregate
  D_nat  : nd_compress x 8 (p = 2, s = 8, per-bucket norms) + nd_aggregate
  sparse : nd_sparse_compact_compress_batch (keep 1 %, p = inf, s = 4, 3-bit codes)
           + nd_sparse_compact_aggregate (all workers, one launch)
  ref    : nc_sum_fp32 (uncompressed 8-way sum, the reference point)
The metric is worker-entries taken through the whole path per second (n * d per step).
Inputs (818 MB) are larger than the 126 MB L2, so no flush is needed between steps.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (under torchrun) every rank runs an independent replica of the same workload
("replicas only": the path has no exchange step on one node) and the value is the sum.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

N_WORKERS = 8
P_DITHER, S_DITHER = 2, 8
S_SPARSE = 4
SPARSE_CAP_FRACTION = 0.0125
METRIC = "hot-path throughput (C_nat + D_nat + sparse compress / decode-accumulate)"
UNIT = "Gelem/s"

# Per-launch DRAM traffic of the dominant kernel (nc_compress_kernel, 8-worker batch launch):
# dram__bytes_read.sum + dram__bytes_write.sum of the 2-worker capture summarised in
# profiles/nc_compress_c2_2workers.md (204.48 MB + 31.59 MB), scaled by 4 to the 8-worker launch
# (traffic is proportional to the number of workers).  The write part is below the 28.75 MB per
# worker that the kernel stores because some output is still dirty in L2 when the kernel ends.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 4 * (204_482_816 + 31_589_376)


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

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
                "samples": len(self.samples)}


def physical_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


DOMINANT_MARKS = ("start", "nc_compress")


class HotPath:
    """Device buffers for one replica of the workload and the sequence of C-ABI calls of a step."""

    GROUPS = ("nc_compress", "nc_aggregate", "nd_compress", "nd_aggregate", "sparse_compress",
              "sparse_accumulate", "sum_fp32")

    def __init__(self, nc, rank, device, n_workers=N_WORKERS, only=None):
        from paper_1905_10988_b200 import workloads
        self.nc = nc
        self.n = n_workers
        self.only = only
        sizes = workloads.resnet50_tensor_sizes()
        off = workloads.offsets_from_sizes(sizes)
        self.d, self.B = off[-1], len(sizes)
        n, d, B = self.n, self.d, self.B
        u8 = dict(dtype=torch.uint8, device=device)
        f32 = dict(dtype=torch.float32, device=device)
        from paper_1905_10988_b200 import timing
        self.workers = timing.replica_worker_ids(rank, n)
        self.x = [workloads.config2_vector(w, device, sizes) for w in self.workers]
        self.off = torch.tensor(off, dtype=torch.int64, device=device)
        self.exp = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
        self.sign = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
        self.out_nc = torch.empty(d, **f32)
        self.norms = [torch.empty(B, **f32) for _ in range(n)]
        self.level = [torch.empty(nc.nd_level_bytes(d), **u8) for _ in range(n)]
        self.sign_nd = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
        self.ws_bytes = nc.nd_batch_workspace_bytes(d, B, n)
        self.ws = torch.empty(self.ws_bytes, **u8)
        self.out_nd = torch.empty(d, **f32)
        self.cap = int(d * SPARSE_CAP_FRACTION)
        self.idx = [torch.empty(self.cap, dtype=torch.int32, device=device) for _ in range(n)]
        self.codes = [torch.empty(nc.nd_sparse_plane_bytes(self.cap, S_SPARSE), **u8)
                      for _ in range(n)]
        self.count = [torch.zeros(1, dtype=torch.int32, device=device) for _ in range(n)]
        self.snorm = [torch.zeros(1, **f32) for _ in range(n)]
        self.sws_bytes = nc.nd_sparse_batch_workspace_bytes(d, self.cap, n)
        self.sws = torch.empty(self.sws_bytes, **u8)
        self.out_sp = torch.empty(d, **f32)
        self.out_sum = torch.empty(d, **f32)
        # nc_compress_batch 1, nc_aggregate 1, nd_compress_batch 3, nd_aggregate 1,
        # nd_sparse_compact_compress_batch 6, nd_sparse_compact_aggregate 1, nc_sum_fp32 1
        self.launches_per_step = 1 + 1 + 3 + 1 + 6 + 1 + 1
        self.seed = 0

    def step(self, marks=None, mark_names=None):
        nc, n, d, B = self.nc, self.n, self.d, self.B
        from paper_1905_10988_b200 import workloads

        def mark(name):
            if marks is not None and (mark_names is None or name in mark_names):
                ev = torch.cuda.Event(enable_timing=True)
                ev.record()
                marks.append((name, ev))

        def want(name):
            return self.only is None or self.only == name

        mark("start")
        if want("nc_compress"):
            nc.nc_compress_batch(self.x, d, self.seed, self.workers, self.exp, self.sign, n)
        mark("nc_compress")
        if want("nc_aggregate"):
            nc.nc_aggregate(self.exp, self.sign, n, d, self.out_nc)
        mark("nc_aggregate")
        if want("nd_compress"):
            nc.nd_compress_batch(self.x, d, self.off, B, P_DITHER, S_DITHER, self.seed,
                                 self.workers, self.norms, self.level, self.sign_nd, n, self.ws,
                                 self.ws_bytes)
        mark("nd_compress")
        if want("nd_aggregate"):
            nc.nd_aggregate(self.norms, self.level, self.sign_nd, n, d, self.off, B, S_DITHER,
                            self.out_nd)
        mark("nd_aggregate")
        if want("sparse_compress"):
            nc.nd_sparse_compact_compress_batch(self.x, d, workloads.KEEP_1PCT_THRESHOLD,
                                                workloads.KEEP_1PCT_SCALE, nc.P_INF, S_SPARSE,
                                                self.seed, self.workers, self.idx, self.codes,
                                                self.count, self.snorm, self.cap, n, self.sws,
                                                self.sws_bytes)
        mark("sparse_compress")
        if want("sparse_accumulate"):
            nc.nd_sparse_compact_aggregate(self.idx, self.codes, self.count, self.snorm, n,
                                           S_SPARSE, d, self.cap, self.out_sp)
        mark("sparse_accumulate")
        if want("sum_fp32"):
            nc.nc_sum_fp32(self.x, n, d, self.out_sum)
        mark("sum_fp32")

    STREAM_GROUPS = (("nc_compress", "nc_aggregate"), ("nd_compress", "nd_aggregate"),
                     ("sparse_compress", "sparse_accumulate"), ("sum_fp32",))

    def step_on_streams(self, streams):
        """The same step with its four independent call chains on four streams (fork from the
        current stream, join back into it): the HBM-bound and the integer-bound kernels of
        different chains overlap at their tails."""
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        keep = self.only
        for stream, chain in zip(streams, self.STREAM_GROUPS):
            stream.wait_event(fork)
            with torch.cuda.stream(stream):
                for g in chain:
                    self.only = g
                    self.step()
            done = torch.cuda.Event()
            done.record(stream)
            main.wait_event(done)
        self.only = keep

    def algorithmic_bytes(self):
        """Compulsory HBM bytes per call group (per step)."""
        n, d = self.n, self.d
        kept = 0.01 * d
        return {
            "nc_compress": n * d * (4 + 1.125),
            "nc_aggregate": d * (1.125 * n + 4),
            "nd_compress": n * d * (4 + 4 + 0.625),        # x is read by the norm and rounding passes
            "nd_aggregate": d * (0.625 * n + 4),
            # kept entries are read as 32-byte sectors in three passes (norm, filter, emit);
            # about half of them survive the level-0 filter and are listed (4 B index + 3 bits)
            "sparse_compress": n * kept * (3 * 32 + 0.5 * 4.375),
            # dense output written once; the listed entries (about half of the kept) read once
            "sparse_accumulate": 4 * d + n * kept * 0.5 * 4.375,
            "sum_fp32": d * (4 * n + 4),
        }


def cpu_baseline_sample(steps=1):
    """Times the CPU oracle, as it stands, on a bounded sample of the same workload: the first
    tensors of the ResNet-50 layout (about 1.6 M entries) for all 8 workers, whole path."""
    import oracle
    from paper_1905_10988_b200 import workloads
    sizes_all = workloads.resnet50_tensor_sizes()
    sizes, tot = [], 0
    for s in sizes_all:
        if tot + s > 1_700_000:
            break
        sizes.append(s)
        tot += s
    off = workloads.offsets_from_sizes(sizes)
    d, n = off[-1], N_WORKERS
    xs = [workloads.config2_vector(w, "cpu", sizes).numpy() for w in range(n)]
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        packed = [oracle.nc_compress(xs[w], 0, w) for w in range(n)]
        oracle.nc_aggregate([p[0] for p in packed], [p[1] for p in packed], d)
        dn = [oracle.nd_compress(xs[w], off, P_DITHER, S_DITHER, 0, w) for w in range(n)]
        oracle.nd_aggregate([q[0] for q in dn], [q[1] for q in dn], [q[2] for q in dn], off,
                            S_DITHER, d)
        acc = np.zeros(d, np.float32)
        for w in range(n):
            idx, planes, count, nrm = oracle.sparse_compact_compress(
                xs[w], workloads.KEEP_1PCT_THRESHOLD, workloads.KEEP_1PCT_SCALE, oracle.P_INF,
                S_SPARSE, 0, w)
            oracle.sparse_compact_decode_accumulate(idx, planes, count, nrm, S_SPARSE, acc)
        oracle.sum_fp32(xs)
        times.append(time.perf_counter() - t0)
    sample = ("first %d tensors of the ResNet-50 layout (%d entries) x %d workers, whole path; "
              "C_nat and the sums use OpenMP over entries, D_nat and sparse legs are serial"
              % (len(sizes), d, n))
    return n * d, times, oracle.max_threads(), sample


def run_reference(args, rank):
    if rank != 0:
        return
    units, times, cores, sample = cpu_baseline_sample(steps=1)      # untimed warm-up of the build
    all_t = []
    for _ in range(max(1, args.warmup) - 1):
        cpu_baseline_sample(steps=1)
    for _ in range(args.steps):
        _, t, _, _ = cpu_baseline_sample(steps=1)
        all_t.extend(t)
    total = sum(all_t)
    value = units * len(all_t) / total / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(all_t),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32+f32",
        "data": "synthetic",
        "config": {"workload": "c2: ResNet-50-shaped gradients, n=8 workers (bounded sample)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--only", default=None, choices=list(HotPath.GROUPS),
                    help="profiling aid: time one call group alone")
    ap.add_argument("--workers", type=int, default=N_WORKERS,
                    help="number of simulated workers with --only")
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
    from paper_1905_10988_b200 import timing

    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    if args.only:
        # profiling aid: one call group alone, on a smaller case (still larger than L2)
        hp = HotPath(nc, rank, device, n_workers=args.workers)
        hp.step()                               # produces the planes the master-side calls read
        hp.only = args.only
        for _ in range(args.warmup):
            hp.step()
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            hp.step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.steps
        gb = hp.algorithmic_bytes()[args.only]
        print(json.dumps({"only": args.only, "workers": hp.n, "d": hp.d, "ms": ms,
                          "algorithmic_GBps": gb / ms / 1e6}))
        return

    hp = HotPath(nc, rank, device)
    for _ in range(args.warmup):
        hp.step()
    torch.cuda.synchronize()

    sampler = ClockSampler(physical_gpu_index(local_rank))
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
        hp.step(marks, DOMINANT_MARKS)       # events around the dominant kernel only
        marks_all.append(marks)
    t_stop.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    elapsed_ms = t_start.elapsed_time(t_stop)
    elapsed_ms = timing.max_over_ranks(elapsed_ms, dist, device)

    # the dominant kernel: average device time over the timed steps themselves; the other call
    # groups: a second pass with an event after every group (those events cost about 2 % of a
    # step, so they stay out of the timed region)
    group_ms = {g: 0.0 for g in HotPath.GROUPS}
    for marks in marks_all:
        group_ms["nc_compress"] += marks[0][1].elapsed_time(marks[1][1])
    group_ms["nc_compress"] /= args.steps
    k_groups = min(args.steps, 100)
    marks_all = []
    for _ in range(k_groups):
        marks = []
        hp.step(marks)
        marks_all.append(marks)
    torch.cuda.synchronize()
    for marks in marks_all:
        for (_, e0), (name, e1) in zip(marks[:-1], marks[1:]):
            if name != "nc_compress":
                group_ms[name] += e0.elapsed_time(e1) / k_groups

    units_per_step = hp.n * hp.d
    ms_per_step = elapsed_ms / args.steps
    value = world * units_per_step / (ms_per_step * 1e-3) / 1e9

    peak, peak_kind = measured_hbm_peak()
    alg = hp.algorithmic_bytes()
    kernels = {}
    for g in HotPath.GROUPS:
        gbs = alg[g] / (group_ms[g] * 1e-3) / 1e9 if group_ms[g] > 0 else None
        kernels[g] = {"ms": round(group_ms[g], 4), "algorithmic_GBps": round(gbs, 1),
                      "frac_of_measured_peak": round(gbs / peak, 4)}
    kernels["nc_compress"]["Gelem_per_s"] = round(units_per_step / group_ms["nc_compress"] / 1e6, 1)
    kernels["nc_aggregate"]["Gelem_per_s"] = round(hp.d / group_ms["nc_aggregate"] / 1e6, 1)
    kernels["nd_compress"]["Gelem_per_s"] = round(units_per_step / group_ms["nd_compress"] / 1e6, 1)
    kernels["nd_aggregate"]["Gelem_per_s"] = round(hp.d / group_ms["nd_aggregate"] / 1e6, 1)
    kernels["sparse_compress"]["Gcoord_per_s"] = round(
        units_per_step / group_ms["sparse_compress"] / 1e6, 1)
    kernels["sum_fp32"]["Gelem_per_s"] = round(hp.d / group_ms["sum_fp32"] / 1e6, 1)

    dom = "nc_compress"          # one launch per step: the batch kernel over 8 workers
    achieved = alg[dom] / (group_ms[dom] * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "nc_compress_kernel (8-worker batch launch)",
                "achieved": round(achieved, 1), "peak": peak, "peak_kind": peak_kind,
                "unit": "GB/s", "frac": round(achieved / peak, 4),
                "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH,
                "algorithmic_bytes_per_launch": alg[dom],
                # the second resource of this kernel: the generator needs 18 wide 32x32->64
                # multiplies per 4 entries, and a sub-partition issues one per 4 cycles:
                # 148 SMs x 4 x 32 lanes x f_SM / 4 / 4.5 entries per second at the sampled SM clock
                "generator_view": {
                    "achieved_Gelem_per_s": round(units_per_step / group_ms[dom] / 1e6, 1),
                    "multiplier_pipe_peak_Gelem_per_s": round(
                        148 * 4 * 32 * (clocks.get("sm_mhz") or 1965) * 1e6 / 4 / 4.5 / 1e9, 1)}}
    gv = roofline["generator_view"]
    gv["frac"] = round(gv["achieved_Gelem_per_s"] / gv["multiplier_pipe_peak_Gelem_per_s"], 4)

    # the same step with its independent call chains on four streams (reported beside `value`,
    # which stays the single-stream figure the per-group times belong to)
    streams = [torch.cuda.Stream() for _ in HotPath.STREAM_GROUPS]
    k_conc = min(args.steps, 100)
    for _ in range(3):
        hp.step_on_streams(streams)
    torch.cuda.synchronize()
    c0 = torch.cuda.Event(enable_timing=True)
    c1 = torch.cuda.Event(enable_timing=True)
    c0.record()
    for _ in range(k_conc):
        hp.step_on_streams(streams)
    c1.record()
    torch.cuda.synchronize()
    conc_ms = timing.max_over_ranks(c0.elapsed_time(c1) / k_conc, dist, device)
    concurrent = {"ms_per_step": conc_ms, "streams": len(streams), "steps": k_conc,
                  "value": world * units_per_step / (conc_ms * 1e-3) / 1e9, "unit": UNIT}

    # the same single-stream step replayed from a CUDA graph (no launch gaps); reported beside
    # `value` as well
    graph_replay = None
    try:
        graph_stream = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(graph_stream):
            # thread-local capture mode: a CUDA call from another thread of this process (a
            # communication library's watchdog, the clock sampler) must not break the capture
            with torch.cuda.graph(graph, stream=graph_stream, capture_error_mode="thread_local"):
                hp.step()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        g0 = torch.cuda.Event(enable_timing=True)
        g1 = torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(k_conc):
            graph.replay()
        g1.record()
        torch.cuda.synchronize()
        graph_ms = g0.elapsed_time(g1) / k_conc
    except RuntimeError as exc:               # the leg is optional: report why it is missing
        graph_ms = None
        graph_error = str(exc).splitlines()[0][:200]
    if dist is not None:
        # every rank reaches the reduction, also one whose capture failed
        worst = timing.max_over_ranks(graph_ms if graph_ms is not None else -1.0, dist, device)
        graph_ms = None if graph_ms is None else worst
    if graph_ms is not None and graph_ms > 0:
        graph_replay = {"ms_per_step": graph_ms, "steps": k_conc,
                        "value": world * units_per_step / (graph_ms * 1e-3) / 1e9, "unit": UNIT}
    elif graph_ms is None:
        graph_replay = {"unavailable": locals().get("graph_error", "capture failed on a rank")}

    # end to end: host buffers -> device -> whole path -> aggregates back on the host
    e2e = None
    if args.e2e_steps > 0:
        e2e = timing.e2e_host_steps(nc, hp, args.e2e_steps)
        e2e_ms = timing.max_over_ranks(e2e["ms_per_step"], dist, device)
        e2e["value"] = world * units_per_step / (e2e_ms * 1e-3) / 1e9
        e2e["ms_per_step"] = e2e_ms
        e2e["unit"] = UNIT

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        units, times, cores, sample = cpu_baseline_sample(steps=1)     # first call builds/loads
        units, times, cores, sample = cpu_baseline_sample(steps=2)
        cpu = {"value": units * len(times) / sum(times) / 1e9, "unit": UNIT, "cores": cores,
               "kind": "oracle", "sample": sample}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u32+f32", "data": "synthetic",
            "config": {"workload": "c2: ResNet-50-shaped gradients, n=8 workers, d=25557032 in "
                                   "161 buckets; C_nat + D_nat^{2,8} + sparse(1%) D_nat^{inf,4} "
                                   "+ fp32 8-way sum per step",
                       "unit_definition": "worker-entries (n*d) through the whole path per second",
                       "l2": "inputs are 818 MB per replica, larger than the 126 MB L2; no flush",
                       "multi_gpu": "replicas only"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": hp.launches_per_step * args.steps,
            "concurrent_streams": concurrent,
            "graph_replay": graph_replay,
            "roofline": roofline, "cpu_baseline": cpu, "kernels": kernels,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
