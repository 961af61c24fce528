"""Per-call timings on the five benchmark workloads (one GPU).

    python -m paper_1905_10988_b200.config_bench --config c4 [--iters 20]

For every C-ABI call the workload uses it prints one JSON line with the device time (CUDA
events, median and best over the iterations, after warm-up), the rate in Gelem/s and the
algorithmic HBM bytes per second.  bench.py at the repository root is the whole-path step
benchmark on c2; this tool covers the other shapes: c1 (small, launch-bound), c3 (D_nat on the
c2 buffers), c4 (n = 16, d = 335 M, beside the uncompressed 16-way sum) and c5 (sparse, d = 2^28).
"""
from __future__ import annotations

import argparse
import json
import statistics

import torch

from . import binding as nc
from . import workloads

HBM_PEAK_FALLBACK = 6650.0


REPS = 1     # calls between one pair of events (--reps)


def _time(fn, iters, warmup=3):
    """Median and best device time of one call, in ms.  With --reps > 1 that many calls are queued
    back to back between two events, so that the host's marshalling of a call overlaps the
    previous call's kernels (a lone call between two events counts about 10 us of idle GPU as
    its own)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    times = []
    for _ in range(iters):
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(REPS):
            fn()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / REPS)
    return statistics.median(times), min(times)


def _report(config, call, ms_med, ms_best, elems, nbytes, peak, extra=None):
    line = {"config": config, "call": call, "ms_median": round(ms_med, 4),
            "ms_best": round(ms_best, 4), "Gelem_per_s": round(elems / ms_med / 1e6, 1),
            "algorithmic_GBps": round(nbytes / ms_med / 1e6, 1),
            "frac_of_hbm_peak": round(nbytes / ms_med / 1e6 / peak, 4)}
    if extra:
        line.update(extra)
    print(json.dumps(line), flush=True)


def run_cnat(config, n, d, make_vector, iters, peak, with_sum=True):
    dev = "cuda"
    u8 = dict(dtype=torch.uint8, device=dev)
    xs = [make_vector(w) for w in range(n)]
    es = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
    ss = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
    out = torch.empty(d, dtype=torch.float32, device=dev)
    ge = torch.empty(nc.nc_exp_bytes(d), **u8)
    gs = torch.empty(nc.nc_sign_bytes(d), **u8)
    workers = list(range(n))
    m, b = _time(lambda: nc.nc_compress_batch(xs, d, 0, workers, es, ss, n), iters)
    _report(config, "nc_compress_batch", m, b, n * d, n * d * 5.125, peak, {"n": n, "d": d})
    m_det, b = _time(lambda: nc.nc_compress_nearest_batch(xs, d, es, ss, n), iters)
    _report(config, "nc_compress_nearest_batch (no sampling)", m_det, b, n * d, n * d * 5.125, peak,
            {"sampling_overhead": round(m / m_det - 1.0, 3)})
    nc.nc_compress_batch(xs, d, 0, workers, es, ss, n)       # planes of the stochastic operator
    m, b = _time(lambda: nc.nc_aggregate(es, ss, n, d, out), iters)
    _report(config, "nc_aggregate", m, b, d, d * (1.125 * n + 4), peak)
    m, b = _time(lambda: nc.nc_aggregate_compress(es, ss, n, d, 0, 0xFFFFFFFF, ge, gs), iters)
    _report(config, "nc_aggregate_compress", m, b, d, d * (1.125 * n + 1.125), peak)
    # the paper's 8-bit wire format with integer (order-independent) aggregation
    m, b = _time(lambda: nc.nc8_compress_batch(xs, d, 0, workers, es, n), iters)
    _report(config, "nc8_compress_batch (8-bit codes)", m, b, n * d, n * d * 5.0, peak)
    m, b = _time(lambda: nc.nc8_aggregate(es, n, d, out), iters)
    _report(config, "nc8_aggregate (int64 sums)", m, b, d, d * (1.0 * n + 4), peak)
    # 16-bit inputs (the same operator on bfloat16 / binary16 gradients): 2 + 1.125 bytes per entry
    for name, tdt, code in (("bf16", torch.bfloat16, nc.DTYPE_BF16),
                            ("f16", torch.float16, nc.DTYPE_F16)):
        xh = [x.to(tdt) for x in xs]
        m, b = _time(lambda: nc.nc_compress_typed_batch(xh, code, d, 0, workers, es, ss, n), iters)
        _report(config, "nc_compress_typed_batch (%s inputs)" % name, m, b, n * d, n * d * 3.125,
                peak, {"note": "generator-bound: the multiplier-pipe ceiling is about 1860-2070 "
                               "Gelem/s, the HBM roof 2093 Gelem/s"})
        if code == nc.DTYPE_BF16:
            m, b = _time(lambda: nc.nc_compress_bf16_r8_batch(xh, d, 0, workers, es, ss, n), iters)
            _report(config, "nc_compress_bf16_r8_batch (bf16 inputs, 7-bit thresholds)", m, b,
                    n * d, n * d * 3.125, peak,
                    {"note": "one generator block per 16 entries: memory-bound"})
        if code == nc.DTYPE_F16:
            m, b = _time(lambda: nc.nc_compress_f16_r16_batch(xh, d, 0, workers, es, ss, n), iters)
            _report(config, "nc_compress_f16_r16_batch (f16 inputs, 10-bit thresholds)", m, b,
                    n * d, n * d * 3.125, peak, {"note": "one generator block per 8 entries"})
        del xh
    if with_sum:
        m, b = _time(lambda: nc.nc_sum_fp32(xs, n, d, out), iters)
        _report(config, "nc_sum_fp32 (uncompressed reference point)", m, b, d, d * (4 * n + 4),
                peak)


def run_cnat64(config, n, d, iters, peak):
    dev = "cuda"
    u8 = dict(dtype=torch.uint8, device=dev)
    g = torch.Generator(device=dev)
    g.manual_seed(64)
    xs = [torch.randn(d, dtype=torch.float64, device=dev, generator=g) * 1e-3 for _ in range(n)]
    es = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
    hs = [torch.empty(nc.nd_level_bytes(d), **u8) for _ in range(n)]
    out = torch.empty(d, dtype=torch.float64, device=dev)
    workers = list(range(n))
    m, b = _time(lambda: nc.nc64_compress_batch(xs, d, 0, workers, es, hs, n), iters)
    _report(config, "nc64_compress_batch (binary64, 12-bit codes)", m, b, n * d, n * d * 9.5, peak,
            {"n": n, "d": d})
    m, b = _time(lambda: nc.nc64_aggregate(es, hs, n, d, out), iters)
    _report(config, "nc64_aggregate", m, b, d, d * (1.5 * n + 8), peak)


def run_dnat(config, n, sizes, iters, peak, p=2, s=8):
    dev = "cuda"
    u8 = dict(dtype=torch.uint8, device=dev)
    off = workloads.offsets_from_sizes(sizes)
    d, B = off[-1], len(sizes)
    off_dev = torch.tensor(off, dtype=torch.int64, device=dev)
    xs = [workloads.config2_vector(w, dev, sizes) for w in range(n)]
    norms = [torch.empty(B, dtype=torch.float32, device=dev) for _ in range(n)]
    levels = [torch.empty(nc.nd_level_bytes(d), **u8) for _ in range(n)]
    signs = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
    ws_bytes = nc.nd_batch_workspace_bytes(d, B, n)
    ws = torch.empty(ws_bytes, **u8)
    out = torch.empty(d, dtype=torch.float32, device=dev)
    workers = list(range(n))
    m, b = _time(lambda: nc.nd_compress_batch(xs, d, off_dev, B, p, s, 0, workers, norms, levels,
                                              signs, n, ws, ws_bytes), iters)
    _report(config, "nd_compress_batch", m, b, n * d, n * d * 8.625, peak,
            {"n": n, "d": d, "B": B, "note": "bytes count x twice (norm pass + rounding pass)"})
    m, b = _time(lambda: nc.nd_aggregate(norms, levels, signs, n, d, off_dev, B, s, out), iters)
    _report(config, "nd_aggregate", m, b, d, d * (0.625 * n + 4), peak)


def run_sparse(config, n, d, iters, peak, s=4):
    dev = "cuda"
    u8 = dict(dtype=torch.uint8, device=dev)
    cap = int(d * 0.0125)
    xs = [workloads.config5_vector(w, d, dev) for w in range(n)]
    idx = [torch.empty(cap, dtype=torch.int32, device=dev) for _ in range(n)]
    codes = [torch.empty((cap + 1) // 2 + 16, **u8) for _ in range(n)]
    count = [torch.zeros(1, dtype=torch.int32, device=dev) for _ in range(n)]
    norm = [torch.zeros(1, dtype=torch.float32, device=dev) for _ in range(n)]
    ws_bytes = nc.nd_sparse_batch_workspace_bytes(d, cap, n)
    ws = torch.empty(ws_bytes, **u8)
    acc = torch.zeros(d, dtype=torch.float32, device=dev)
    workers = list(range(n))
    thr, scale = workloads.KEEP_1PCT_THRESHOLD, workloads.KEEP_1PCT_SCALE
    m, b = _time(lambda: nc.nd_sparse_compress_batch(xs, d, thr, scale, nc.P_INF, s, 0, workers,
                                                     idx, codes, count, norm, cap, n, ws,
                                                     ws_bytes), iters)
    kept = 0.01 * d
    _report(config, "nd_sparse_compress_batch", m, b, n * d, n * kept * 68.5, peak,
            {"n": n, "d": d, "Gcoord_per_s": round(n * d / m / 1e6, 1),
             "note": "ALU-bound: one Philox block per 4 coordinates; the multiplier-pipe ceiling "
                     "is about 2070 Gcoord/s at 1965 MHz"})

    def accumulate():
        for w in range(n):
            nc.nd_sparse_decode_accumulate(idx[w], codes[w], count[w], norm[w], s, d, cap, acc)

    m, b = _time(accumulate, iters)
    _report(config, "nd_sparse_decode_accumulate x n", m, b, n * kept, n * kept * 68.5, peak)

    # the same update without the index list: the master regenerates the kept set from the seed
    rws_bytes = nc.nd_sparse_regen_workspace_bytes(d)
    rws = torch.empty(rws_bytes, **u8)

    def accumulate_regen():
        for w in range(n):
            nc.nd_sparse_regen_decode_accumulate(codes[w], count[w], norm[w], d, thr, s, 0, w, cap,
                                                 acc, rws, rws_bytes)

    m, b = _time(accumulate_regen, iters)
    _report(config, "nd_sparse_regen_decode_accumulate x n (no index list)", m, b, n * kept,
            n * kept * 64.5, peak, {"Gcoord_per_s": round(n * d / m / 1e6, 1),
                                    "wire_bytes_per_kept_entry": 0.5})

    # the compact format: level-0 entries dropped, 3-bit codes as bit planes
    planes = [torch.empty(nc.nd_sparse_plane_bytes(cap, s), **u8) for _ in range(n)]
    m, b = _time(lambda: nc.nd_sparse_compact_compress_batch(xs, d, thr, scale, nc.P_INF, s, 0,
                                                             workers, idx, planes, count, norm,
                                                             cap, n, ws, ws_bytes), iters)
    listed = sum(int(c.cpu().numpy().view("uint32")[0]) for c in count)
    _report(config, "nd_sparse_compact_compress_batch", m, b, n * d,
            n * kept * 96 + listed * 4.375, peak,
            {"Gcoord_per_s": round(n * d / m / 1e6, 1), "listed_fraction_of_kept":
             round(listed / (n * kept), 3)})

    def accumulate_compact():
        for w in range(n):
            nc.nd_sparse_compact_decode_accumulate(idx[w], planes[w], count[w], norm[w], s, d,
                                                   cap, acc)

    m, b = _time(accumulate_compact, iters)
    _report(config, "nd_sparse_compact_decode_accumulate x n", m, b, listed, listed * 68.4, peak)

    m, b = _time(lambda: nc.nd_sparse_compact_aggregate(idx, planes, count, norm, n, s, d, cap,
                                                        acc), iters)
    _report(config, "nd_sparse_compact_aggregate (all workers, one launch, dense output)", m, b,
            listed, 4.0 * d + listed * 4.375, peak)

    # exactly q = d / 100 kept coordinates (radix select over the selection words), one worker
    q = d // 100
    sel_bytes = nc.nc_select_workspace_bytes(d, cap)
    sel_ws = torch.empty(sel_bytes, **u8)
    m, b = _time(lambda: nc.nd_sparse_exact_compress(xs[0], d, q, scale, nc.P_INF, s, 0, 0, idx[0],
                                                     planes[0], count[0], norm[0], cap, sel_ws,
                                                     sel_bytes), iters)
    _report(config, "nd_sparse_exact_compress (1 worker)", m, b, d, q * 96.0, peak,
            {"Gcoord_per_s": round(d / m / 1e6, 1),
             "note": "two sweeps over the selection stream (digit histogram, mark) + candidate list"})
    # TopK then C_nat, K = d / 100, one worker: x is read three times (2 histograms + mark)
    K = q
    tidx = torch.empty(K, dtype=torch.int32, device=dev)
    texp = torch.empty(K, **u8)
    tsign = torch.empty(4 * ((K + 31) // 32) + 16, **u8)
    m, b = _time(lambda: nc.nc_topk_compress(xs[0], d, K, 0, 0, tidx, texp, tsign, sel_ws,
                                             sel_bytes), iters)
    _report(config, "nc_topk_compress (1 worker)", m, b, d, d * 4.0 + K * 5.125, peak,
            {"Gcoord_per_s": round(d / m / 1e6, 1), "hbm_bytes_actually_read": d * 12})


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", required=True, choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--peak-gbs", type=float, default=HBM_PEAK_FALLBACK,
                    help="HBM bandwidth the fractions are quoted against")
    ap.add_argument("--reps", type=int, default=1,
                    help="calls queued back to back between one pair of events")
    ap.add_argument("--workers", type=int, default=0,
                    help="override the number of simulated workers (smaller cases for profiling)")
    ap.add_argument("--log2-d", type=int, default=0,
                    help="override the vector length of c5 with 2^LOG2_D")
    args = ap.parse_args()
    global REPS
    REPS = max(1, args.reps)
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    peak = args.peak_gbs
    if args.config == "c1":
        d = 1 << 20
        run_cnat("c1", 4, d, lambda w: workloads.config1_vector(w, d, "cuda"), args.iters, peak)
    elif args.config == "c2":
        sizes = workloads.resnet50_tensor_sizes()
        d = sum(sizes)
        n = args.workers or 8
        run_cnat("c2", n, d, lambda w: workloads.config2_vector(w, "cuda", sizes), args.iters,
                 peak)
        run_cnat64("c2", n, d, args.iters, peak)
    elif args.config == "c3":
        run_dnat("c3", 8, workloads.resnet50_tensor_sizes(), args.iters, peak)
    elif args.config == "c4":
        d = sum(workloads.bert_large_bucket_sizes())
        run_cnat("c4", 16, d, lambda w: workloads.config4_vector(w, d, "cuda"), args.iters, peak)
    else:
        run_sparse("c5", args.workers or 8, 1 << (args.log2_d or 28), args.iters, peak)


if __name__ == "__main__":
    main()
