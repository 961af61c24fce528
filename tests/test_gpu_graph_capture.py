"""The library calls only enqueue kernels on the given stream (no allocation, no synchronisation),
so a whole step can be captured into a CUDA graph and replayed: outputs of a replay on new
inputs must equal those of the eager calls, bit for bit."""
import numpy as np
import pytest
import torch

import paper_1905_10988_b200 as nc
from paper_1905_10988_b200 import workloads

pytestmark = pytest.mark.gpu


def test_whole_step_replays_from_a_cuda_graph():
    n, d, s_nd, s_sp = 4, 300_007, 8, 4
    off = workloads.small_bucket_table(d, seed=3)
    B = len(off) - 1
    off_dev = torch.tensor(off, dtype=torch.int64, device="cuda")
    u8 = dict(dtype=torch.uint8, device="cuda")
    f32 = dict(dtype=torch.float32, device="cuda")
    x = [torch.empty(d, **f32) for _ in range(n)]
    workers = list(range(n))
    es = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
    ss = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
    out_nc = torch.empty(d, **f32)
    norms = [torch.empty(B, **f32) for _ in range(n)]
    levels = [torch.empty(nc.nd_level_bytes(d), **u8) for _ in range(n)]
    signs = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
    ws_bytes = nc.nd_batch_workspace_bytes(d, B, n)
    ws = torch.empty(ws_bytes, **u8)
    out_nd = torch.empty(d, **f32)
    cap = d
    idx = [torch.empty(cap, dtype=torch.int32, device="cuda") for _ in range(n)]
    planes = [torch.empty(nc.nd_sparse_plane_bytes(cap, s_sp), **u8) for _ in range(n)]
    count = [torch.zeros(1, dtype=torch.int32, device="cuda") for _ in range(n)]
    snorm = [torch.zeros(1, **f32) for _ in range(n)]
    sws_bytes = nc.nd_sparse_batch_workspace_bytes(d, cap, n)
    sws = torch.empty(sws_bytes, **u8)
    out_sp = torch.empty(d, **f32)
    # exact-count selection and TopK keep per-device state that is set up on the first call
    q = d // 50
    sel_bytes = nc.nc_select_workspace_bytes(d, cap)
    sel_ws = torch.empty(sel_bytes, **u8)
    xidx = torch.empty(cap, dtype=torch.int32, device="cuda")
    xplanes = torch.empty(nc.nd_sparse_plane_bytes(cap, s_sp), **u8)
    xcount = torch.zeros(1, dtype=torch.int32, device="cuda")
    xnorm = torch.zeros(1, **f32)
    tidx = torch.empty(q, dtype=torch.int32, device="cuda")
    texp = torch.empty(q + 16, **u8)
    tsign = torch.empty(4 * ((q + 31) // 32) + 16, **u8)

    def step():
        nc.nc_compress_batch(x, d, 1, workers, es, ss, n)
        nc.nc_aggregate(es, ss, n, d, out_nc)
        nc.nd_compress_batch(x, d, off_dev, B, 2, s_nd, 1, workers, norms, levels, signs, n, ws,
                             ws_bytes)
        nc.nd_aggregate(norms, levels, signs, n, d, off_dev, B, s_nd, out_nd)
        nc.nd_sparse_compact_compress_batch(x, d, 1 << 28, 16.0, nc.P_INF, s_sp, 1, workers, idx,
                                            planes, count, snorm, cap, n, sws, sws_bytes)
        nc.nd_sparse_compact_aggregate(idx, planes, count, snorm, n, s_sp, d, cap, out_sp)
        nc.nd_sparse_exact_compress(x[0], d, q, float(d) / q, nc.P_INF, s_sp, 1, 0, xidx, xplanes,
                                    xcount, xnorm, cap, sel_ws, sel_bytes)
        nc.nc_topk_compress(x[1], d, q, 1, 1, tidx, texp, tsign, sel_ws, sel_bytes)

    outputs = [out_nc, out_nd, out_sp, xidx, xplanes, xcount, xnorm, tidx, texp, tsign]

    def fill(seed):
        g = torch.Generator(device="cuda")
        g.manual_seed(seed)
        for w in range(n):
            x[w].normal_(0.0, 1e-2, generator=g)

    fill(0)
    step()                                          # first call outside the capture
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            step()
    for seed in (1, 2):
        fill(seed)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        listed = int(xcount.cpu().numpy().view(np.uint32)[0])
        got = [o.clone() for o in outputs]
        for o in outputs:
            o.zero_()
        step()
        torch.cuda.synchronize()
        assert listed == int(xcount.cpu().numpy().view(np.uint32)[0])
        for name, a, b in zip(("nc", "nd", "sp", "xidx", "xplanes", "xcount", "xnorm", "tidx",
                               "texp", "tsign"), got, outputs):
            if name == "xidx":
                a, b = a[:listed], b[:listed]          # entries past the count are not written
            if name == "texp":
                a, b = a[:q], b[:q]
            if name == "tsign":
                a, b = a[:4 * ((q + 31) // 32)], b[:4 * ((q + 31) // 32)]
            assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), name
