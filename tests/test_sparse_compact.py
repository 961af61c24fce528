"""The compact sparse format (zero levels dropped, 3-bit codes as bit planes for s <= 4):
oracle pins on CPU, GPU parity through the C ABI (bit-exact: indices, planes, count, max-norm)."""
import numpy as np
import pytest

import oracle
from paper_1905_10988_b200 import workloads

THR, SCALE = workloads.KEEP_1PCT_THRESHOLD, workloads.KEEP_1PCT_SCALE


def _codes_from_planes(planes, count, s):
    nbits = oracle.code_bits(s)
    k = np.arange(count)
    code = np.zeros(count, np.uint32)
    for b in range(nbits):
        code |= ((planes[(k // 32) * nbits + b] >> (k % 32).astype(np.uint32)) & 1) << np.uint32(b)
    return code


def test_compact_form_is_the_listed_form_without_zero_levels():
    # the 4-bit listed form is pinned against the dense dithering path; dropping its level-0
    # entries and re-coding must give the compact form, and both decode to the same vector
    rng = np.random.default_rng(31)
    d = 120_000
    x = rng.standard_normal(d).astype(np.float32)
    for p, s, thr, scale in [(oracle.P_INF, 4, THR * 10, 10.0), (2, 3, 1 << 30, 4.0),
                             (oracle.P_INF, 8, 1 << 32, 1.0), (1, 1, THR * 10, 10.0)]:
        i4, c4, n4, nm4 = oracle.sparse_compress(x, thr, scale, p, min(s, 7), 9, 4) if s <= 7 \
            else (None, None, None, None)
        i3, planes, n3, nm3 = oracle.sparse_compact_compress(x, thr, scale, p, s, 9, 4)
        assert oracle.code_bits(s) == {1: 1, 3: 3, 4: 3, 8: 4}[s]
        codes = _codes_from_planes(planes, n3, s)
        nb = oracle.code_bits(s) - 1
        level = (codes & ((1 << nb) - 1)) + 1
        assert n3 == i3.size and np.all(np.diff(i3.astype(np.int64)) > 0)
        assert level.min() >= 1 and level.max() <= s
        b = np.zeros(d, np.float32)
        oracle.sparse_compact_decode_accumulate(i3, planes, n3, nm3, s, b)
        if i4 is not None:
            c = np.stack([c4 & 0xF, c4 >> 4], 1).ravel()[:n4]
            live = (c & 7) > 0
            assert nm3 == nm4
            assert np.array_equal(i4[live], i3)
            assert np.array_equal((c[live] & 7), level)
            assert np.array_equal(c[live] >> 3, codes >> nb)
            a = np.zeros(d, np.float32)
            oracle.sparse_decode_accumulate(i4, c4, n4, nm4, s, a)
            assert np.array_equal(a, b)
        # padding bits of the last group and unused groups are zero
        total_words = ((d + 31) // 32) * oracle.code_bits(s)
        assert planes.size == total_words
        used = ((n3 + 31) // 32) * oracle.code_bits(s)
        assert np.all(planes[used:] == 0)
        if n3 % 32:
            assert np.all(planes[used - oracle.code_bits(s):used] >> np.uint32(n3 % 32) == 0)


def test_compact_degenerate_and_cap():
    x = np.zeros(5000, np.float32)
    i3, planes, n3, nm3 = oracle.sparse_compact_compress(x, 1 << 31, 2.0, oracle.P_INF, 4, 1, 0)
    assert n3 == 0 and nm3 == 0 and not planes.any()
    rng = np.random.default_rng(5)
    x = rng.standard_normal(50_000).astype(np.float32)
    full = oracle.sparse_compact_compress(x, 1 << 30, 4.0, oracle.P_INF, 4, 2, 1)
    capped = oracle.sparse_compact_compress(x, 1 << 30, 4.0, oracle.P_INF, 4, 2, 1, cap=1000)
    assert capped[2] == full[2] > 1000 and np.array_equal(capped[0], full[0][:1000])
    nbits = oracle.code_bits(4)
    assert np.array_equal(capped[1][:(1000 // 32) * nbits], full[1][:(1000 // 32) * nbits])


def _gpu_compact(nc, x_dev, thr, scale, p, s, seed, worker, cap):
    import torch
    from gpu_util import Guarded
    d = x_dev.numel()
    idx = Guarded(4 * cap)
    planes = Guarded(nc.nd_sparse_plane_bytes(cap, s))
    count = Guarded(4)
    norm = Guarded(4)
    ws_bytes = nc.nd_sparse_workspace_bytes(d, cap)
    ws = Guarded(ws_bytes)
    nc.nd_sparse_compact_compress(x_dev, d, thr, scale, p, s, seed, worker, idx.buf, planes.buf,
                                  count.buf, norm.buf, cap, ws.buf, ws_bytes)
    torch.cuda.synchronize()
    for g in (idx, planes, count, norm, ws):
        g.check()
    return idx, planes, int(count.numpy(np.uint32)[0]), norm.numpy(np.float32)[0]


@pytest.mark.gpu
@pytest.mark.parametrize("d,thr,scale,s", [(1, 1 << 32, 1.0, 4), (1000, 1 << 30, 4.0, 4),
                                           (4097, THR, SCALE, 4), (200_003, THR * 4, 25.0, 3),
                                           ((1 << 20) + 9, THR, SCALE, 4),
                                           (70_000, 1 << 31, 2.0, 8), (5000, 1 << 32, 1.0, 1)])
def test_gpu_compact_matches_oracle(d, thr, scale, s):
    import paper_1905_10988_b200 as nc
    from gpu_util import dev
    rng = np.random.default_rng(d + s)
    x = rng.standard_normal(d).astype(np.float32)
    cap = d
    idx, planes, count, norm = _gpu_compact(nc, dev(x), thr, scale, nc.P_INF, s, d, 2, cap)
    i_ref, p_ref, c_ref, n_ref = oracle.sparse_compact_compress(x, thr, scale, oracle.P_INF, s, d,
                                                                2, cap=cap)
    assert count == c_ref and norm == n_ref
    assert np.array_equal(idx.numpy(np.uint32)[:count], i_ref)
    assert np.array_equal(planes.numpy(np.uint32)[:p_ref.size], p_ref)


@pytest.mark.gpu
def test_gpu_compact_batch_cap_and_accumulate_in_worker_order():
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import Guarded, dev
    rng = np.random.default_rng(77)
    n, d, s = 4, 300_000, 4
    thr, scale = THR * 8, 12.5
    cap = 9000                                  # below the ~19,000 surviving entries
    xs = [rng.standard_normal(d).astype(np.float32) for _ in range(n)]
    xd = [dev(x) for x in xs]
    workers = [3, 0, 8, 1]
    idx = [Guarded(4 * cap) for _ in range(n)]
    planes = [Guarded(nc.nd_sparse_plane_bytes(cap, s)) for _ in range(n)]
    count = [Guarded(4) for _ in range(n)]
    norm = [Guarded(4) for _ in range(n)]
    ws_bytes = nc.nd_sparse_batch_workspace_bytes(d, cap, n)
    ws = Guarded(ws_bytes)
    nc.nd_sparse_compact_compress_batch(xd, d, thr, scale, nc.P_INF, s, 5, workers,
                                        [g.buf for g in idx], [g.buf for g in planes],
                                        [g.buf for g in count], [g.buf for g in norm], cap, n,
                                        ws.buf, ws_bytes)
    acc = Guarded(4 * d)
    start = rng.standard_normal(d).astype(np.float32)
    acc.buf.copy_(dev(start).view(torch.uint8))
    for i in range(n):
        nc.nd_sparse_compact_decode_accumulate(idx[i].buf, planes[i].buf, count[i].buf,
                                               norm[i].buf, s, d, cap, acc.buf)
    torch.cuda.synchronize()
    for g in idx + planes + count + norm + [ws, acc]:
        g.check()
    ref = start.copy()
    for i in range(n):
        i_ref, p_ref, c_ref, n_ref = oracle.sparse_compact_compress(xs[i], thr, scale,
                                                                    oracle.P_INF, s, 5,
                                                                    workers[i], cap=cap)
        cnt = int(count[i].numpy(np.uint32)[0])
        assert cnt == c_ref > cap and norm[i].numpy(np.float32)[0] == n_ref
        assert np.array_equal(idx[i].numpy(np.uint32), i_ref)
        assert np.array_equal(planes[i].numpy(np.uint32)[:p_ref.size], p_ref)
        oracle.sparse_compact_decode_accumulate(i_ref, p_ref, min(c_ref, cap), n_ref, s, ref)
    assert np.array_equal(acc.numpy(np.uint32), ref.view(np.uint32))


@pytest.mark.gpu
def test_config5_full_size_compact_one_worker():
    # d = 2^28, keep 1 %, D_nat^{inf,4}, 3-bit codes: one worker in full against the oracle
    import torch
    import paper_1905_10988_b200 as nc
    d, s = 1 << 28, 4
    cap = int(d * 0.0125)
    x = workloads.config5_vector(1, d, "cuda")
    idx = torch.empty(cap, dtype=torch.int32, device="cuda")
    planes = torch.empty(nc.nd_sparse_plane_bytes(cap, s), dtype=torch.uint8, device="cuda")
    count = torch.zeros(1, dtype=torch.int32, device="cuda")
    norm = torch.zeros(1, dtype=torch.float32, device="cuda")
    ws_bytes = nc.nd_sparse_workspace_bytes(d, cap)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    nc.nd_sparse_compact_compress(x, d, THR, SCALE, nc.P_INF, s, 0, 1, idx, planes, count, norm,
                                  cap, ws, ws_bytes)
    acc = torch.zeros(d, dtype=torch.float32, device="cuda")
    nc.nd_sparse_compact_decode_accumulate(idx, planes, count, norm, s, d, cap, acc)
    torch.cuda.synchronize()
    i_ref, p_ref, c_ref, n_ref = oracle.sparse_compact_compress(x.cpu().numpy(), THR, SCALE,
                                                                oracle.P_INF, s, 0, 1, cap=cap)
    cnt = int(count.cpu().numpy().view(np.uint32)[0])
    assert cnt == c_ref <= cap and float(norm.cpu()[0]) == float(n_ref)
    assert np.array_equal(idx[:cnt].cpu().numpy().view(np.uint32), i_ref)
    assert np.array_equal(planes.cpu().numpy().view(np.uint32)[:p_ref.size], p_ref)
    ref = np.zeros(d, np.float32)
    oracle.sparse_compact_decode_accumulate(i_ref, p_ref, c_ref, n_ref, s, ref)
    assert np.array_equal(acc.cpu().numpy().view(np.uint32), ref.view(np.uint32))


@pytest.mark.gpu
def test_config5_full_size_all_workers_batch_and_aggregate():
    # config 5 at its own shape in the calls the benchmark times: d = 2^28, n = 8, one batch
    # compress call and the one-launch aggregate; every list and the whole dense sum compared
    import torch
    import paper_1905_10988_b200 as nc
    n, d, s = 8, 1 << 28, 4
    free, _ = torch.cuda.mem_get_info()
    if free < 16 * (1 << 30):
        pytest.skip("needs ~12 GB of free device memory")
    cap = int(d * 0.0125)
    u8 = dict(dtype=torch.uint8, device="cuda")
    xd = [workloads.config5_vector(w, d, "cuda") for w in range(n)]
    idx = [torch.empty(cap, dtype=torch.int32, device="cuda") for _ in range(n)]
    planes = [torch.empty(nc.nd_sparse_plane_bytes(cap, s), **u8) for _ in range(n)]
    count = [torch.zeros(1, dtype=torch.int32, device="cuda") for _ in range(n)]
    norm = [torch.zeros(1, dtype=torch.float32, device="cuda") for _ in range(n)]
    ws_bytes = nc.nd_sparse_batch_workspace_bytes(d, cap, n)
    ws = torch.empty(ws_bytes, **u8)
    nc.nd_sparse_compact_compress_batch(xd, d, THR, SCALE, nc.P_INF, s, 0, list(range(n)), idx,
                                        planes, count, norm, cap, n, ws, ws_bytes)
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nd_sparse_compact_aggregate(idx, planes, count, norm, n, s, d, cap, out)
    torch.cuda.synchronize()
    ref = np.zeros(d, np.float32)
    for w in range(n):
        i_ref, p_ref, c_ref, n_ref = oracle.sparse_compact_compress(xd[w].cpu().numpy(), THR, SCALE,
                                                                    oracle.P_INF, s, 0, w, cap=cap)
        cnt = int(count[w].cpu().numpy().view(np.uint32)[0])
        assert cnt == c_ref <= cap and float(norm[w].cpu()[0]) == float(n_ref)
        assert np.array_equal(idx[w][:cnt].cpu().numpy().view(np.uint32), i_ref)
        assert np.array_equal(planes[w].cpu().numpy().view(np.uint32)[:p_ref.size], p_ref)
        oracle.sparse_compact_decode_accumulate(i_ref, p_ref, c_ref, n_ref, s, ref)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32))
    del xd, out
    torch.cuda.empty_cache()


@pytest.mark.gpu
@pytest.mark.parametrize("n,d,thr,scale,cap_frac", [(1, 5, 1 << 32, 1.0, 1.0),
                                                    (3, 8192, 1 << 30, 4.0, 1.0),
                                                    (4, 300_000, THR * 8, 12.5, 1.0),
                                                    (8, (1 << 20) + 77, THR, SCALE, 1.0),
                                                    (16, 50_001, 1 << 31, 2.0, 0.1),
                                                    (64, 20_000, 1 << 32, 1.0, 1.0)])
def test_gpu_compact_aggregate_one_launch_matches_oracle(n, d, thr, scale, cap_frac):
    # dense sum of n compact lists in worker order; equals the oracle's zero fill followed by the
    # per-worker decode-accumulate, and the GPU's own per-worker calls
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import Guarded, dev
    rng = np.random.default_rng(n * 7 + d)
    s = 4
    cap = max(int(d * cap_frac), 1)
    xs = [rng.standard_normal(d).astype(np.float32) for _ in range(n)]
    workers = list(range(20, 20 + n))
    idx = [Guarded(4 * cap) for _ in range(n)]
    planes = [Guarded(nc.nd_sparse_plane_bytes(cap, s)) for _ in range(n)]
    count = [Guarded(4) for _ in range(n)]
    norm = [Guarded(4) for _ in range(n)]
    ws_bytes = nc.nd_sparse_batch_workspace_bytes(d, cap, n)
    ws = Guarded(ws_bytes)
    nc.nd_sparse_compact_compress_batch([dev(x) for x in xs], d, thr, scale, nc.P_INF, s, 9,
                                        workers, [g.buf for g in idx], [g.buf for g in planes],
                                        [g.buf for g in count], [g.buf for g in norm], cap, n,
                                        ws.buf, ws_bytes)
    out = Guarded(4 * d)
    out.buf.fill_(0x7F)                                  # the call must overwrite everything
    nc.nd_sparse_compact_aggregate([g.buf for g in idx], [g.buf for g in planes],
                                   [g.buf for g in count], [g.buf for g in norm], n, s, d, cap,
                                   out.buf)
    acc = Guarded(4 * d)
    acc.buf.zero_()
    for i in range(n):
        nc.nd_sparse_compact_decode_accumulate(idx[i].buf, planes[i].buf, count[i].buf,
                                               norm[i].buf, s, d, cap, acc.buf)
    torch.cuda.synchronize()
    out.check()
    ref = np.zeros(d, np.float32)
    for i in range(n):
        i_ref, p_ref, c_ref, n_ref = oracle.sparse_compact_compress(xs[i], thr, scale,
                                                                    oracle.P_INF, s, 9,
                                                                    workers[i], cap=cap)
        oracle.sparse_compact_decode_accumulate(i_ref, p_ref, min(c_ref, cap), n_ref, s, ref)
    assert np.array_equal(out.numpy(np.uint32), ref.view(np.uint32))
    assert np.array_equal(out.numpy(np.uint32), acc.numpy(np.uint32))


@pytest.mark.gpu
def test_compact_bench_launch_configuration_full_size():
    # exactly what the benchmark step runs for the sparse part: 8 workers, d = 25,557,032, one
    # batch compress call and one aggregate call; every output compared in full
    import torch
    import paper_1905_10988_b200 as nc
    n, s = 8, 4
    sizes = workloads.resnet50_tensor_sizes()
    d = sum(sizes)
    cap = int(d * 0.0125)
    u8 = dict(dtype=torch.uint8, device="cuda")
    xd = [workloads.config2_vector(w, "cuda", sizes) for w in range(n)]
    idx = [torch.empty(cap, dtype=torch.int32, device="cuda") for _ in range(n)]
    planes = [torch.empty(nc.nd_sparse_plane_bytes(cap, s), **u8) for _ in range(n)]
    count = [torch.zeros(1, dtype=torch.int32, device="cuda") for _ in range(n)]
    norm = [torch.zeros(1, dtype=torch.float32, device="cuda") for _ in range(n)]
    ws_bytes = nc.nd_sparse_batch_workspace_bytes(d, cap, n)
    ws = torch.empty(ws_bytes, **u8)
    nc.nd_sparse_compact_compress_batch(xd, d, THR, SCALE, nc.P_INF, s, 0, list(range(n)), idx,
                                        planes, count, norm, cap, n, ws, ws_bytes)
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nd_sparse_compact_aggregate(idx, planes, count, norm, n, s, d, cap, out)
    torch.cuda.synchronize()
    ref = np.zeros(d, np.float32)
    for w in range(n):
        i_ref, p_ref, c_ref, n_ref = oracle.sparse_compact_compress(xd[w].cpu().numpy(), THR, SCALE,
                                                                    oracle.P_INF, s, 0, w, cap=cap)
        cnt = int(count[w].cpu().numpy().view(np.uint32)[0])
        assert cnt == c_ref <= cap and float(norm[w].cpu()[0]) == float(n_ref)
        assert np.array_equal(idx[w][:cnt].cpu().numpy().view(np.uint32), i_ref)
        assert np.array_equal(planes[w].cpu().numpy().view(np.uint32)[:p_ref.size], p_ref)
        oracle.sparse_compact_decode_accumulate(i_ref, p_ref, c_ref, n_ref, s, ref)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32))
