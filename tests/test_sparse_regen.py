"""Sparse update without an index list: the receiver regenerates the kept set from the seed.
Oracle pins on CPU, GPU parity (bit-exact) through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_1905_10988_b200 import workloads

THR, SCALE = workloads.KEEP_1PCT_THRESHOLD, workloads.KEEP_1PCT_SCALE


def test_regenerated_update_equals_the_update_with_the_index_list():
    rng = np.random.default_rng(0)
    d, s = 80_000, 4
    x = rng.standard_normal(d).astype(np.float32)
    for thr, scale, p in [(THR * 20, 5.0, oracle.P_INF), (1 << 31, 2.0, 2), (1 << 32, 1.0, 1),
                          (0, 1.0, oracle.P_INF)]:
        idx, codes, count, nrm = oracle.sparse_compress(x, thr, scale, p, s, 6, 2)
        start = rng.standard_normal(d).astype(np.float32)
        a, b = start.copy(), start.copy()
        oracle.sparse_decode_accumulate(idx, codes, count, nrm, s, a)
        oracle.sparse_regen_decode_accumulate(codes, count, nrm, thr, s, 6, 2, b)
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
        # the regenerated set is "stream word < threshold" and nothing else
        kept = np.nonzero(oracle.stream_words(6, 2, 2, 0, d).astype(np.uint64) < thr)[0]
        assert np.array_equal(kept.astype(np.uint32), idx)
    # a truncated list applies only its first entries
    idx, codes, count, nrm = oracle.sparse_compress(x, 1 << 30, 4.0, oracle.P_INF, s, 6, 2)
    a, b = np.zeros(d, np.float32), np.zeros(d, np.float32)
    oracle.sparse_decode_accumulate(idx[:100], codes, 100, nrm, s, a)
    oracle.sparse_regen_decode_accumulate(codes, 100, nrm, 1 << 30, s, 6, 2, b)
    assert np.array_equal(a, b) and np.count_nonzero(b[idx[100]:]) == 0


@pytest.mark.gpu
@pytest.mark.parametrize("d,thr,scale", [(1, 1 << 32, 1.0), (1000, 1 << 30, 4.0), (4097, THR, SCALE),
                                         (200_003, THR * 4, 25.0), ((1 << 20) + 9, THR, SCALE),
                                         (5000, 0, 1.0), (70_000, 1 << 32, 1.0)])
def test_gpu_regen_matches_oracle(d, thr, scale):
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import Guarded, dev
    rng = np.random.default_rng(d)
    s = 4
    x = rng.standard_normal(d).astype(np.float32)
    cap = d
    idx = Guarded(4 * cap)
    codes = Guarded((cap + 1) // 2 + 16)
    count = Guarded(4)
    norm = Guarded(4)
    ws_bytes = nc.nd_sparse_workspace_bytes(d, cap)
    ws = Guarded(ws_bytes)
    nc.nd_sparse_compress(dev(x), d, thr, scale, nc.P_INF, s, 3, 7, idx.buf, codes.buf, count.buf,
                          norm.buf, cap, ws.buf, ws_bytes)
    start = rng.standard_normal(d).astype(np.float32)
    acc = Guarded(4 * d)
    acc.buf.copy_(dev(start).view(torch.uint8))
    rws_bytes = nc.nd_sparse_regen_workspace_bytes(d)
    rws = Guarded(rws_bytes)
    nc.nd_sparse_regen_decode_accumulate(codes.buf, count.buf, norm.buf, d, thr, s, 3, 7, cap,
                                         acc.buf, rws.buf, rws_bytes)
    torch.cuda.synchronize()
    for g in (idx, codes, count, norm, ws, acc, rws):
        g.check()
    i_ref, c_ref, n_ref, nm_ref = oracle.sparse_compress(x, thr, scale, oracle.P_INF, s, 3, 7)
    ref = start.copy()
    oracle.sparse_regen_decode_accumulate(c_ref, n_ref, nm_ref, thr, s, 3, 7, ref)
    assert np.array_equal(acc.numpy(np.uint32), ref.view(np.uint32))
    # and it equals the GPU's own update with the index list
    acc2 = Guarded(4 * d)
    acc2.buf.copy_(dev(start).view(torch.uint8))
    nc.nd_sparse_decode_accumulate(idx.buf, codes.buf, count.buf, norm.buf, s, d, cap, acc2.buf)
    torch.cuda.synchronize()
    assert np.array_equal(acc.numpy(np.uint32), acc2.numpy(np.uint32))


@pytest.mark.gpu
def test_gpu_regen_respects_cap_on_config5_shape():
    import torch
    import paper_1905_10988_b200 as nc
    d, s = 1 << 24, 4
    x = workloads.config5_vector(3, d, "cuda")
    cap = 100_000                                      # fewer than the ~167,000 kept entries
    u8 = dict(dtype=torch.uint8, device="cuda")
    idx = torch.empty(cap, dtype=torch.int32, device="cuda")
    codes = torch.empty((cap + 1) // 2 + 16, **u8)
    count = torch.zeros(1, dtype=torch.int32, device="cuda")
    norm = torch.zeros(1, dtype=torch.float32, device="cuda")
    ws_bytes = nc.nd_sparse_workspace_bytes(d, cap)
    ws = torch.empty(ws_bytes, **u8)
    nc.nd_sparse_compress(x, d, THR, SCALE, nc.P_INF, s, 0, 3, idx, codes, count, norm, cap, ws,
                          ws_bytes)
    acc = torch.zeros(d, dtype=torch.float32, device="cuda")
    rws = torch.empty(nc.nd_sparse_regen_workspace_bytes(d), **u8)
    nc.nd_sparse_regen_decode_accumulate(codes, count, norm, d, THR, s, 0, 3, cap, acc, rws,
                                         rws.numel())
    torch.cuda.synchronize()
    i_ref, c_ref, n_ref, nm_ref = oracle.sparse_compress(x.cpu().numpy(), THR, SCALE, oracle.P_INF,
                                                         s, 0, 3, cap=cap)
    assert n_ref > cap
    ref = np.zeros(d, np.float32)
    oracle.sparse_regen_decode_accumulate(c_ref, cap, nm_ref, THR, s, 0, 3, ref)
    assert np.array_equal(acc.cpu().numpy().view(np.uint32), ref.view(np.uint32))
