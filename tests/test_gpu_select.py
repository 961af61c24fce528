"""GPU parity for the exact-count selection calls: S^q (exactly q kept coordinates) then D_nat in
the compact format, and TopK then C_nat.  Bit-exact against the oracle (indices, planes, counts,
exponent bytes, sign words; max-norm), p = 1, 2 norms within 1e-6 and codes against the given norm."""
import numpy as np
import pytest
import torch

import oracle
import paper_1905_10988_b200 as nc
from paper_1905_10988_b200 import workloads
from gpu_util import Guarded, dev

pytestmark = pytest.mark.gpu


def _gpu_exact(x, q, scale, p, s, seed, worker, cap):
    d = x.size
    idx = Guarded(4 * cap)
    planes = Guarded(nc.nd_sparse_plane_bytes(cap, s))
    count = Guarded(4)
    norm = Guarded(4)
    ws_bytes = nc.nc_select_workspace_bytes(d, cap)
    ws = Guarded(ws_bytes)
    nc.nd_sparse_exact_compress(dev(x), d, q, scale, p, s, seed, worker, idx.buf, planes.buf,
                                count.buf, norm.buf, cap, ws.buf, ws_bytes)
    torch.cuda.synchronize()
    for g in (idx, planes, count, norm, ws):
        g.check()
    return idx, planes, int(count.numpy(np.uint32)[0]), norm.numpy(np.float32)[0]


@pytest.mark.parametrize("d,q,s", [(1, 1, 4), (7, 3, 4), (1000, 10, 4), (1024, 1024, 4),
                                   (4097, 41, 4), (8192 * 3 + 5, 700, 3), (200_003, 2000, 4),
                                   ((1 << 20) + 9, 10_486, 4), (70_000, 35_000, 8),
                                   (5000, 4999, 1), (3000, 0, 4), (3000, 9999, 2)])
def test_exact_sparsifier_matches_oracle_max_norm(d, q, s):
    rng = np.random.default_rng(d + q)
    x = rng.standard_normal(d).astype(np.float32)
    scale = np.float32(d / max(min(q, d), 1))
    cap = d
    idx, planes, count, norm = _gpu_exact(x, q, scale, nc.P_INF, s, d, 3, cap)
    i_ref, p_ref, c_ref, n_ref = oracle.sparse_exact_compress(x, q, scale, oracle.P_INF, s, d, 3,
                                                              cap=cap)
    assert count == c_ref and norm == n_ref
    assert np.array_equal(idx.numpy(np.uint32)[:count], i_ref)
    assert np.array_equal(planes.numpy(np.uint32)[:p_ref.size], p_ref)


@pytest.mark.parametrize("p", [1, 2])
def test_exact_sparsifier_p_norms_and_cap(p):
    rng = np.random.default_rng(40 + p)
    d, q, s = 300_000, 30_000, 4
    x = (rng.standard_normal(d) * 10.0 ** rng.uniform(-3, 0, d)).astype(np.float32)
    scale = np.float32(d / q)
    cap = 300 if p == 2 else 4                   # below the number of listed entries
    idx, planes, count, norm = _gpu_exact(x, q, scale, p, s, 11, 6, cap)
    _, _, _, n_def = oracle.sparse_exact_compress(x, q, scale, p, s, 11, 6, cap=cap)
    assert abs(float(norm) - float(n_def)) <= 1e-6 * float(n_def)
    i_ref, p_ref, c_ref, _ = oracle.sparse_exact_compress(x, q, scale, p, s, 11, 6, cap=cap,
                                                          given_norm=norm)
    assert count == c_ref > cap
    assert np.array_equal(idx.numpy(np.uint32), i_ref)
    assert np.array_equal(planes.numpy(np.uint32)[:p_ref.size], p_ref)


def test_exact_sparsifier_keeps_exactly_q_with_s_large_enough_to_list_all():
    # with the max-norm and many levels almost every kept entry is listed; the selected set is the
    # q smallest selection words: check the count of selected coordinates through the norm path by
    # using x = 1 everywhere (every kept entry has level s, so listed == kept == q exactly)
    d, q, s = 123_457, 4321, 4
    x = np.ones(d, np.float32)
    idx, planes, count, norm = _gpu_exact(x, q, np.float32(1.0), nc.P_INF, s, 77, 0, d)
    assert count == q and norm == 1.0
    mask = oracle.select_smallest(oracle.stream_words(77, 0, 2, 0, d), q)
    assert np.array_equal(idx.numpy(np.uint32)[:q], np.nonzero(mask)[0].astype(np.uint32))


def _gpu_topk(x, K, seed, worker):
    d = x.size
    listed = min(K, d)
    idx = Guarded(4 * max(listed, 1))
    exp = Guarded(max(listed, 1))
    sign = Guarded(4 * max((listed + 31) // 32, 1))
    ws_bytes = nc.nc_select_workspace_bytes(d, max(listed, 1))
    ws = Guarded(ws_bytes)
    nc.nc_topk_compress(dev(x), d, K, seed, worker, idx.buf, exp.buf, sign.buf, ws.buf, ws_bytes)
    torch.cuda.synchronize()
    for g in (idx, exp, sign, ws):
        g.check()
    return idx, exp, sign, listed


@pytest.mark.parametrize("d,K", [(1, 1), (33, 5), (1024, 1024), (4097, 100), (50_000, 49_999),
                                 (200_003, 2000), ((1 << 20) + 9, 10_486), (3000, 5000)])
def test_topk_cnat_matches_oracle(d, K):
    rng = np.random.default_rng(d * 3 + K)
    x = (rng.standard_normal(d) * 10.0 ** rng.uniform(-4, 1, d)).astype(np.float32)
    idx, exp, sign, listed = _gpu_topk(x, K, 19, 5)
    i_ref, e_ref, s_ref = oracle.topk_compress(x, K, 19, 5)
    assert np.array_equal(idx.numpy(np.uint32)[:listed], i_ref)
    assert np.array_equal(exp.numpy(np.uint8)[:listed], e_ref)
    assert np.array_equal(sign.numpy(np.uint32)[:s_ref.size], s_ref)


def test_topk_ties_specials_and_decode_accumulate():
    rng = np.random.default_rng(8)
    d, K = 100_000, 3000
    x = rng.standard_normal(d).astype(np.float32)
    # quantise so that thousands of entries share the magnitude at the cut; add specials
    x = (np.round(x * 4) / 4).astype(np.float32)
    x[[5, 70_000]] = [np.inf, -np.inf]
    x[123] = np.nan
    x[[9, 10]] = [3.0e38, -1e-45]
    idx, exp, sign, listed = _gpu_topk(x, K, 2, 1)
    i_ref, e_ref, s_ref = oracle.topk_compress(x, K, 2, 1)
    cut = np.sort(np.abs(x[np.isfinite(x)]))[::-1][K]
    assert (np.abs(x) == cut).sum() > 100            # the tie case is really exercised
    assert np.array_equal(idx.numpy(np.uint32)[:listed], i_ref)
    assert np.array_equal(exp.numpy(np.uint8)[:listed], e_ref)
    assert np.array_equal(sign.numpy(np.uint32)[:s_ref.size], s_ref)
    # master side: scatter-add into a non-zero accumulator; entries decode to finite powers of
    # two, +-inf for the non-finite inputs
    start = rng.standard_normal(d).astype(np.float32)
    acc = Guarded(4 * d)
    acc.buf.copy_(dev(start).view(torch.uint8))
    nc.nc_topk_decode_accumulate(idx.buf, exp.buf, sign.buf, listed, d, acc.buf)
    torch.cuda.synchronize()
    acc.check()
    ref = start.copy()
    oracle.topk_decode_accumulate(i_ref, e_ref, s_ref, ref)
    assert np.array_equal(acc.numpy(np.uint32), ref.view(np.uint32))
    # all-equal input: the first K indices
    y = np.full(5000, -2.5, np.float32)
    idx, exp, sign, listed = _gpu_topk(y, 77, 2, 1)
    assert np.array_equal(idx.numpy(np.uint32)[:77], np.arange(77, dtype=np.uint32))


@pytest.mark.parametrize("kind", ["one_binade_slice", "all_equal", "two_values"])
def test_topk_every_selection_route(kind):
    # the device picks between three routes by how many keys share the leading digits of the
    # K-th key: candidates after the first digit (the cases above), candidates after the second
    # digit (more than 2^18 keys share the first 11 key bits), and all three digit passes with
    # ties broken by index (more than 2^18 keys equal in the first 22 bits)
    rng = np.random.default_rng(12)
    d = (1 << 20) + 77
    if kind == "one_binade_slice":
        x = (1.0 + rng.random(d) * 0.0624).astype(np.float32)
        x *= rng.choice(np.float32([-1, 1]), d)
        K = 5000
    elif kind == "all_equal":
        x = np.full(d, 0.75, np.float32)
        K = 300_001
    else:
        x = np.where(rng.random(d) < 0.4, np.float32(2.0), np.float32(-1.0)).astype(np.float32)
        K = int((x == 2.0).sum()) + 123_456          # all the 2.0 and the first 123,456 of the -1.0
    idx, exp, sign, listed = _gpu_topk(x, K, 4, 9)
    i_ref, e_ref, s_ref = oracle.topk_compress(x, K, 4, 9)
    assert np.array_equal(idx.numpy(np.uint32)[:listed], i_ref)
    assert np.array_equal(exp.numpy(np.uint8)[:listed], e_ref)
    assert np.array_equal(sign.numpy(np.uint32)[:s_ref.size], s_ref)


def test_exact_and_topk_on_config5_shape_sampled():
    # d = 2^26 of the sparse workload (the full 2^28 case is timed by the config bench): exact
    # count and threshold property checked in full, listed entries against the oracle on a prefix
    d, s = 1 << 26, 4
    q = d // 100
    x = workloads.config5_vector(2, d, "cuda")
    cap = q
    idx = torch.empty(cap, dtype=torch.int32, device="cuda")
    planes = torch.empty(nc.nd_sparse_plane_bytes(cap, s), dtype=torch.uint8, device="cuda")
    count = torch.zeros(1, dtype=torch.int32, device="cuda")
    norm = torch.zeros(1, dtype=torch.float32, device="cuda")
    ws_bytes = nc.nc_select_workspace_bytes(d, cap)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    nc.nd_sparse_exact_compress(x, d, q, 100.0, nc.P_INF, s, 0, 2, idx, planes, count, norm, cap,
                                ws, ws_bytes)
    torch.cuda.synchronize()
    xh = x.cpu().numpy()
    i_ref, p_ref, c_ref, n_ref = oracle.sparse_exact_compress(xh, q, 100.0, oracle.P_INF, s, 0, 2,
                                                              cap=cap)
    cnt = int(count.cpu().numpy().view(np.uint32)[0])
    assert cnt == c_ref and float(norm.cpu()[0]) == float(n_ref)
    assert np.array_equal(idx[:cnt].cpu().numpy().view(np.uint32), i_ref)
    assert np.array_equal(planes.cpu().numpy().view(np.uint32)[:p_ref.size], p_ref)
    # TopK on the same vector
    K = q
    tidx = torch.empty(K, dtype=torch.int32, device="cuda")
    texp = torch.empty(K, dtype=torch.uint8, device="cuda")
    tsign = torch.empty((K + 31) // 32, dtype=torch.int32, device="cuda")
    nc.nc_topk_compress(x, d, K, 0, 2, tidx, texp, tsign, ws, ws_bytes)
    torch.cuda.synchronize()
    i_ref, e_ref, s_ref = oracle.topk_compress(xh, K, 0, 2)
    assert np.array_equal(tidx.cpu().numpy().view(np.uint32), i_ref)
    assert np.array_equal(texp.cpu().numpy(), e_ref)
    assert np.array_equal(tsign.cpu().numpy().view(np.uint32), s_ref)
