"""GPU parity, natural dithering: norms within 1e-6 relative (max-norm exact); level codes
bit-exact against the oracle run on the GPU's own norms (given-norm mode) and within
1e-5 adjacent-only differences against the oracle's definition mode; signs, padding and the
decode / n-way sum bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import paper_1905_10988_b200 as nc
from paper_1905_10988_b200 import workloads
from gpu_util import Guarded, assert_same_floats, dev, unpack_nibbles

pytestmark = pytest.mark.gpu

NORM_RTOL = 1e-6
CODE_MISMATCH = 1e-5


def gpu_nd_compress(x_dev, off, p, s, seed, worker):
    d = x_dev.numel()
    B = len(off) - 1
    off_dev = dev(np.asarray(off, np.uint64).view(np.int64))
    norms = Guarded(4 * B)
    level = Guarded(nc.nd_level_bytes(d))
    sign = Guarded(nc.nc_sign_bytes(d))
    ws_bytes = nc.nd_workspace_bytes(d, B)
    ws = Guarded(ws_bytes)
    nc.nd_compress(x_dev, d, off_dev, B, p, s, seed, worker, norms.buf, level.buf, sign.buf,
                   ws.buf, ws_bytes)
    torch.cuda.synchronize()
    for g in (norms, level, sign, ws):
        g.check()
    return norms, level, sign


def check_against_oracle(x, off, p, s, seed, worker, norms, level, sign):
    d = x.size
    gn = norms.numpy(np.float32)
    lv = level.numpy(np.uint8)
    sg = sign.numpy(np.uint32)
    # definition mode: the oracle's own norms
    n0, l0, s0 = oracle.nd_compress(x, off, p, s, seed, worker)
    finite = np.isfinite(n0)
    assert np.array_equal(np.isnan(gn), np.isnan(n0))
    assert np.array_equal(np.isinf(gn), np.isinf(n0))
    if p == nc.P_INF:
        assert np.array_equal(gn[finite], n0[finite])
    else:
        assert np.all(np.abs(gn[finite] - n0[finite]) <= NORM_RTOL * np.abs(n0[finite]))
    nw = (d + 31) // 32
    assert np.array_equal(sg[:nw], s0) and np.all(sg[nw:] == 0)
    assert np.all(lv[(d + 1) // 2:] == 0)
    cg = unpack_nibbles(lv, d).astype(np.int64)
    # given-norm mode: same norms as the GPU -> codes must be identical
    _, l1, _ = oracle.nd_compress(x, off, p, s, seed, worker, given_norms=gn)
    assert np.array_equal(lv[:(d + 1) // 2], l1), "level plane differs from given-norm oracle"
    # definition mode: few, adjacent differences only
    c0 = unpack_nibbles(l0, d).astype(np.int64)
    diff = cg != c0
    assert diff.sum() <= int(CODE_MISMATCH * d)       # at small d: no difference at all
    assert np.all(np.abs(cg - c0)[diff] == 1)
    return gn


@pytest.mark.parametrize("p", [1, 2, 0])
@pytest.mark.parametrize("d,s", [(1, 4), (33, 1), (1000, 8), (1024, 8), (5000, 15), (70001, 8),
                                 ((1 << 18) + 40, 4)])
def test_compress_ragged_bucket_tables(d, s, p):
    rng = np.random.default_rng(d * 31 + s)
    off = workloads.small_bucket_table(d, seed=d + s)
    sig = 10.0 ** rng.uniform(-5, -2, len(off) - 1)
    x = (rng.standard_normal(d) * np.repeat(sig, np.diff(off))).astype(np.float32)
    norms, level, sign = gpu_nd_compress(dev(x), off, p, s, seed=d, worker=s)
    check_against_oracle(x, off, p, s, d, s, norms, level, sign)


def test_compress_single_bucket_and_aligned_buckets():
    rng = np.random.default_rng(5)
    d = 1 << 17
    x = (rng.standard_normal(d) * 2e-3).astype(np.float32)
    for off in ([0, d], list(range(0, d + 1, 4096)), [0, 1024, 1024, 2048, d]):
        norms, level, sign = gpu_nd_compress(dev(x), off, 2, 8, seed=1, worker=0)
        check_against_oracle(x, off, 2, 8, 1, 0, norms, level, sign)


def test_compress_degenerate_buckets():
    rng = np.random.default_rng(6)
    d = 6000
    x = (rng.standard_normal(d) * 1e-2).astype(np.float32)
    off = [0, 100, 1500, 1500, 2600, 4000, 5000, d]
    x[100:1500] = 0.0                  # x = 0 -> D(x) = 0
    x[100:1500:2] = -0.0
    x[2600:4000] = (rng.standard_normal(1400) * 1e-42).astype(np.float32)   # subnormal norm
    x[4100] = np.inf                   # non-finite norm
    x[5100] = np.nan
    for p in (1, 2, 0):
        norms, level, sign = gpu_nd_compress(dev(x), off, p, 8, seed=2, worker=1)
        gn = check_against_oracle(x, off, p, 8, 2, 1, norms, level, sign)
        c = unpack_nibbles(level.numpy(np.uint8), d)
        assert gn[1] == 0 and gn[2] == 0 and 0 < gn[4] < 2.0 ** -126
        assert np.isinf(gn[5]) and np.isnan(gn[6])
        for b in (1, 5, 6):
            assert np.all(c[off[b]:off[b + 1]] == 0)
        assert np.any(c[off[3]:off[4]] > 0)
        assert np.any(c[off[4]:off[5]] > 0)     # a subnormal norm is an ordinary norm
        assert np.any(c[:100] > 0)


def _random_planes(rng, n, d, B, s):
    norms = [(10.0 ** rng.uniform(-6, 1, B)).astype(np.float32) for _ in range(n)]
    levels, signs = [], []
    for _ in range(n):
        c = rng.integers(0, s + 1, nc.nd_level_bytes(d) * 2).astype(np.uint8)
        levels.append((c[0::2] | (c[1::2] << 4)).astype(np.uint8))
        signs.append(rng.integers(0, 1 << 32, nc.nc_sign_bytes(d) // 4, dtype=np.uint64)
                     .astype(np.uint32))
    return norms, levels, signs


# the last case has more tiles than are resident at once: its tail runs as 256-entry pieces
@pytest.mark.parametrize("n,d,s", [(1, 999, 8), (3, 4096, 4), (8, 70001, 8), (16, 5000, 15),
                                   (64, 2100, 1), (2, 5_000_333, 8)])
def test_aggregate_and_decode_accumulate_are_bit_exact(n, d, s):
    rng = np.random.default_rng(n * 7 + d)
    off = workloads.small_bucket_table(d, seed=n + d)
    B = len(off) - 1
    norms, levels, signs = _random_planes(rng, n, d, B, s)
    norms[0][0] = 2.0 ** -130                  # subnormal products
    if B > 2:
        norms[-1][1] = np.inf                  # level 0 stays 0, any other level decodes to inf
        norms[0][2] = 0.0
    if B > 4:
        norms[n // 2][3] = np.nan              # likewise NaN
        norms[0][4] = 2.0 ** -140              # a subnormal norm
    off_dev = dev(np.asarray(off, np.uint64).view(np.int64))
    nd_ = [dev(a) for a in norms]
    ld = [dev(a) for a in levels]
    sd = [dev(a) for a in signs]
    out = Guarded(4 * d)
    nc.nd_aggregate(nd_, ld, sd, n, d, off_dev, B, s, out.buf)
    torch.cuda.synchronize()
    out.check()
    want = oracle.nd_aggregate(norms, [l[:(d + 1) // 2] for l in levels], signs, off, s, d)
    assert_same_floats(out.numpy(np.float32), want)
    if B > 2:
        assert np.any(np.isinf(want[off[1]:off[2]])) or off[2] - off[1] < 4
    acc = Guarded(4 * d)
    start = rng.standard_normal(d).astype(np.float32)
    acc.buf.copy_(dev(start).view(torch.uint8))
    ref = start.copy()
    for i in range(n):
        nc.nd_decode_accumulate(nd_[i], ld[i], sd[i], d, off_dev, B, s, acc.buf)
        oracle.nd_decode_accumulate(norms[i], levels[i][:(d + 1) // 2], signs[i], off, s, ref)
    torch.cuda.synchronize()
    acc.check()
    assert_same_floats(acc.numpy(np.float32), ref)


def test_status_reports_buckets_that_are_not_finite():
    """A bucket holding an inf or a NaN is compressed to level 0 everywhere; the optional status
    word of the compress calls, and nd_norm_status on stored norms, count such buckets."""
    rng = np.random.default_rng(8)
    d = 9000
    off = [0, 1000, 1000, 3000, 5000, 7000, d]
    B = len(off) - 1
    xs = [(rng.standard_normal(d) * 1e-2).astype(np.float32) for _ in range(3)]
    xs[0][1500] = np.inf
    xs[0][5500] = np.nan
    xs[2][8999] = -np.inf
    off_dev = dev(np.asarray(off, np.uint64).view(np.int64))
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    n = len(xs)
    ws_bytes = nc.nd_batch_workspace_bytes(d, B, n)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    norms = [torch.empty(B, dtype=torch.float32, device="cuda") for _ in range(n)]
    levels = [torch.empty(nc.nd_level_bytes(d), dtype=torch.uint8, device="cuda") for _ in range(n)]
    signs = [torch.empty(nc.nc_sign_bytes(d), dtype=torch.uint8, device="cuda") for _ in range(n)]
    for p, expect in ((2, 3), (nc.P_INF, 6), (1, 9)):          # the word accumulates over calls
        nc.nd_compress_batch([dev(x) for x in xs], d, off_dev, B, p, 8, 0, [0, 1, 2], norms, levels,
                             signs, n, ws, ws_bytes, status=status[0:1])
        torch.cuda.synchronize()
        assert status.cpu().tolist() == [expect, 0]
    nc.nd_compress(dev(xs[1]), d, off_dev, B, 2, 8, 0, 1, norms[1], levels[1], signs[1], ws,
                   ws_bytes, status=status[0:1])               # a clean vector adds nothing
    nc.nd_norm_status(norms, n, B, status[1:2])
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [9, 3]
    # what the master sees when it aggregates all the same: the three buckets add zeros
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nd_aggregate(norms, levels, signs, n, d, off_dev, B, 8, out)
    torch.cuda.synchronize()
    ref = oracle.nd_aggregate([a.cpu().numpy() for a in norms],
                              [a.cpu().numpy()[:(d + 1) // 2] for a in levels],
                              [a.cpu().numpy().view(np.uint32)[:(d + 31) // 32] for a in signs],
                              off, 8, d)
    assert_same_floats(out.cpu().numpy(), ref)
    assert np.all(np.isfinite(ref))


def test_config3_full_size():
    # D_nat^{2,8} on the ResNet-50-shaped buckets, n = 8; every worker's norms, level and sign
    # planes in full against the oracle, and the whole aggregate
    n, p, s = 8, 2, 8
    sizes = workloads.resnet50_tensor_sizes()
    off = workloads.offsets_from_sizes(sizes)
    d, B = off[-1], len(sizes)
    off_dev = dev(np.asarray(off, np.uint64).view(np.int64))
    xd = [workloads.config2_vector(w, "cuda", sizes) for w in range(n)]
    ws_bytes = nc.nd_batch_workspace_bytes(d, B, n)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    norms = [torch.empty(B, dtype=torch.float32, device="cuda") for _ in range(n)]
    levels = [torch.empty(nc.nd_level_bytes(d), dtype=torch.uint8, device="cuda")
              for _ in range(n)]
    signs = [torch.empty(nc.nc_sign_bytes(d), dtype=torch.uint8, device="cuda") for _ in range(n)]
    # the launch configuration the benchmark times: one batch call for the 8 workers
    nc.nd_compress_batch(xd, d, off_dev, B, p, s, 0, list(range(n)), norms, levels, signs, n, ws,
                         ws_bytes)
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nd_aggregate(norms, levels, signs, n, d, off_dev, B, s, out)
    torch.cuda.synchronize()
    refs = []
    for w in range(n):
        x = xd[w].cpu().numpy()
        gn = norms[w].cpu().numpy()
        n0, l0, s0 = oracle.nd_compress(x, off, p, s, 0, w)
        assert np.all(np.abs(gn - n0) <= NORM_RTOL * n0)
        assert np.array_equal(signs[w].cpu().numpy().view(np.uint32)[:(d + 31) // 32], s0)
        _, l1, _ = oracle.nd_compress(x, off, p, s, 0, w, given_norms=gn)
        lv = levels[w].cpu().numpy()[:(d + 1) // 2]
        assert np.array_equal(lv, l1)
        cg = unpack_nibbles(lv, d).astype(np.int64)
        c0 = unpack_nibbles(l0, d).astype(np.int64)
        diff = cg != c0
        assert diff.sum() <= CODE_MISMATCH * d
        assert np.all(np.abs(cg - c0)[diff] == 1)
        refs.append((gn, lv, s0))
    # the aggregate of the planes the GPU wrote (they equal the given-norm oracle's, checked above)
    want = oracle.nd_aggregate([r[0] for r in refs], [r[1] for r in refs], [r[2] for r in refs],
                               off, s, d)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_unbiasedness_of_the_gpu_path_over_seeds():
    # E D(x) = x (Def. 3): average the decoded GPU output over many seeds
    rng = np.random.default_rng(9)
    d, s, trials = 2048, 4, 400
    x = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    off = [0, 700, d]
    off_dev = dev(np.asarray(off, np.uint64).view(np.int64))
    xdev = dev(x)
    ws_bytes = nc.nd_workspace_bytes(d, 2)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    norms = torch.empty(2, dtype=torch.float32, device="cuda")
    level = torch.empty(nc.nd_level_bytes(d), dtype=torch.uint8, device="cuda")
    sign = torch.empty(nc.nc_sign_bytes(d), dtype=torch.uint8, device="cuda")
    acc = torch.zeros(d, dtype=torch.float32, device="cuda")
    for t in range(trials):
        nc.nd_compress(xdev, d, off_dev, 2, 2, s, t, 0, norms, level, sign, ws, ws_bytes)
        nc.nd_decode_accumulate(norms, level, sign, d, off_dev, 2, s, acc)
    torch.cuda.synchronize()
    mean = acc.cpu().numpy().astype(np.float64) / trials
    nrm = norms.cpu().numpy().astype(np.float64)
    per = np.repeat(nrm, np.diff(off))
    # per-entry variance <= max(y (2^(1-s)) , y^2 / 8) * norm^2 <= norm^2 * 2^(1-s) * max(y, ...)
    sigma = per * np.sqrt(np.maximum(np.abs(x) / per * 2.0 ** (1 - s), (x / per) ** 2 / 8))
    assert np.all(np.abs(mean - x) <= 6 * sigma / np.sqrt(trials) + 1e-12)


def test_batch_launch_equals_single_launches():
    rng = np.random.default_rng(33)
    n, d, p, s = 5, 70001 + 96, 2, 8
    off = workloads.small_bucket_table(d, seed=3)
    B = len(off) - 1
    off_dev = dev(np.asarray(off, np.uint64).view(np.int64))
    xs = [(rng.standard_normal(d) * 10.0 ** rng.uniform(-4, -1)).astype(np.float32)
          for _ in range(n)]
    xd = [dev(x) for x in xs]
    workers = [7, 3, 0, 12, 5]
    norms = [Guarded(4 * B) for _ in range(n)]
    levels = [Guarded(nc.nd_level_bytes(d)) for _ in range(n)]
    signs = [Guarded(nc.nc_sign_bytes(d)) for _ in range(n)]
    ws_bytes = nc.nd_batch_workspace_bytes(d, B, n)
    ws = Guarded(ws_bytes)
    nc.nd_compress_batch(xd, d, off_dev, B, p, s, 11, workers, [g.buf for g in norms],
                         [g.buf for g in levels], [g.buf for g in signs], n, ws.buf, ws_bytes)
    torch.cuda.synchronize()
    for g in norms + levels + signs + [ws]:
        g.check()
    # the two halves as calls of their own give the same bytes (the rounding call finds the
    # bucket of each tile itself instead of reading the map the norm pass leaves behind)
    norms2 = [Guarded(4 * B) for _ in range(n)]
    levels2 = [Guarded(nc.nd_level_bytes(d)) for _ in range(n)]
    signs2 = [Guarded(nc.nc_sign_bytes(d)) for _ in range(n)]
    nc.nd_norms_batch(xd, d, off_dev, B, p, [g.buf for g in norms2], n, ws.buf, ws_bytes)
    ws.buf.fill_(0x5A)                       # the rounding call must not depend on the workspace
    nc.nd_round_batch(xd, d, off_dev, B, s, 11, workers, [g.buf for g in norms2],
                      [g.buf for g in levels2], [g.buf for g in signs2], n)
    torch.cuda.synchronize()
    for a, b in zip(norms + levels + signs, norms2 + levels2 + signs2):
        b.check()
        assert np.array_equal(a.numpy(np.uint8), b.numpy(np.uint8))
    for i in range(n):
        n1, l1, s1 = gpu_nd_compress(xd[i], off, p, s, 11, workers[i])
        assert np.array_equal(norms[i].numpy(np.uint32), n1.numpy(np.uint32))
        assert np.array_equal(levels[i].numpy(np.uint8), l1.numpy(np.uint8))
        assert np.array_equal(signs[i].numpy(np.uint32), s1.numpy(np.uint32))
        check_against_oracle(xs[i], off, p, s, 11, workers[i], norms[i], levels[i], signs[i])


def test_round_batch_against_norms_that_are_not_the_entries_own():
    """nd_round_batch rounds against whatever norms the caller gives (norms that were compressed
    and decoded again, combined partial norms).  Ratios above 1 and NaN ratios take the top
    level, degenerate norms give level 0; codes equal the given-norm oracle's bit for bit."""
    rng = np.random.default_rng(77)
    n, d, s = 3, 70001 + 2048, 8
    off = workloads.small_bucket_table(d, seed=12)
    B = len(off) - 1
    off_dev = dev(np.asarray(off, np.uint64).view(np.int64))
    xs = [(rng.standard_normal(d) * 1e-2).astype(np.float32) for _ in range(n)]
    xs[1][rng.choice(d, 50, replace=False)] = np.nan
    xs[2][rng.choice(d, 50, replace=False)] = np.inf
    workers = [4, 9, 2]
    given = []
    for i, x in enumerate(xs):
        own = oracle.norms(np.nan_to_num(x, nan=0.0, posinf=0.0), off, 2)
        g = own * (2.0 ** rng.integers(-6, 3, B)).astype(np.float32)   # far too small .. too large
        g[rng.choice(B, max(B // 10, 1), replace=False)] = [0.0, np.inf, np.nan][i]
        g[rng.choice(B, 2, replace=False)] = [-1.0, 1e-42]              # negative; subnormal
        given.append(g.astype(np.float32))
    norms = [dev(g) for g in given]
    levels = [Guarded(nc.nd_level_bytes(d)) for _ in range(n)]
    signs = [Guarded(nc.nc_sign_bytes(d)) for _ in range(n)]
    nc.nd_round_batch([dev(x) for x in xs], d, off_dev, B, s, 5, workers, norms,
                      [g.buf for g in levels], [g.buf for g in signs], n)
    torch.cuda.synchronize()
    for i in range(n):
        levels[i].check()
        signs[i].check()
        _, l_ref, s_ref = oracle.nd_compress(xs[i], off, 2, s, 5, workers[i], given_norms=given[i])
        assert np.array_equal(levels[i].numpy(np.uint8)[:(d + 1) // 2], l_ref), i
        assert np.array_equal(signs[i].numpy(np.uint32)[:(d + 31) // 32], s_ref), i
        c = unpack_nibbles(l_ref, d)
        assert np.any(c == s) and np.all(c <= s)


def test_one_element_buckets_and_many_empty_buckets():
    # every tile takes the multi-bucket path: B = d one-element buckets, then a table that is
    # mostly empty buckets
    rng = np.random.default_rng(55)
    d = 3000
    x = (rng.standard_normal(d) * 1e-2).astype(np.float32)
    x[7] = 0.0
    off = list(range(d + 1))
    for p in (2, 0):
        norms, level, sign = gpu_nd_compress(dev(x), off, p, 8, seed=4, worker=2)
        gn = check_against_oracle(x, off, p, 8, 4, 2, norms, level, sign)
        assert np.array_equal(gn, np.abs(x))            # a one-element bucket: norm = |x|
        c = unpack_nibbles(level.numpy(np.uint8), d)
        assert c[7] == 0 and np.all(c[np.abs(x) >= 2.0 ** -126] == 8)   # y = 1 exactly
    off2 = sorted([0] + list(rng.integers(0, d, 40)) * 3 + [d])
    norms, level, sign = gpu_nd_compress(dev(x), off2, 1, 4, seed=5, worker=0)
    check_against_oracle(x, off2, 1, 4, 5, 0, norms, level, sign)


def test_beyond_2_to_32_entries_sampled():
    # one vector of 2^32 + 2^21 + 13 entries (17 GB) in three buckets whose boundaries sit at odd
    # places around 2^31 and 2^32: 64-bit element indices in the norm pass, the rounding pass and
    # the aggregate.  Norms against float64 sums on the device data, level and sign planes on
    # sampled slices against the oracle (given the norm, slice offset as first element index).
    d = (1 << 32) + (1 << 21) + 13
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * (1 << 30):
        pytest.skip("needs ~50 GB of free device memory")
    p, s = 2, 8
    off = [0, (1 << 31) + 5, (1 << 32) + 1029, d]
    B = 3
    off_dev = dev(np.asarray(off, np.uint64).view(np.int64))
    x = torch.empty(d, dtype=torch.float32, device="cuda")
    g = torch.Generator(device="cuda")
    g.manual_seed(32)
    chunk = 1 << 28
    for a in range(0, d, chunk):
        x[a:min(d, a + chunk)].normal_(0.0, 1e-3, generator=g)
    ws_bytes = nc.nd_workspace_bytes(d, B)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    norms = torch.empty(B, dtype=torch.float32, device="cuda")
    level = torch.empty(nc.nd_level_bytes(d), dtype=torch.uint8, device="cuda")
    sign = torch.empty(nc.nc_sign_bytes(d), dtype=torch.uint8, device="cuda")
    nc.nd_compress(x, d, off_dev, B, p, s, 3, 1, norms, level, sign, ws, ws_bytes)
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nd_aggregate([norms], [level], [sign], 1, d, off_dev, B, s, out)
    torch.cuda.synchronize()
    gn = norms.cpu().numpy()
    for b in range(B):
        sq = 0.0
        for a in range(off[b], off[b + 1], chunk):
            sq += float((x[a:min(off[b + 1], a + chunk)].double() ** 2).sum())
        assert abs(float(gn[b]) - sq ** 0.5) <= NORM_RTOL * sq ** 0.5
    length = 4096
    # (slice start, bucket): inside each bucket, on both sides of 2^32, and the ragged tail
    picks = [(0, 0), ((1 << 31) - 4096, 0), ((1 << 31) + 32, 1), ((1 << 32) - 4096, 1),
             ((1 << 32), 1), ((1 << 32) + 2048, 2), (((d - length) // 32) * 32, 2)]
    for o, b in picks:
        hi = min(d, o + length, off[b + 1])
        assert off[b] <= o and hi <= off[b + 1]
        xs = x[o:hi].cpu().numpy()
        _, l_ref, s_ref = oracle.nd_compress(xs, [0, hi - o], p, s, 3, 1, given_norms=gn[b:b + 1],
                                             j0=o)
        m = hi - o                                  # a slice may end inside a byte / sign word
        lv = level[o // 2:(hi + 1) // 2].cpu().numpy()
        assert np.array_equal(unpack_nibbles(lv, m), unpack_nibbles(l_ref, m)), o
        sw = sign.view(torch.int32)[o // 32:(hi + 31) // 32].cpu().numpy().view(np.uint32)
        k = np.arange(m)
        assert np.array_equal((sw[k // 32] >> (k % 32)) & 1, (s_ref[k // 32] >> (k % 32)) & 1), o
        want = oracle.nd_aggregate([gn[b:b + 1]], [l_ref], [s_ref], [0, hi - o], s, hi - o)
        assert np.array_equal(out[o:hi].cpu().numpy().view(np.uint32), want.view(np.uint32)), o
    del x, level, sign, out, ws
    torch.cuda.empty_cache()
