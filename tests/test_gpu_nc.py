"""GPU parity, natural compression and aggregation: the CUDA library against the CPU oracle,
element by element on the same seeded inputs.  Integer / bit work is compared bit-exactly."""
import numpy as np
import pytest
import torch

import oracle
import paper_1905_10988_b200 as nc
from paper_1905_10988_b200 import workloads
from gpu_util import Guarded, check_nc_planes, dev, gpu_nc_compress, special_values

pytestmark = pytest.mark.gpu

SIZES = [1, 3, 4, 31, 32, 33, 127, 128, 129, 1023, 1024, 1025, 4095, 4097, 8192 + 17,
         (1 << 20) - 1, (1 << 20) + 1]


@pytest.mark.parametrize("d", SIZES)
def test_compress_matches_oracle_over_sizes(d):
    rng = np.random.default_rng(d)
    x = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    if d >= 32:
        sp = special_values(rng, d // 8)
        x[rng.choice(d, sp.size, replace=False)] = sp
    seed, worker = 0xABCDEF0123456789 ^ d, d % 7
    e, s = gpu_nc_compress(dev(x), seed, worker)
    e_ref, s_ref = oracle.nc_compress(x, seed, worker)
    check_nc_planes(e, s, d, e_ref, s_ref)


def test_compress_every_exponent_sign_and_boundary_mantissa():
    # every sign x exponent with mantissas {0, 1, 2^22, 2^23-1} and 60 random ones
    rng = np.random.default_rng(1)
    mant = np.concatenate([np.uint32([0, 1, 1 << 22, (1 << 23) - 1]),
                           rng.integers(0, 1 << 23, 60, dtype=np.uint64).astype(np.uint32)])
    expo = np.arange(256, dtype=np.uint32)
    bits = ((np.arange(2, dtype=np.uint32)[:, None, None] << 31) | (expo[None, :, None] << 23)
            | mant[None, None, :]).ravel()
    x = bits.view(np.float32)
    for seed in (0, 1, 0xFFFFFFFFFFFFFFFF):
        e, s = gpu_nc_compress(dev(x), seed, 3)
        e_ref, s_ref = oracle.nc_compress(x, seed, 3)
        check_nc_planes(e, s, x.size, e_ref, s_ref)


def test_compress_random_bit_patterns():
    rng = np.random.default_rng(2)
    d = (1 << 22) + 5
    x = rng.integers(0, 1 << 32, d, dtype=np.uint64).astype(np.uint32).view(np.float32)
    e, s = gpu_nc_compress(dev(x), 99, 0)
    e_ref, s_ref = oracle.nc_compress(x, 99, 0)
    check_nc_planes(e, s, d, e_ref, s_ref)


def test_compress_all_2_to_32_bit_patterns():
    """Every binary32 bit pattern once, as one vector of 2^32 entries (element j holds the pattern
    j xor 2^31), in two sweeps with different streams: closes every sign / exponent / mantissa
    corner of the field rule (Sec. 2), of the kernel's unguarded fast path and of the edge
    policy.  Compared with the oracle chunk by chunk."""
    d = 1 << 32
    free, _ = torch.cuda.mem_get_info()
    if free < 30 * (1 << 30):
        pytest.skip("needs ~22 GB of free device memory")
    x = torch.arange(-(1 << 31), 1 << 31, dtype=torch.int32, device="cuda").view(torch.float32)
    e = torch.empty(nc.nc_exp_bytes(d), dtype=torch.uint8, device="cuda")
    s = torch.empty(nc.nc_sign_bytes(d), dtype=torch.uint8, device="cuda")
    chunk = 1 << 27
    for seed, worker in ((0, 0), ((1 << 63) + 5, 0xFFFFFFFF)):
        e.fill_(0xEE)
        s.fill_(0xEE)
        nc.nc_compress(x, d, seed, worker, e, s)
        torch.cuda.synchronize()
        for j0 in range(0, d, chunk):
            xs = x[j0:j0 + chunk].cpu().numpy()
            e_ref, s_ref = oracle.nc_compress(xs, seed, worker, j0=j0)
            assert np.array_equal(e[j0:j0 + chunk].cpu().numpy(), e_ref), (seed, j0)
            got = s[j0 // 8:(j0 + chunk) // 8].cpu().numpy().view(np.uint32)
            assert np.array_equal(got, s_ref), (seed, j0)
    del x, e, s
    torch.cuda.empty_cache()


def _aggregate_gpu(exps, signs, d):
    out = Guarded(4 * d)
    nc.nc_aggregate(exps, signs, len(exps), d, out.buf)
    torch.cuda.synchronize()
    out.check()
    return out.numpy(np.float32)


def test_config1_compress_and_aggregate():
    n, d = 4, 1 << 20
    xs = [workloads.config1_vector(w, d) for w in range(n)]
    xd = [x.cuda() for x in xs]
    es = [torch.empty(nc.nc_exp_bytes(d), dtype=torch.uint8, device="cuda") for _ in range(n)]
    ss = [torch.empty(nc.nc_sign_bytes(d), dtype=torch.uint8, device="cuda") for _ in range(n)]
    nc.nc_compress_batch(xd, d, 0, list(range(n)), es, ss, n)
    got = _aggregate_gpu(es, ss, d)
    refs = [oracle.nc_compress(x.numpy(), 0, w) for w, x in enumerate(xs)]
    for w in range(n):
        assert np.array_equal(es[w].cpu().numpy()[:d], refs[w][0])
        assert np.array_equal(ss[w].cpu().numpy().view(np.uint32)[:d // 32], refs[w][1])
    want = oracle.nc_aggregate([r[0] for r in refs], [r[1] for r in refs], d)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # the batch launch and single launches agree
    e1, s1 = gpu_nc_compress(xd[2], 0, 2)
    assert np.array_equal(e1.numpy(np.uint8), es[2].cpu().numpy())
    assert np.array_equal(s1.numpy(np.uint8), ss[2].cpu().numpy())


@pytest.mark.parametrize("n,d", [(1, 1000), (2, 1024), (3, 5000), (8, 4097), (16, 70001),
                                 (64, 2048 + 3)])
def test_aggregate_random_codes_and_identity_with_decode_accumulate(n, d):
    rng = np.random.default_rng(n * 1000 + d)
    exps = [rng.integers(0, 256, nc.nc_exp_bytes(d)).astype(np.uint8) for _ in range(n)]
    for e in exps:                       # mostly moderate exponents, some 0 / 254 / 255
        body = rng.integers(100, 150, e.size).astype(np.uint8)
        keep = rng.random(e.size) < 0.9
        e[keep] = body[keep]
    signs = [rng.integers(0, 1 << 32, nc.nc_sign_bytes(d) // 4, dtype=np.uint64)
             .astype(np.uint32) for _ in range(n)]
    ed = [dev(e) for e in exps]
    sd = [dev(s) for s in signs]
    got = _aggregate_gpu(ed, sd, d)
    want = oracle.nc_aggregate([e[:d] for e in exps], signs, d)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # zero-fill + n x decode_accumulate, worker order
    acc = Guarded(4 * d)
    acc.buf.zero_()
    for i in range(n):
        nc.nc_decode_accumulate(ed[i], sd[i], d, acc.buf)
    torch.cuda.synchronize()
    acc.check()
    assert np.array_equal(acc.numpy(np.uint32), want.view(np.uint32))


def test_decode_accumulate_adds_to_existing_values():
    rng = np.random.default_rng(4)
    d = 3000
    x = (rng.standard_normal(d) * 0.1).astype(np.float32)
    e_ref, s_ref = oracle.nc_compress(x, 5, 1)
    start = rng.standard_normal(d).astype(np.float32)
    acc = Guarded(4 * d)
    acc.buf.copy_(dev(start).view(torch.uint8))
    e = np.zeros(nc.nc_exp_bytes(d), np.uint8)
    e[:d] = e_ref
    s = np.zeros(nc.nc_sign_bytes(d) // 4, np.uint32)
    s[:s_ref.size] = s_ref
    nc.nc_decode_accumulate(dev(e), dev(s), d, acc.buf)
    torch.cuda.synchronize()
    acc.check()
    want = start.copy()
    oracle.nc_decode_accumulate(e_ref, s_ref, want)
    assert np.array_equal(acc.numpy(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("n,d", [(1, 77), (4, 1 << 16), (16, 40000 + 3)])
def test_sum_fp32_reference_point(n, d):
    rng = np.random.default_rng(n + d)
    xs = [(rng.standard_normal(d) * 10.0 ** rng.integers(-5, 3)).astype(np.float32)
          for _ in range(n)]
    out = Guarded(4 * d)
    nc.nc_sum_fp32([dev(x) for x in xs], n, d, out.buf)
    torch.cuda.synchronize()
    out.check()
    assert np.array_equal(out.numpy(np.uint32), oracle.sum_fp32(xs).view(np.uint32))


def _sample_offsets(rng, d, count, length):
    offs = (rng.integers(0, (d - length) // 1024, count) * 1024).tolist()
    offs += [0, ((d - length) // 32) * 32]          # head and the ragged tail
    return sorted(set(int(o) for o in offs))


def test_config2_full_size_sampled():
    # the launch configuration the benchmark times: 8 workers, d = 25,557,032, one batch launch
    n = 8
    sizes = workloads.resnet50_tensor_sizes()
    d = sum(sizes)
    xd = [workloads.config2_vector(w, "cuda", sizes) for w in range(n)]
    es = [torch.empty(nc.nc_exp_bytes(d), dtype=torch.uint8, device="cuda") for _ in range(n)]
    ss = [torch.empty(nc.nc_sign_bytes(d), dtype=torch.uint8, device="cuda") for _ in range(n)]
    nc.nc_compress_batch(xd, d, 0, list(range(n)), es, ss, n)
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nc_aggregate(es, ss, n, d, out)
    torch.cuda.synchronize()
    rng = np.random.default_rng(0)
    length = 4096
    for o in _sample_offsets(rng, d, 24, length):
        hi = min(d, o + length) if o + length < d - 64 else d
        refs = []
        for w in range(n):
            xw = xd[w][o:hi].cpu().numpy()
            e_ref, s_ref = oracle.nc_compress(xw, 0, w, j0=o)
            assert np.array_equal(es[w][o:hi].cpu().numpy(), e_ref)
            sw = ss[w].view(torch.int32)[o // 32:(hi + 31) // 32].cpu().numpy().view(np.uint32)
            assert np.array_equal(sw, s_ref)
            refs.append((e_ref, s_ref))
        want = oracle.nc_aggregate([r[0] for r in refs], [r[1] for r in refs], hi - o)
        assert np.array_equal(out[o:hi].cpu().numpy().view(np.uint32), want.view(np.uint32))
    # properties that hold at any size: signs are the input's sign bits, exponent moves by 0 or 1
    for w in (0, n - 1):
        bits = xd[w].view(torch.int32)
        ex_in = (bits >> 23) & 0xFF
        diff = es[w][:d].to(torch.int32) - ex_in
        assert int(diff.min()) >= 0 and int(diff.max()) <= 1


def test_config4_full_size_sampled():
    # d = 335,141,888, n = 16 (21 GB of inputs): sampled slices, worker by worker
    n = 16
    d = sum(workloads.bert_large_bucket_sizes())
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs ~32 GB of free device memory")
    xd = [workloads.config4_vector(w, d, "cuda") for w in range(n)]
    es = [torch.empty(nc.nc_exp_bytes(d), dtype=torch.uint8, device="cuda") for _ in range(n)]
    ss = [torch.empty(nc.nc_sign_bytes(d), dtype=torch.uint8, device="cuda") for _ in range(n)]
    nc.nc_compress_batch(xd, d, 0, list(range(n)), es, ss, n)
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nc_aggregate(es, ss, n, d, out)
    ref_sum = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nc_sum_fp32(xd, n, d, ref_sum)
    torch.cuda.synchronize()
    rng = np.random.default_rng(4)
    length = 2048
    for o in _sample_offsets(rng, d, 12, length):
        hi = min(d, o + length)
        refs = []
        for w in range(n):
            e_ref, s_ref = oracle.nc_compress(xd[w][o:hi].cpu().numpy(), 0, w, j0=o)
            assert np.array_equal(es[w][o:hi].cpu().numpy(), e_ref)
            sw = ss[w].view(torch.int32)[o // 32:(hi + 31) // 32].cpu().numpy().view(np.uint32)
            assert np.array_equal(sw, s_ref)
            refs.append((e_ref, s_ref))
        want = oracle.nc_aggregate([r[0] for r in refs], [r[1] for r in refs], hi - o)
        assert np.array_equal(out[o:hi].cpu().numpy().view(np.uint32), want.view(np.uint32))
        want_sum = oracle.sum_fp32([xd[w][o:hi].cpu().numpy() for w in range(n)])
        assert np.array_equal(ref_sum[o:hi].cpu().numpy().view(np.uint32),
                              want_sum.view(np.uint32))
    # unbiasedness at scale: the compressed sum tracks the exact sum within the variance bound
    # E||sum_i C(x_i) - sum_i x_i||^2 <= (1/8) sum_i ||x_i||^2 (Thm. 1, independent workers)
    err2 = float(((out.double() - ref_sum.double()) ** 2).sum())
    x2 = sum(float((x.double() ** 2).sum()) for x in xd)
    assert err2 <= x2 / 8 * 1.02
    assert err2 >= x2 / 8 * 0.3


def test_beyond_2_to_34_entries_sampled():
    # one vector of 2^34 + 2^20 + 77 entries (69 GB): tile bases above 2^32 (64-bit addressing)
    # and above 2^34, where the high word of the generator's counter becomes non-zero; sampled
    # slices against the oracle, which takes the offset of a slice as its first element index
    d = (1 << 34) + (1 << 20) + 77
    free, _ = torch.cuda.mem_get_info()
    if free < 110 * (1 << 30):
        pytest.skip("needs ~90 GB of free device memory")
    x = torch.empty(d, dtype=torch.float32, device="cuda")
    g = torch.Generator(device="cuda")
    g.manual_seed(34)
    chunk = 1 << 28
    for a in range(0, d, chunk):
        x[a:min(d, a + chunk)].normal_(0.0, 1e-3, generator=g)
    e = torch.empty(nc.nc_exp_bytes(d), dtype=torch.uint8, device="cuda")
    s = torch.empty(nc.nc_sign_bytes(d), dtype=torch.uint8, device="cuda")
    nc.nc_compress(x, d, 5, 9, e, s)
    torch.cuda.synchronize()
    length = 4096
    offs = [0, (1 << 32) - 2048, (1 << 32), (1 << 33) + 1024 * 777, (1 << 34) - 2048, (1 << 34),
            (1 << 34) + 1024 * 500, ((d - length) // 32) * 32]
    for o in offs:
        hi = min(d, o + length)
        e_ref, s_ref = oracle.nc_compress(x[o:hi].cpu().numpy(), 5, 9, j0=o)
        assert np.array_equal(e[o:hi].cpu().numpy(), e_ref), o
        sw = s.view(torch.int32)[o // 32:(hi + 31) // 32].cpu().numpy().view(np.uint32)
        assert np.array_equal(sw, s_ref), o
    # the two sides of 2^34 draw from different counter blocks: same inputs, different rounding
    a = e[(1 << 34) - 4096:(1 << 34)].cpu().numpy()
    b = e[(1 << 34):(1 << 34) + 4096].cpu().numpy()
    assert not np.array_equal(a, b)
    del x, e, s
    torch.cuda.empty_cache()
