"""The paper's 8-bit wire format (sign, zero flag, exponent clipped to -50..10) and the integer
aggregation of its aggregator: oracle pins on CPU, GPU parity (bit-exact) through the C ABI."""
import numpy as np
import pytest

import oracle


def test_code8_layout_clipping_and_relation_to_the_nine_bit_code():
    x = np.float32([2.5, -0.75, 0.0, -0.0, 1e-20, 3000.0, np.inf, -np.inf, 2.0 ** -50,
                    2.0 ** 10, -2.0 ** 11])
    c = oracle.nc8_compress(x, 3, 1)
    e9, s9 = oracle.nc_compress(x, 3, 1)                       # same stream, 9-bit code
    for j in range(x.size):
        sign, zero, e6 = c[j] >> 7, (c[j] >> 6) & 1, c[j] & 0x3F
        assert sign == (s9[0] >> j) & 1
        if e9[j] == 0:
            assert zero == 1 and e6 == 0
        else:
            assert zero == 0 and e6 == min(max(int(e9[j]) - 127, -50), 10) + 50
    dec = oracle.nc8_decode(c)
    assert dec[4] == 2.0 ** -50 and dec[5] == 1024 and dec[6] == 1024 and dec[7] == -1024
    assert dec[2] == 0 and dec[3] == 0 and dec[10] == -1024
    # inside the clip range the 8-bit and 9-bit codes decode to the same values
    rng = np.random.default_rng(0)
    y = (rng.standard_normal(50_000) * 10.0 ** rng.uniform(-9, 2, 50_000)).astype(np.float32)
    y = y[(np.abs(y) > 2.0 ** -49) & (np.abs(y) < 2.0 ** 9)]
    c = oracle.nc8_compress(y, 5, 2)
    e9, s9 = oracle.nc_compress(y, 5, 2)
    j = np.arange(y.size)
    ref = oracle.cnat_decode(e9, ((s9[j // 32] >> (j % 32)) & 1).astype(np.uint8))
    assert np.array_equal(oracle.nc8_decode(c), ref)


def test_integer_aggregation_is_exact_and_order_independent():
    rng = np.random.default_rng(1)
    n, d = 7, 20_000
    codes = [rng.integers(0, 256, d).astype(np.uint8) for _ in range(n)]
    for c in codes:
        c[(c & 0x3F) > 60] &= 0xC0 | 60                       # exponent field at most 60
    out, sums = oracle.nc8_aggregate(codes, d)
    # python integers: exact reference
    want = np.zeros(d, dtype=object)
    for c in codes:
        v = np.where(c & 0x40, 0, 1 << (c & 0x3F).astype(object))
        want = want + np.where(c & 0x80, -v, v)
    assert all(int(a) == int(b) for a, b in zip(sums[:2000], want[:2000]))
    # fl32(sum) with a single rounding (x87 long double holds any |sum| < 2^63 exactly)
    assert np.finfo(np.longdouble).nmant >= 63
    one_rounding = sums.astype(np.longdouble).astype(np.float32) * np.float32(2.0 ** -50)
    assert np.array_equal(out.view(np.uint32), one_rounding.view(np.uint32))
    perm = rng.permutation(n)
    out2, sums2 = oracle.nc8_aggregate([codes[i] for i in perm], d)
    assert np.array_equal(sums, sums2) and np.array_equal(out.view(np.uint32), out2.view(np.uint32))
    # unlike the fp32 sum: (2^10 + 2^-50) - 2^10 keeps the small term
    a = [np.uint8([60]), np.uint8([0]), np.uint8([0x80 | 60])]
    assert oracle.nc8_aggregate(a, 1)[0][0] == np.float32(2.0 ** -50)


def test_master_compression_of_the_integer_sum_is_unbiased():
    # S = 2^e (1 + f): up with probability f (truncated to 23 bits); check by exhaustive counting
    # over many coordinates (each coordinate has its own stream word)
    d = 1 << 18
    for ints in ([1 << 20, 1 << 19], [1 << 30, 1 << 29, 1 << 28], [2, 1], [1 << 40, -(1 << 38)]):
        codes = []
        for v in ints:
            c = np.uint8((0x80 if v < 0 else 0) | (abs(v).bit_length() - 1))
            codes.append(np.full(d, c, np.uint8))
        s = sum(ints)
        out = oracle.nc8_aggregate_compress(codes, d, 11, 0xFFFFFFFF)
        dec = oracle.nc8_decode(out).astype(np.float64) * 2.0 ** 50
        e = abs(s).bit_length() - 1
        assert set(np.unique(dec)) <= {float(2 ** e), float(2 ** (e + 1))}
        p_up = (abs(s) - 2 ** e) / 2 ** e
        got = float((dec == 2 ** (e + 1)).mean())
        assert abs(got - p_up) <= 4 * np.sqrt(max(p_up * (1 - p_up), 1e-9) / d) + 2.0 ** -23
        # draw for draw it is the threshold rule on the C_nat stream of the master
        r23 = oracle.stream_words(11, 0xFFFFFFFF, 0, 0, d) & 0x7FFFFF
        thr = ((abs(s) - 2 ** e) << 23) >> e
        assert np.array_equal(dec == 2 ** (e + 1), r23 < thr)
    zero = oracle.nc8_aggregate_compress([np.uint8([5]), np.uint8([0x85])], 1, 0, 0)
    assert zero[0] == 0x40


# ------------------------------------------------------------------------------- GPU parity
@pytest.mark.gpu
@pytest.mark.parametrize("d", [1, 3, 33, 1024, 4097, (1 << 20) + 5])
def test_gpu_nc8_compress_matches_oracle(d):
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import Guarded, dev, special_values
    rng = np.random.default_rng(d)
    x = (rng.standard_normal(d) * 10.0 ** rng.uniform(-20, 5, d)).astype(np.float32)
    if d >= 32:
        sp = special_values(rng, d // 8)
        x[rng.choice(d, sp.size, replace=False)] = sp
    code = Guarded(nc.nc_exp_bytes(d))
    nc.nc8_compress(dev(x), d, 21, 4, code.buf)
    torch.cuda.synchronize()
    code.check()
    got = code.numpy(np.uint8)
    assert np.array_equal(got[:d], oracle.nc8_compress(x, 21, 4))
    assert np.all(got[d:] == 0)


@pytest.mark.gpu
@pytest.mark.parametrize("n,d", [(1, 7), (4, 4096), (7, 70001), (16, 5000), (64, 1030)])
def test_gpu_nc8_aggregate_and_master_compress_match_oracle(n, d):
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import Guarded, dev
    rng = np.random.default_rng(n * 17 + d)
    codes = []
    for _ in range(n):
        c = rng.integers(0, 256, nc.nc_exp_bytes(d)).astype(np.uint8)
        top = 60 if n <= 7 else 50                 # keep |sum| < 2^63 for the larger n
        e6 = np.minimum(c & 0x3F, top).astype(np.uint8)
        codes.append(((c & 0xC0) | e6).astype(np.uint8))
    cd = [dev(c) for c in codes]
    out = Guarded(4 * d)
    nc.nc8_aggregate(cd, n, d, out.buf)
    oc = Guarded(nc.nc_exp_bytes(d))
    nc.nc8_aggregate_compress(cd, n, d, 9, 0xFFFFFFFF, oc.buf)
    torch.cuda.synchronize()
    out.check()
    oc.check()
    want, _ = oracle.nc8_aggregate([c[:d] for c in codes], d)
    assert np.array_equal(out.numpy(np.uint32), want.view(np.uint32))
    want_c = oracle.nc8_aggregate_compress([c[:d] for c in codes], d, 9, 0xFFFFFFFF)
    got_c = oc.numpy(np.uint8)
    assert np.array_equal(got_c[:d], want_c) and np.all(got_c[d:] == 0)


@pytest.mark.gpu
def test_gpu_nc8_round_trip_on_config1():
    import torch
    import paper_1905_10988_b200 as nc
    from paper_1905_10988_b200 import workloads
    n, d = 4, 1 << 20
    xs = [workloads.config1_vector(w, d) for w in range(n)]
    xd = [x.cuda() for x in xs]
    codes = [torch.empty(nc.nc_exp_bytes(d), dtype=torch.uint8, device="cuda") for _ in range(n)]
    nc.nc8_compress_batch(xd, d, 0, list(range(n)), codes, n)
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nc8_aggregate(codes, n, d, out)
    torch.cuda.synchronize()
    refs = [oracle.nc8_compress(x.numpy(), 0, w) for w, x in enumerate(xs)]
    for w in range(n):
        assert np.array_equal(codes[w].cpu().numpy()[:d], refs[w])
    want, _ = oracle.nc8_aggregate(refs, d)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want.view(np.uint32))
    # all entries of this workload lie inside the clip range, so the integer sum equals the exact
    # real sum of the workers' rounded values
    exact = np.sum([oracle.nc8_decode(r).astype(np.float64) for r in refs], axis=0)
    assert np.array_equal(want.astype(np.float64), exact.astype(np.float32).astype(np.float64))
