"""C_nat of binary64 vectors (11-bit exponent + sign = 12-bit codes): oracle pins on CPU, GPU
parity (bit-exact) through the C ABI."""
import numpy as np
import pytest

import oracle


def _codes(exp_lo, hi, d):
    j = np.arange(d)
    nib = (hi[j // 2] >> (4 * (j % 2))) & 0xF
    return ((nib & 7).astype(np.int64) << 8) | exp_lo[:d], nib >> 3


def test_field_rule_of_sec2_equals_the_real_valued_definition():
    # Sec. 2: exponent e with probability 1 - m, e + 1 with probability m.  With the 52-bit
    # threshold that is "up iff r52 < mantissa field"; the oracle evaluates Def. 1 on real numbers.
    rng = np.random.default_rng(0)
    d = 200_000
    x = rng.standard_normal(d) * 10.0 ** rng.uniform(-300, 300, d)
    x[:8] = [0.0, -0.0, np.inf, -np.inf, np.nan, 5e-324, -1.5e-310, 1.7e308]
    exp_lo, hi = oracle.nc64_compress(x, 9, 4)
    e11, sgn = _codes(exp_lo, hi, d)
    bits = x.view(np.uint64)
    field = ((bits >> np.uint64(52)) & np.uint64(0x7FF)).astype(np.int64)
    mant = bits & np.uint64((1 << 52) - 1)
    w0 = oracle.stream_words(9, 4, 0, 0, d).astype(np.uint64)
    w3 = oracle.stream_words(9, 4, 3, 0, d).astype(np.uint64)
    r52 = ((w0 & np.uint64(0x7FFFFF)) << np.uint64(29)) | (w3 >> np.uint64(3))
    up = (r52 < mant) & (field < 2046)
    want = field + up
    want[field == 2047] = 2047
    assert np.array_equal(e11, want)
    assert np.array_equal(sgn, (bits >> np.uint64(63)).astype(np.uint8))


def test_binary32_representable_inputs_round_like_the_binary32_operator():
    # for such t the 52-bit rule reduces to "r23 < 23-bit mantissa" on the same domain-0 word
    rng = np.random.default_rng(1)
    x32 = (rng.standard_normal(50_000) * 10.0 ** rng.uniform(-30, 30, 50_000)).astype(np.float32)
    x32[:3] = [2.5, -2.75, 0.75]
    exp_lo, hi = oracle.nc64_compress(x32.astype(np.float64), 5, 1)
    e11, sgn = _codes(exp_lo, hi, x32.size)
    e8, s32 = oracle.nc_compress(x32, 5, 1)
    normal = np.abs(x32) >= np.float32(2.0 ** -126)
    assert np.array_equal(e11[normal] - 1023, e8[normal].astype(np.int64) - 127)
    j = np.arange(x32.size)
    assert np.array_equal(sgn, (s32[j // 32] >> (j % 32)) & 1)


def test_unbiased_and_second_moment_bound_on_long_mantissas():
    # E C(t) = t and E C(t)^2 <= 9/8 t^2 (Thm. 1) for doubles whose mantissa needs all 52 bits
    rng = np.random.default_rng(2)
    t = np.array([np.pi, -np.e * 1e-200, 4 / 3, 1 + 2.0 ** -30])
    n = 400_000
    r52 = rng.integers(0, 1 << 52, n, dtype=np.uint64)
    for v in t:
        c = oracle.cnat64_values(np.full(n, v), r52)
        lo = 2.0 ** np.floor(np.log2(abs(v)))
        assert set(np.unique(np.abs(c))) <= {lo, 2 * lo}
        p_up = (abs(v) - lo) / lo
        assert abs((np.abs(c) == 2 * lo).mean() - p_up) < 5 * np.sqrt(max(p_up * (1 - p_up), 1e-12) / n) + 1e-9
        assert (c.astype(np.float64) ** 2).mean() <= 9 / 8 * v * v * (1 + 1e-2)
    # the threshold is exact at both ends: r52 = M - 1 goes up, r52 = M stays
    v = 1 + 2.0 ** -52 * 12345
    assert oracle.cnat64_values([v, v], np.uint64([12344, 12345])).tolist() == [2.0, 1.0]


def test_aggregate_is_the_ordered_binary64_sum():
    rng = np.random.default_rng(3)
    n, d = 5, 10_001
    xs = [rng.standard_normal(d) * 10.0 ** rng.uniform(-5, 5, d) for _ in range(n)]
    planes = [oracle.nc64_compress(x, 2, w) for w, x in enumerate(xs)]
    out = oracle.nc64_aggregate([p[0] for p in planes], [p[1] for p in planes], d)
    ref = np.zeros(d)
    for e, h in planes:
        e11, sgn = _codes(e, h, d)
        val = np.where(e11 == 0, 0.0, np.ldexp(1.0, (e11 - 1023).astype(np.int32)))
        ref = ref + np.where(sgn == 1, -val, val)
    assert np.array_equal(out, ref)
    assert np.all(np.abs(out - np.sum(xs, axis=0)) <= np.sum(np.abs(xs), axis=0))


# ------------------------------------------------------------------------------- GPU parity
@pytest.mark.gpu
@pytest.mark.parametrize("d", [1, 2, 31, 1024, 1025, 4097, (1 << 20) + 7])
def test_gpu_nc64_compress_matches_oracle(d):
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import Guarded, dev
    rng = np.random.default_rng(d)
    x = rng.standard_normal(d) * 10.0 ** rng.uniform(-300, 300, d)
    if d >= 31:
        sp = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, 5e-324, -1.5e-310, 1.7e308, -1.0, 2.0 ** -1022])
        x[rng.choice(d, sp.size, replace=False)] = sp
    e = Guarded(nc.nc_exp_bytes(d))
    h = Guarded(nc.nd_level_bytes(d))
    nc.nc64_compress(dev(x), d, 3, 8, e.buf, h.buf)
    torch.cuda.synchronize()
    e.check()
    h.check()
    e_ref, h_ref = oracle.nc64_compress(x, 3, 8)
    ge, gh = e.numpy(np.uint8), h.numpy(np.uint8)
    assert np.array_equal(ge[:d], e_ref) and np.all(ge[d:] == 0)
    assert np.array_equal(gh[:h_ref.size], h_ref) and np.all(gh[h_ref.size:] == 0)


@pytest.mark.gpu
@pytest.mark.parametrize("n,d", [(1, 9), (4, 4096), (8, 70_001), (16, 3000)])
def test_gpu_nc64_batch_and_aggregate_match_oracle(n, d):
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import Guarded, dev
    rng = np.random.default_rng(n + d)
    xs = [rng.standard_normal(d) * 10.0 ** rng.uniform(-8, 8, d) for _ in range(n)]
    for x in xs:
        x[rng.choice(d, max(d // 50, 1), replace=False)] = 0.0
    if d > 100:
        xs[0][5], xs[n - 1][5] = np.inf, -np.inf          # inf - inf: a NaN column
    es = [Guarded(nc.nc_exp_bytes(d)) for _ in range(n)]
    hs = [Guarded(nc.nd_level_bytes(d)) for _ in range(n)]
    workers = list(range(10, 10 + n))
    nc.nc64_compress_batch([dev(x) for x in xs], d, 6, workers, [g.buf for g in es],
                           [g.buf for g in hs], n)
    out = Guarded(8 * d)
    nc.nc64_aggregate([g.buf for g in es], [g.buf for g in hs], n, d, out.buf)
    torch.cuda.synchronize()
    for g in es + hs + [out]:
        g.check()
    refs = [oracle.nc64_compress(x, 6, w) for x, w in zip(xs, workers)]
    for g, r in zip(es, refs):
        assert np.array_equal(g.numpy(np.uint8)[:d], r[0])
    for g, r in zip(hs, refs):
        assert np.array_equal(g.numpy(np.uint8)[:r[1].size], r[1])
    want = oracle.nc64_aggregate([r[0] for r in refs], [r[1] for r in refs], d)
    got = out.numpy(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint64), want[~nan].view(np.uint64))
