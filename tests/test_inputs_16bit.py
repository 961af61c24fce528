"""C_nat of bfloat16 / binary16 inputs: oracle pins on CPU, GPU parity (bit-exact) through the ABI."""
import numpy as np
import pytest

import oracle

BF16, F16 = oracle.DTYPE_BF16, oracle.DTYPE_F16


def _all_patterns():
    return np.arange(1 << 16, dtype=np.uint32).astype(np.uint16)


def test_every_16bit_pattern_decodes_as_numpy_does():
    h = _all_patterns()
    got = oracle.values_of_16bit(h, F16)
    want = h.view(np.float16).astype(np.float32)
    assert np.array_equal(got.view(np.uint32)[~np.isnan(want)], want.view(np.uint32)[~np.isnan(want)])
    assert np.all(np.isnan(got[np.isnan(want)]))
    got = oracle.values_of_16bit(h, BF16)
    want = (h.astype(np.uint32) << 16).view(np.float32)
    ok = ~np.isnan(want)
    assert np.array_equal(got.view(np.uint32)[ok], want.view(np.uint32)[ok])
    assert np.all(np.isnan(got[~ok]))


def test_typed_compress_is_the_binary32_operator_on_the_converted_value():
    h = _all_patterns()
    for dtype in (BF16, F16):
        e, s = oracle.nc_compress_typed(h, dtype, 5, 2)
        e32, s32 = oracle.nc_compress(oracle.values_of_16bit(h, dtype), 5, 2)
        assert np.array_equal(e, e32) and np.array_equal(s, s32)


def test_up_probability_is_the_short_mantissa_fraction():
    # bfloat16 1.0 + 37/128 and binary16 (1 + 300/1024) * 2^-3, binary16 subnormal 77 * 2^-24:
    # count the thresholds r23 that round up, over all 2^23 of them
    r = np.arange(1 << 23, dtype=np.uint32)
    for dtype, pattern, lo, frac in [(BF16, 0x3F80 | 37, 1.0, 37 / 128),
                                     (F16, (12 << 10) | 300, 2.0 ** -3, 300 / 1024),
                                     (F16, 77, 2.0 ** -18, (77 - 64) / 64)]:
        t = oracle.values_of_16bit(np.uint16([pattern]), dtype)[0]
        vals = oracle.cnat_values(np.full(r.size, t, np.float32), r)
        assert set(np.unique(vals)) == {np.float32(lo), np.float32(2 * lo)}
        assert int((vals == np.float32(2 * lo)).sum()) == round(frac * (1 << 23))


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [BF16, F16])
@pytest.mark.parametrize("d", [1, 5, 1024, 4097, 65536, (1 << 20) + 33])
def test_gpu_typed_compress_matches_oracle(dtype, d):
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import Guarded, check_nc_planes, dev
    rng = np.random.default_rng(d + dtype)
    if d == 65536:
        h = _all_patterns()                       # every pattern, specials included
    else:
        x = (rng.standard_normal(d) * 10.0 ** rng.uniform(-6, 3, d)).astype(np.float32)
        if dtype == F16:
            h = x.astype(np.float16).view(np.uint16)
        else:
            h = (x.view(np.uint32) >> 16).astype(np.uint16)
    e = Guarded(nc.nc_exp_bytes(d))
    s = Guarded(nc.nc_sign_bytes(d))
    nc.nc_compress_typed(dev(h.view(np.int16)), dtype, d, 7, 3, e.buf, s.buf)
    torch.cuda.synchronize()
    e_ref, s_ref = oracle.nc_compress_typed(h, dtype, 7, 3)
    check_nc_planes(e, s, d, e_ref, s_ref)


@pytest.mark.gpu
def test_gpu_typed_batch_and_aggregate_round_trip():
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import dev
    rng = np.random.default_rng(3)
    n, d = 4, 300_000
    hs = [rng.standard_normal(d).astype(np.float16).view(np.uint16) for _ in range(n)]
    xd = [dev(h.view(np.int16)) for h in hs]
    u8 = dict(dtype=torch.uint8, device="cuda")
    es = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
    ss = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
    nc.nc_compress_typed_batch(xd, F16, d, 1, [5, 6, 7, 8], es, ss, n)
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nc_aggregate(es, ss, n, d, out)
    torch.cuda.synchronize()
    refs = [oracle.nc_compress_typed(h, F16, 1, 5 + i) for i, h in enumerate(hs)]
    want = oracle.nc_aggregate([r[0] for r in refs], [r[1] for r in refs], d)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want.view(np.uint32))
    with pytest.raises(nc.NatcompError):
        nc.nc_compress_typed(xd[0], 9, d, 1, 0, es[0], ss[0])


# ---- bfloat16 with 7-bit thresholds: one stream byte per entry --------------------------------
def test_bf16_short_threshold_rounds_up_in_exactly_m_of_128_draws():
    # every finite bfloat16 pattern against every 7-bit draw: the number of draws that round up
    # is the mantissa field (so P(up) = m exactly), and the mean over the draws is the value itself
    h = _all_patterns()
    t = oracle.values_of_16bit(h, BF16)
    e_field = (h >> 7) & 0xFF
    m_field = (h & 0x7F).astype(np.int64)
    finite = e_field < 254                       # 254: never up (saturation); 255: inf / NaN
    ups = np.zeros(h.size, np.int64)
    total = np.zeros(h.size, np.float64)
    lo_e, _ = oracle.cnat_codes(t, np.full(h.size, 127 << 16, np.uint32))   # r7 = 127: never up
    for r7 in range(128):
        vals = oracle.cnat_values(t, np.full(h.size, r7 << 16, np.uint32))
        e, _ = oracle.cnat_codes(t, np.full(h.size, r7 << 16, np.uint32))
        ups += (e != lo_e)
        total += np.where(finite, vals.astype(np.float64), 0.0)
    assert np.array_equal(ups[finite], m_field[finite])
    assert np.all(ups[~finite] == 0)
    want = np.where(finite, t.astype(np.float64), 0.0)
    assert np.array_equal(total / 128.0, want)           # exact: sums of 128 powers of two


def test_bf16_short_threshold_stream_mapping():
    # entry j draws byte (j mod 4) of stream word j / 4 of domain 4 (the word stream itself is
    # pinned by the generator's known answers); the codes are those of the binary32 rule with
    # r23 = r7 * 2^16
    rng = np.random.default_rng(11)
    d = 4099
    h = rng.integers(0, 1 << 16, d).astype(np.uint16)
    seed, worker = 0xABCDEF0123, 9
    words = oracle.stream_words(seed, worker, 4, 0, (d + 3) // 4)
    j = np.arange(d)
    r7 = (words[j // 4] >> (8 * (j % 4)).astype(np.uint32)) & 0x7F
    e_want, s_want = oracle.cnat_codes(oracle.values_of_16bit(h, BF16), (r7 << 16).astype(np.uint32))
    e, s = oracle.nc_compress_bf16_r8(h, seed, worker)
    assert np.array_equal(e, e_want)
    bits = (s[j // 32] >> (j % 32).astype(np.uint32)) & 1
    assert np.array_equal(bits.astype(np.uint8), s_want)
    # a different stream from the 23-bit variant's (domain 0)
    e23, _ = oracle.nc_compress_typed(h, BF16, seed, worker)
    assert not np.array_equal(e, e23)


def test_bf16_short_threshold_frequency():
    d = 1 << 20
    h = np.full(d, 0x3F80 | 37, np.uint16)               # 1 + 37/128
    e, _ = oracle.nc_compress_bf16_r8(h, 3, 1)
    p = 37 / 128
    assert abs((e == 128).mean() - p) < 5 * np.sqrt(p * (1 - p) / d)
    assert set(np.unique(e)) == {127, 128}


@pytest.mark.gpu
@pytest.mark.parametrize("d", [1, 5, 31, 1024, 2048, 4097, 65536, 6 * 2048 + 515, (1 << 20) + 33])
def test_gpu_bf16_short_threshold_matches_oracle(d):
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import Guarded, check_nc_planes, dev
    rng = np.random.default_rng(d)
    if d == 65536:
        h = _all_patterns()                       # every pattern, specials included
    else:
        x = (rng.standard_normal(d) * 10.0 ** rng.uniform(-6, 3, d)).astype(np.float32)
        h = (x.view(np.uint32) >> 16).astype(np.uint16)
        h[rng.random(d) < 0.01] = 0x7F00 | 0x55   # exponent field 254: must not round up
        h[rng.random(d) < 0.01] = 0x0033          # subnormal
    e = Guarded(nc.nc_exp_bytes(d))
    s = Guarded(nc.nc_sign_bytes(d))
    nc.nc_compress_bf16_r8(dev(h.view(np.int16)), d, 7, 3, e.buf, s.buf)
    torch.cuda.synchronize()
    e_ref, s_ref = oracle.nc_compress_bf16_r8(h, 7, 3)
    check_nc_planes(e, s, d, e_ref, s_ref)


@pytest.mark.gpu
def test_gpu_bf16_short_threshold_batch_aggregate_and_errors():
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import dev
    rng = np.random.default_rng(5)
    n, d = 3, 200_003
    hs = [(rng.standard_normal(d).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
          for _ in range(n)]
    xd = [dev(h.view(np.int16)) for h in hs]
    u8 = dict(dtype=torch.uint8, device="cuda")
    es = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
    ss = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
    nc.nc_compress_bf16_r8_batch(xd, d, 1, [5, 6, 7], es, ss, n)
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nc_aggregate(es, ss, n, d, out)
    torch.cuda.synchronize()
    refs = [oracle.nc_compress_bf16_r8(h, 1, 5 + i) for i, h in enumerate(hs)]
    want = oracle.nc_aggregate([r[0] for r in refs], [r[1] for r in refs], d)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want.view(np.uint32))
    with pytest.raises(nc.NatcompError):
        nc.nc_compress_bf16_r8(xd[0][1:], d - 1, 1, 0, es[0], ss[0])       # misaligned input
    nc.nc_compress_bf16_r8(xd[0], 0, 1, 0, es[0], ss[0])                   # d = 0: nothing to do


@pytest.mark.gpu
def test_gpu_bf16_short_threshold_full_size_batch():
    # the benchmark shape: 2 of the 8 workers of the ResNet-50-sized vector in one batch launch,
    # whole planes compared
    import torch
    import paper_1905_10988_b200 as nc
    d, n = 25_557_032, 2
    g = torch.Generator(device="cuda").manual_seed(2001)
    xs = [(torch.randn(d, device="cuda", generator=g) * 1e-3).to(torch.bfloat16) for _ in range(n)]
    u8 = dict(dtype=torch.uint8, device="cuda")
    es = [torch.full((nc.nc_exp_bytes(d),), 0xCD, **u8) for _ in range(n)]
    ss = [torch.full((nc.nc_sign_bytes(d),), 0xCD, **u8) for _ in range(n)]
    nc.nc_compress_bf16_r8_batch(xs, d, 0, [0, 1], es, ss, n)
    torch.cuda.synchronize()
    for w in range(n):
        h = xs[w].view(torch.int16).cpu().numpy().view(np.uint16)
        e_ref, s_ref = oracle.nc_compress_bf16_r8(h, 0, w)
        assert np.array_equal(es[w].cpu().numpy()[:d], e_ref)
        assert np.array_equal(ss[w].cpu().numpy().view(np.uint32)[:s_ref.size], s_ref)


# ---- binary16 with 10-bit thresholds: one stream half-word per entry ---------------------------
def test_f16_short_threshold_rounds_up_in_exactly_m_of_1024_draws():
    # every finite binary16 pattern against every 10-bit draw: the draws that round up number
    # m * 1024 (the mantissa field of a normal value, the normalised fraction of a subnormal), and
    # the mean over the draws is the value itself
    h = _all_patterns()
    t = oracle.values_of_16bit(h, F16)
    e_field = (h >> 10) & 0x1F
    m_field = (h & 0x3FF).astype(np.int64)
    finite = e_field < 31
    want_ups = m_field.copy()
    sub = (e_field == 0) & (m_field > 0)
    lead = np.floor(np.log2(np.maximum(m_field, 1))).astype(np.int64)
    want_ups[sub] = ((m_field[sub] - (1 << lead[sub])) << (10 - lead[sub]))
    ups = np.zeros(h.size, np.int64)
    total = np.zeros(h.size, np.float64)
    lo_e, _ = oracle.cnat_codes(t, np.full(h.size, 1023 << 13, np.uint32))   # never up
    for r10 in range(1024):
        r23 = np.full(h.size, r10 << 13, np.uint32)
        e, _ = oracle.cnat_codes(t, r23)
        ups += (e != lo_e)
        total += np.where(finite, oracle.cnat_values(t, r23).astype(np.float64), 0.0)
    assert np.array_equal(ups[finite], want_ups[finite])
    assert np.all(ups[~finite] == 0)
    assert np.array_equal(total / 1024.0, np.where(finite, t.astype(np.float64), 0.0))


def test_f16_short_threshold_stream_mapping_and_frequency():
    rng = np.random.default_rng(12)
    d = 4099
    h = rng.integers(0, 1 << 16, d).astype(np.uint16)
    seed, worker = 0x1234567, 4
    words = oracle.stream_words(seed, worker, 5, 0, (d + 1) // 2)
    j = np.arange(d)
    r10 = (words[j // 2] >> (16 * (j % 2)).astype(np.uint32)) & 0x3FF
    e_want, s_want = oracle.cnat_codes(oracle.values_of_16bit(h, F16), (r10 << 13).astype(np.uint32))
    e, s = oracle.nc_compress_f16_r16(h, seed, worker)
    assert np.array_equal(e, e_want)
    bits = (s[j // 32] >> (j % 32).astype(np.uint32)) & 1
    assert np.array_equal(bits.astype(np.uint8), s_want)
    n = 1 << 20
    e, _ = oracle.nc_compress_f16_r16(np.full(n, (15 << 10) | 300, np.uint16), 3, 1)   # 1 + 300/1024
    p = 300 / 1024
    assert abs((e == 128).mean() - p) < 5 * np.sqrt(p * (1 - p) / n)
    assert set(np.unique(e)) == {127, 128}


@pytest.mark.gpu
@pytest.mark.parametrize("d", [1, 5, 31, 1024, 4097, 65536, 6 * 1024 + 515, (1 << 20) + 33])
def test_gpu_f16_short_threshold_matches_oracle(d):
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import Guarded, check_nc_planes, dev
    rng = np.random.default_rng(d + 1)
    if d == 65536:
        h = _all_patterns()                       # every pattern: subnormals, inf, NaN
    else:
        x = (rng.standard_normal(d) * 10.0 ** rng.uniform(-7, 3, d)).astype(np.float32)
        h = x.astype(np.float16).view(np.uint16)
    e = Guarded(nc.nc_exp_bytes(d))
    s = Guarded(nc.nc_sign_bytes(d))
    nc.nc_compress_f16_r16(dev(h.view(np.int16)), d, 7, 3, e.buf, s.buf)
    torch.cuda.synchronize()
    e_ref, s_ref = oracle.nc_compress_f16_r16(h, 7, 3)
    check_nc_planes(e, s, d, e_ref, s_ref)


@pytest.mark.gpu
def test_gpu_f16_short_threshold_batch():
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import dev
    rng = np.random.default_rng(6)
    n, d = 3, 200_003
    hs = [rng.standard_normal(d).astype(np.float16).view(np.uint16) for _ in range(n)]
    xd = [dev(h.view(np.int16)) for h in hs]
    u8 = dict(dtype=torch.uint8, device="cuda")
    es = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
    ss = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
    nc.nc_compress_f16_r16_batch(xd, d, 1, [5, 6, 7], es, ss, n)
    torch.cuda.synchronize()
    for i, h in enumerate(hs):
        e_ref, s_ref = oracle.nc_compress_f16_r16(h, 1, 5 + i)
        assert np.array_equal(es[i].cpu().numpy()[:d], e_ref)
        assert np.array_equal(ss[i].cpu().numpy().view(np.uint32)[:s_ref.size], s_ref)
    with pytest.raises(nc.NatcompError):
        nc.nc_compress_f16_r16(xd[0][1:], d - 1, 1, 0, es[0], ss[0])       # misaligned input
