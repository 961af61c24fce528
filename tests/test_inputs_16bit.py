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
