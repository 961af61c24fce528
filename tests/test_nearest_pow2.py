"""The deterministic control variant (rounding to the nearest power of two, no sampling):
oracle pins on CPU, GPU parity through the C ABI."""
import numpy as np
import pytest

import oracle


def _decode(e, s, d):
    j = np.arange(d)
    return oracle.cnat_decode(e, ((s[j // 32] >> (j % 32)) & 1).astype(np.uint8))


def test_oracle_nearest_values_and_relation_to_cnat():
    x = np.float32([2.5, 3.0, 3.5, -2.75, 0.75, 1.0, 0.0, -0.0, 1e-40, 7e-39, np.inf, -np.inf,
                    3.4e38, -5e-324])
    e, s = oracle.nc_compress_nearest(x)
    got = _decode(e, s, x.size)
    want = np.float32([2, 4, 4, -2, 1, 1, 0, -0.0, 0, 2.0 ** -126, np.inf, -np.inf, 2.0 ** 127,
                       -0.0])
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # numpy cross-check on random normal numbers: nearest of {2^floor, 2^(floor+1)}, ties up
    rng = np.random.default_rng(1)
    y = (rng.standard_normal(100_000) * 10.0 ** rng.uniform(-6, 6, 100_000)).astype(np.float32)
    y = y[y != 0]
    e, s = oracle.nc_compress_nearest(y)
    a = np.abs(y.astype(np.float64))
    lo = 2.0 ** np.floor(np.log2(a))
    ref = np.where(a - lo >= 2 * lo - a, 2 * lo, lo) * np.sign(y)
    assert np.array_equal(_decode(e, s, y.size).astype(np.float64), ref)
    # it is the C_nat rule with the fixed threshold 2^22 - 1 in place of the random bits
    ec, sc = oracle.cnat_codes(y, np.full(y.size, (1 << 22) - 1, np.uint32))
    assert np.array_equal(e, ec)
    # biased, unlike C_nat: E over a mantissa-uniform input is not the input
    t = np.float32(1.25)
    assert _decode(*oracle.nc_compress_nearest(np.float32([t])), 1)[0] == 1.0


@pytest.mark.gpu
@pytest.mark.parametrize("d", [1, 33, 1024, 4097, (1 << 20) + 7])
def test_gpu_nearest_matches_oracle(d):
    import torch
    import paper_1905_10988_b200 as nc
    from gpu_util import Guarded, check_nc_planes, dev, special_values
    rng = np.random.default_rng(d)
    x = (rng.standard_normal(d) * 10.0 ** rng.uniform(-8, 3, d)).astype(np.float32)
    if d >= 32:
        sp = special_values(rng, d // 8)
        x[rng.choice(d, sp.size, replace=False)] = sp
        x[:4] = np.float32([3.0, -0.75, 1.5, 2.0 ** -127])        # exact midpoints
    e = Guarded(nc.nc_exp_bytes(d))
    s = Guarded(nc.nc_sign_bytes(d))
    nc.nc_compress_nearest(dev(x), d, e.buf, s.buf)
    torch.cuda.synchronize()
    e.check()
    s.check()
    e_ref, s_ref = oracle.nc_compress_nearest(x)
    check_nc_planes(e, s, d, e_ref, s_ref)
