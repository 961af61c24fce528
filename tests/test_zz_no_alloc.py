"""nd_compress_static: the dithering compressor for callers that cannot allocate device memory
(for example a gradient hook that runs while a framework's allocator owns the whole device, or
a process with a memory budget fixed at start-up).  Its scratch is a fixed 1 MiB array inside
the library instead of a workspace argument.

The test goes through the C ABI and requires the outputs to be identical to those of
nd_compress, on two calls in a row: the second call reuses the array with whatever the first
one left in it, on a different vector, bucket table and norm.  This file is collected last so
that a run that stops at the first failure has already run every other test; it also passes
when run alone in a fresh process.
"""
import numpy as np
import pytest
import torch

import paper_1905_10988_b200 as nc
from paper_1905_10988_b200 import workloads

pytestmark = pytest.mark.gpu


def _compress_both_ways(x, off, p, s, seed, worker):
    d = x.numel()
    B = len(off) - 1
    off_dev = torch.tensor(off, dtype=torch.int64, device="cuda")
    u8 = dict(dtype=torch.uint8, device="cuda")
    outs = []
    for static in (False, True):
        norms = torch.full((B,), -1.0, dtype=torch.float32, device="cuda")
        level = torch.full((nc.nd_level_bytes(d),), 0xEE, **u8)
        sign = torch.full((nc.nc_sign_bytes(d),), 0xEE, **u8)
        if static:
            nc.nd_compress_static(x, d, off_dev, B, p, s, seed, worker, norms, level, sign)
        else:
            ws_bytes = nc.nd_workspace_bytes(d, B)
            ws = torch.empty(ws_bytes, **u8)
            nc.nd_compress(x, d, off_dev, B, p, s, seed, worker, norms, level, sign, ws, ws_bytes)
        torch.cuda.synchronize()
        outs.append((norms.cpu().numpy(), level.cpu().numpy(), sign.cpu().numpy()))
    return outs


def test_static_scratch_variant_matches_nd_compress_twice_in_a_row():
    assert nc.nd_static_scratch_bytes() == 1 << 20
    cases = [
        # (d, bucket table seed, p, s, seed, worker)
        ((1 << 20) + 333, 5, 2, 8, 17, 3),
        (70_001, 9, nc.P_INF, 4, 18, 1),        # smaller: most of the array keeps stale data
    ]
    for d, tseed, p, s, seed, worker in cases:
        off = workloads.small_bucket_table(d, seed=tseed)
        assert nc.nd_workspace_bytes(d, len(off) - 1) <= nc.nd_static_scratch_bytes()
        g = torch.Generator(device="cuda").manual_seed(d)
        x = torch.randn(d, generator=g, device="cuda", dtype=torch.float32) * 3e-3
        (n0, l0, s0), (n1, l1, s1) = _compress_both_ways(x, off, p, s, seed, worker)
        assert np.array_equal(n0.view(np.uint32), n1.view(np.uint32))
        assert np.array_equal(l0, l1)
        assert np.array_equal(s0, s1)
        assert np.all(n1 >= 0)                  # every norm was written


def test_static_scratch_variant_rejects_sizes_beyond_its_array():
    # A short vector cut into very many (mostly empty) buckets needs more scratch than the array
    # holds.  Every buffer is real and large enough, so if the size check ever stopped working the
    # call would run a valid problem and the test would fail on the status, not fault the device.
    d, B = 1024, 200_000
    assert nc.nd_workspace_bytes(d, B) > nc.nd_static_scratch_bytes()
    off = torch.zeros(B + 1, dtype=torch.int64, device="cuda")
    off[B // 2:] = d // 2
    off[B] = d
    x = torch.ones(d, dtype=torch.float32, device="cuda")
    norms = torch.full((B,), -1.0, dtype=torch.float32, device="cuda")
    level = torch.zeros(nc.nd_level_bytes(d), dtype=torch.uint8, device="cuda")
    sign = torch.zeros(nc.nc_sign_bytes(d), dtype=torch.uint8, device="cuda")
    with pytest.raises(nc.NatcompError) as err:
        nc.nd_compress_static(x, d, off, B, 2, 8, 0, 0, norms, level, sign)
    assert nc.status_string(err.value.status) == "NC_ERR_TOO_LARGE"
    torch.cuda.synchronize()
    assert bool(torch.all(norms == -1.0))       # nothing was launched
