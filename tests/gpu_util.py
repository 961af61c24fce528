"""Helpers for the GPU parity tests: guarded device buffers and thin wrappers that run one
C-ABI call and bring the result back as numpy."""
import numpy as np
import torch

import paper_1905_10988_b200 as nc

GUARD = 256          # canary bytes on each side of every output buffer
CANARY = 0xA5


class Guarded:
    """A device byte buffer of `nbytes` with canary bands before and after it."""

    def __init__(self, nbytes: int, fill: int = 0xCD):
        self.nbytes = int(nbytes)
        self.raw = torch.full((self.nbytes + 2 * GUARD,), CANARY, dtype=torch.uint8, device="cuda")
        self.buf = self.raw[GUARD:GUARD + self.nbytes]
        if self.nbytes:
            self.buf.fill_(fill)       # stale contents must be overwritten by the call
        assert self.buf.data_ptr() % 32 == 0

    def check(self):
        raw = self.raw.cpu().numpy()
        assert np.all(raw[:GUARD] == CANARY), "write before the buffer"
        assert np.all(raw[GUARD + self.nbytes:] == CANARY), "write past the buffer"

    def numpy(self, dtype):
        return self.buf.cpu().numpy().view(dtype)


def assert_same_floats(got, want):
    """Bit for bit, except that any NaN matches any NaN: IEEE 754 leaves the sign and payload of
    a generated NaN open, and the host and the device choose differently."""
    got = np.asarray(got).view(np.float32)
    want = np.asarray(want).view(np.float32)
    gn, wn = np.isnan(got), np.isnan(want)
    assert np.array_equal(gn, wn), "NaN positions differ"
    assert np.array_equal(got.view(np.uint32)[~gn], want.view(np.uint32)[~wn])


def dev(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def gpu_nc_compress(x_dev, seed, worker):
    d = x_dev.numel()
    e = Guarded(nc.nc_exp_bytes(d))
    s = Guarded(nc.nc_sign_bytes(d))
    nc.nc_compress(x_dev, d, seed, worker, e.buf, s.buf)
    torch.cuda.synchronize()
    e.check()
    s.check()
    return e, s


def check_nc_planes(e: Guarded, s: Guarded, d, exp_ref, sign_ref):
    eg = e.numpy(np.uint8)
    sg = s.numpy(np.uint32)
    assert np.array_equal(eg[:d], exp_ref), "exponent plane differs"
    assert np.all(eg[d:] == 0), "exponent padding not zero"
    nw = (d + 31) // 32
    assert np.array_equal(sg[:nw], sign_ref), "sign plane differs"
    assert np.all(sg[nw:] == 0), "sign padding not zero"


def unpack_nibbles(level_bytes, d):
    lv = np.asarray(level_bytes, np.uint8)
    return np.stack([lv & 0xF, lv >> 4], 1).ravel()[:d]


def special_values(rng, count):
    """Bit patterns covering zeros, subnormals, powers of two, the top exponents, inf and NaN."""
    f = np.empty(count, np.uint32)
    kinds = rng.integers(0, 8, count)
    mant = rng.integers(0, 1 << 23, count, dtype=np.uint64).astype(np.uint32)
    sign = rng.integers(0, 2, count, dtype=np.uint64).astype(np.uint32) << 31
    expo = rng.integers(0, 256, count, dtype=np.uint64).astype(np.uint32)
    f[:] = sign | (expo << 23) | mant
    f[kinds == 0] = sign[kinds == 0]                                   # +-0
    f[kinds == 1] = sign[kinds == 1] | mant[kinds == 1]                # subnormal
    f[kinds == 2] = sign[kinds == 2] | (expo[kinds == 2] << 23)        # powers of two, inf, 0
    f[kinds == 3] = sign[kinds == 3] | (np.uint32(254) << 23) | mant[kinds == 3]
    f[kinds == 4] = sign[kinds == 4] | (np.uint32(255) << 23) | mant[kinds == 4]   # NaN / inf
    return f.view(np.float32)
