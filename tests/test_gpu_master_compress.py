"""GPU parity, master-side compression of the aggregate (Algorithm 1: g = C_M(sum_i Delta_i) with
C_M = C_nat): the fused call must equal the oracle's aggregate followed by the oracle's C_nat
with the master's stream, bit for bit, and the unfused pair of calls on the GPU."""
import numpy as np
import pytest
import torch

import oracle
import paper_1905_10988_b200 as nc
from paper_1905_10988_b200 import workloads
from gpu_util import Guarded, check_nc_planes, dev

pytestmark = pytest.mark.gpu

MASTER = 0xFFFFFFFF


def _random_planes(rng, n, d):
    exps, signs = [], []
    for _ in range(n):
        e = rng.integers(100, 150, nc.nc_exp_bytes(d)).astype(np.uint8)
        odd = rng.random(e.size)
        e[odd < 0.05] = 0
        e[(odd > 0.05) & (odd < 0.06)] = 254
        e[(odd > 0.06) & (odd < 0.065)] = 255
        exps.append(e)
        signs.append(rng.integers(0, 1 << 32, nc.nc_sign_bytes(d) // 4, dtype=np.uint64)
                     .astype(np.uint32))
    return exps, signs


@pytest.mark.parametrize("n,d", [(1, 5), (2, 1024), (4, 4097), (8, 70001), (16, 3000),
                                 (64, 2048 + 31)])
def test_fused_aggregate_compress_matches_oracle_composition(n, d):
    rng = np.random.default_rng(n * 131 + d)
    exps, signs = _random_planes(rng, n, d)
    ed = [dev(e) for e in exps]
    sd = [dev(s) for s in signs]
    oe = Guarded(nc.nc_exp_bytes(d))
    os_ = Guarded(nc.nc_sign_bytes(d))
    nc.nc_aggregate_compress(ed, sd, n, d, 7, MASTER, oe.buf, os_.buf)
    torch.cuda.synchronize()
    oe.check()
    os_.check()
    total = oracle.nc_aggregate([e[:d] for e in exps], signs, d)      # fp32, worker order
    e_ref, s_ref = oracle.nc_compress(total, 7, MASTER)
    # inf - inf gives a NaN whose sign IEEE 754 leaves open (x86 and the GPU differ): such an
    # entry must encode as exponent 255 on both sides, its sign bit is not compared
    nan_at = np.nonzero(np.isnan(total))[0]
    if n >= 8:
        assert nan_at.size > 0                 # the case is really exercised
    assert np.all(e_ref[nan_at] == 255)
    got_sign = os_.numpy(np.uint32)
    for j in nan_at:
        bit = np.uint32(1) << np.uint32(j % 32)
        s_ref[j // 32] = (s_ref[j // 32] & ~bit) | (got_sign[j // 32] & bit)
    check_nc_planes(oe, os_, d, e_ref, s_ref)
    # the unfused pair on the GPU gives the same planes
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nc_aggregate(ed, sd, n, d, out)
    e2 = Guarded(nc.nc_exp_bytes(d))
    s2 = Guarded(nc.nc_sign_bytes(d))
    nc.nc_compress(out, d, 7, MASTER, e2.buf, s2.buf)
    torch.cuda.synchronize()
    assert np.array_equal(e2.numpy(np.uint8), oe.numpy(np.uint8))
    assert np.array_equal(s2.numpy(np.uint32), os_.numpy(np.uint32))


def test_bidirectional_round_on_config1():
    # workers compress, the master aggregates and compresses again; the decoded result is an
    # unbiased estimate of the exact sum with second moment within (9/8)^2 (Thm. 3 composition)
    n, d = 4, 1 << 20
    xs = [workloads.config1_vector(w, d) for w in range(n)]
    xd = [x.cuda() for x in xs]
    u8 = dict(dtype=torch.uint8, device="cuda")
    es = [torch.empty(nc.nc_exp_bytes(d), **u8) for _ in range(n)]
    ss = [torch.empty(nc.nc_sign_bytes(d), **u8) for _ in range(n)]
    nc.nc_compress_batch(xd, d, 0, list(range(n)), es, ss, n)
    ge = torch.empty(nc.nc_exp_bytes(d), **u8)
    gs = torch.empty(nc.nc_sign_bytes(d), **u8)
    nc.nc_aggregate_compress(es, ss, n, d, 0, MASTER, ge, gs)
    g = torch.zeros(d, dtype=torch.float32, device="cuda")
    nc.nc_decode_accumulate(ge, gs, d, g)
    torch.cuda.synchronize()
    refs = [oracle.nc_compress(x.numpy(), 0, w) for w, x in enumerate(xs)]
    total = oracle.nc_aggregate([r[0] for r in refs], [r[1] for r in refs], d)
    e_ref, s_ref = oracle.nc_compress(total, 0, MASTER)
    assert np.array_equal(ge.cpu().numpy()[:d], e_ref)
    assert np.array_equal(gs.cpu().numpy().view(np.uint32)[:d // 32], s_ref)
    exact = np.sum([x.numpy().astype(np.float64) for x in xs], axis=0)
    err2 = float(((g.cpu().numpy().astype(np.float64) - exact) ** 2).sum())
    x2 = float(sum((x.numpy().astype(np.float64) ** 2).sum() for x in xs))
    # E||C_M(sum C(x_i)) - sum x_i||^2 <= (1/8) E||sum C(x_i)||^2 + (1/8) sum ||x_i||^2
    s2 = float((exact ** 2).sum())
    assert err2 <= (1 / 8) * (s2 + x2 / 8) + x2 / 8 + 0.02 * x2


def test_dithering_with_naturally_compressed_norm():
    # Def. 3 with C = C_nat on the norm (the variant the paper proposes for in-network
    # aggregation: the norm travels as an 8-bit exponent and decoding is exponent addition).
    # Recipe with the existing calls: nd_compress, then nc_compress on the vector of norms,
    # decode it on the master, nd_aggregate with the decoded (power-of-two) norms.
    rng = np.random.default_rng(3)
    n, d, p, s = 3, 50_000, 2, 8
    off = workloads.small_bucket_table(d, seed=2)
    B = len(off) - 1
    off_dev = dev(np.asarray(off, np.uint64).view(np.int64))
    xs = [(rng.standard_normal(d) * 1e-3).astype(np.float32) for _ in range(n)]
    u8 = dict(dtype=torch.uint8, device="cuda")
    norms, levels, signs, tx = [], [], [], []
    ws_bytes = nc.nd_workspace_bytes(d, B)
    ws = torch.empty(ws_bytes, **u8)
    ref_norms, ref_levels, ref_signs = [], [], []
    for w in range(n):
        nm = torch.empty(B, dtype=torch.float32, device="cuda")
        lv = torch.empty(nc.nd_level_bytes(d), **u8)
        sg = torch.empty(nc.nc_sign_bytes(d), **u8)
        nc.nd_compress(dev(xs[w]), d, off_dev, B, p, s, 1, w, nm, lv, sg, ws, ws_bytes)
        # the norm vector goes through C_nat with its own worker id (here 1000 + w)
        ne = torch.empty(nc.nc_exp_bytes(B), **u8)
        ns = torch.empty(nc.nc_sign_bytes(B), **u8)
        nc.nc_compress(nm, B, 1, 1000 + w, ne, ns)
        dec = torch.zeros(B, dtype=torch.float32, device="cuda")
        nc.nc_decode_accumulate(ne, ns, B, dec)
        norms.append(nm); levels.append(lv); signs.append(sg); tx.append(dec)
        # oracle side of the same recipe
        gn = nm.cpu().numpy()
        r = oracle.nd_compress(xs[w], off, p, s, 1, w, given_norms=gn)
        e_ref, s_ref = oracle.nc_compress(gn, 1, 1000 + w)
        dn = np.zeros(B, np.float32)
        oracle.nc_decode_accumulate(e_ref, s_ref, dn)
        ref_norms.append(dn); ref_levels.append(r[1]); ref_signs.append(r[2])
        assert np.array_equal(dec.cpu().numpy(), dn)
        # a compressed norm is a power of two within a factor two of the norm
        ratio = dn / gn
        assert np.all((ratio > 0.5) & (ratio < 2.0))
        assert np.all(np.frexp(dn)[0] == 0.5)
    out = torch.empty(d, dtype=torch.float32, device="cuda")
    nc.nd_aggregate(tx, levels, signs, n, d, off_dev, B, s, out)
    torch.cuda.synchronize()
    want = oracle.nd_aggregate(ref_norms, ref_levels, ref_signs, off, s, d)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want.view(np.uint32))
