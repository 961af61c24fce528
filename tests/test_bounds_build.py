"""The debug build of the library (-DNC_BOUNDS): every global store of the C_nat and D_nat kernels
is checked against the ranges its call may write, a store outside them is skipped and counted,
nothing traps.  The small ragged sizes of the parity tests run through it; the outputs must equal
the regular library's byte for byte and the count must stay at zero.  The self-test aims one store
past a 16-byte range inside a real buffer, so that the mechanism is seen to work without any
invalid access."""
import ctypes as C
import importlib.util
import os

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _build_module():
    spec = importlib.util.spec_from_file_location(
        "_natcomp_build", os.path.join(ROOT, "paper_1905_10988_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


@pytest.fixture(scope="module")
def dbg():
    lib = C.CDLL(_build_module().build(bounds=True))     # no-op when up to date
    lib.nc_exp_bytes.restype = C.c_size_t
    return lib


def test_regular_library_has_no_bounds_mode():
    import paper_1905_10988_b200 as nc
    v, a = C.c_uint64(7), C.c_uint64(7)
    assert nc.status_string(nc.lib.nc_debug_bounds_status(C.byref(v), C.byref(a), 0)) == \
        "NC_ERR_UNSUPPORTED"
    assert nc.status_string(nc.lib.nc_debug_bounds_selftest(None, None)) == "NC_ERR_UNSUPPORTED"


def test_debug_library_exports_the_same_entry_points(dbg):
    import paper_1905_10988_b200 as nc
    for name in nc.EXPORTS:
        assert hasattr(dbg, name), name


def _status(dbg, reset=False):
    v, a = C.c_uint64(0), C.c_uint64(0)
    assert dbg.nc_debug_bounds_status(C.byref(v), C.byref(a), int(reset)) == 0
    return int(v.value), int(a.value)


@pytest.mark.gpu
def test_checked_stores_same_bytes_and_no_violation(dbg):
    import torch
    import paper_1905_10988_b200 as nc
    from paper_1905_10988_b200 import workloads
    vp, sz = C.c_void_p, C.c_size_t
    stream = vp(torch.cuda.current_stream().cuda_stream)

    def ptrs(ts):
        return (vp * len(ts))(*[t.data_ptr() for t in ts])

    _status(dbg, reset=True)
    rng = np.random.default_rng(3)
    n = 3
    for d in (1, 33, 1000, 4097, 70001, (1 << 18) + 40):
        u8 = dict(dtype=torch.uint8, device="cuda")
        xs = [torch.from_numpy((rng.standard_normal(d) * 1e-2).astype(np.float32)).cuda()
              for _ in range(n)]
        workers = (C.c_uint32 * n)(5, 0, 9)
        off = workloads.small_bucket_table(d, seed=d)
        B = len(off) - 1
        offd = torch.tensor(off, dtype=torch.int64, device="cuda")
        wsb = nc.nd_batch_workspace_bytes(d, B, n)
        results = []
        for lib in (nc.lib, dbg):
            es = [torch.full((nc.nc_exp_bytes(d),), 0xEE, **u8) for _ in range(n)]
            ss = [torch.full((nc.nc_sign_bytes(d),), 0xEE, **u8) for _ in range(n)]
            out = torch.full((d,), 7.0, dtype=torch.float32, device="cuda")
            ref = torch.full((d,), 7.0, dtype=torch.float32, device="cuda")
            norms = [torch.full((B,), -1.0, dtype=torch.float32, device="cuda") for _ in range(n)]
            lv = [torch.full((nc.nd_level_bytes(d),), 0xEE, **u8) for _ in range(n)]
            sg = [torch.full((nc.nc_sign_bytes(d),), 0xEE, **u8) for _ in range(n)]
            ws = torch.empty(wsb, **u8)
            outd = torch.full((d,), 7.0, dtype=torch.float32, device="cuda")
            calls = [
                lib.nc_compress_batch(ptrs(xs), sz(d), C.c_uint64(11), workers, ptrs(es), ptrs(ss),
                                      n, stream),
                lib.nc_aggregate(ptrs(es), ptrs(ss), n, sz(d), vp(out.data_ptr()), stream),
                lib.nc_decode_accumulate(vp(es[0].data_ptr()), vp(ss[0].data_ptr()), sz(d),
                                         vp(out.data_ptr()), stream),
                lib.nc_sum_fp32(ptrs(xs), n, sz(d), vp(ref.data_ptr()), stream),
                lib.nd_compress_batch(ptrs(xs), sz(d), vp(offd.data_ptr()), B, 2, 8, C.c_uint64(11),
                                      workers, ptrs(norms), ptrs(lv), ptrs(sg), n,
                                      vp(ws.data_ptr()), sz(wsb), None, stream),
                lib.nd_aggregate(ptrs(norms), ptrs(lv), ptrs(sg), n, sz(d), vp(offd.data_ptr()), B,
                                 8, vp(outd.data_ptr()), stream),
                lib.nd_decode_accumulate(vp(norms[1].data_ptr()), vp(lv[1].data_ptr()),
                                         vp(sg[1].data_ptr()), sz(d), vp(offd.data_ptr()), B, 8,
                                         vp(outd.data_ptr()), stream),
            ]
            assert calls == [0] * len(calls), calls
            torch.cuda.synchronize()
            results.append([t.cpu().numpy().view(np.uint8)
                            for t in es + ss + [out, ref] + norms + lv + sg + [outd]])
        for a, b in zip(*results):
            assert np.array_equal(a, b), d
        assert _status(dbg) == (0, 0), d


@pytest.mark.gpu
def test_a_store_outside_the_ranges_is_skipped_and_counted(dbg):
    import torch
    _status(dbg, reset=True)
    scratch = torch.zeros(128, dtype=torch.uint8, device="cuda")
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert dbg.nc_debug_bounds_selftest(C.c_void_p(scratch.data_ptr()), stream) == 0
    violations, address = _status(dbg)
    assert violations == 1 and address == scratch.data_ptr() + 64
    assert int(scratch.sum()) == 0                        # the store did not happen
    assert _status(dbg, reset=True)[0] == 1               # reading with reset returns, then clears
    assert _status(dbg) == (0, 0)
