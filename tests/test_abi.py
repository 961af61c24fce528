"""The C-ABI library loads without a GPU, exports every entry point the header declares, and
its host-side argument validation returns the documented status codes (no kernel is launched
by any call in this file)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "natcomp.h")


@pytest.fixture(scope="module")
def nc():
    import importlib.util
    spec = importlib.util.spec_from_file_location(
        "_natcomp_build", os.path.join(ROOT, "paper_1905_10988_b200", "build.py"))
    build = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(build)
    build.build()                               # no-op when the library is up to date
    import paper_1905_10988_b200 as pkg
    return pkg


def _declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = re.findall(r"\b(n[cd](?:8|64)?_[a-z0-9_]+)\s*\(", src)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(nc):
    declared = _declared_functions()
    assert len(declared) >= 16
    raw = C.CDLL(nc.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), "missing export: " + name
    assert set(nc.EXPORTS) == set(declared)
    for name in declared:                      # the binding carries the same names
        assert callable(getattr(nc, name if name != "nc_status_string" else "status_string"))


def test_size_helpers(nc):
    assert nc.nc_exp_bytes(0) == 0 and nc.nc_exp_bytes(1) == 16 and nc.nc_exp_bytes(1024) == 1024
    assert nc.nc_sign_bytes(1) == 16 and nc.nc_sign_bytes(129) == 32
    assert nc.nc_sign_bytes(25_557_032) == 3_194_640          # 798,658 words, padded to 16 B
    assert nc.nd_level_bytes(1) == 16 and nc.nd_level_bytes(33) == 32
    assert nc.nd_workspace_bytes(25_557_032, 161) >= 8 * (24_959 + 161)
    assert nc.nd_sparse_workspace_bytes(1 << 28, 1 << 22) >= (1 << 28) // 8 + (1 << 22)
    assert nc.status_string(0) == "NC_OK" and nc.status_string(-2) == "NC_ERR_ALIGN"


def _scratch_address():
    """An address for pointer arguments that validation must reject before any launch.  On a
    box with a GPU it is real device memory (2 MiB, far more than any size used below), so a
    check that stopped working shows up as a wrong status, not as a fault on the device; without
    a GPU it is a made-up, well-aligned number that nothing dereferences."""
    import torch
    if torch.cuda.is_available():
        buf = torch.zeros(2 << 20, dtype=torch.uint8, device="cuda")
        return buf, (buf.data_ptr() + 255) & ~255
    return None, 1 << 20


def test_argument_validation_needs_no_gpu(nc):
    lib = nc.lib
    keep_alive, A = _scratch_address()
    u32 = (C.c_uint32 * 1)(0)
    one = (C.c_void_p * 1)(A)
    null = (C.c_void_p * 1)(0)

    def st(v):
        return nc.status_string(v)

    assert st(lib.nc_compress(None, 8, 0, 0, A, A, None)) == "NC_ERR_INVALID"
    assert st(lib.nc_compress(A, 8, 0, 0, None, A, None)) == "NC_ERR_INVALID"
    assert st(lib.nc_compress(A + 16, 8, 0, 0, A, A, None)) == "NC_ERR_ALIGN"
    assert st(lib.nc_compress(A, 8, 0, 0, A + 8, A, None)) == "NC_ERR_ALIGN"
    assert st(lib.nc_compress(A, 0, 0, 0, A, A, None)) == "NC_OK"          # d = 0: no launch
    assert st(lib.nc_compress_batch(one, 8, 0, u32, one, one, 0, None)) == "NC_ERR_INVALID"
    assert st(lib.nc_compress_batch(one, 8, 0, u32, one, one, 65, None)) == "NC_ERR_INVALID"
    assert st(lib.nc_aggregate(null, one, 1, 8, A, None)) == "NC_ERR_INVALID"
    assert st(lib.nc_aggregate(one, one, 1, 8, A + 4, None)) == "NC_ERR_ALIGN"
    assert st(lib.nc_aggregate(one, one, 1, 0, A, None)) == "NC_OK"
    assert st(lib.nc_decode_accumulate(A, A, 8, None, None)) == "NC_ERR_INVALID"
    assert st(lib.nc_sum_fp32(one, 0, 8, A, None)) == "NC_ERR_INVALID"
    # dithering: p, s, workspace
    args = dict(x=A, d=64, off=A, B=1, p=2, s=8, seed=0, worker=0, norms=A, level=A, sign=A,
                ws=A, ws_bytes=1 << 20)

    def nd(**kw):
        a = dict(args, **kw)
        return st(lib.nd_compress(C.c_void_p(a["x"]), C.c_size_t(a["d"]), C.c_void_p(a["off"]),
                                  a["B"], a["p"], a["s"], C.c_uint64(a["seed"]), a["worker"],
                                  C.c_void_p(a["norms"]), C.c_void_p(a["level"]),
                                  C.c_void_p(a["sign"]), C.c_void_p(a["ws"]),
                                  C.c_size_t(a["ws_bytes"]), C.c_void_p(a.get("status", 0)), None))

    assert nd(p=3) == "NC_ERR_UNSUPPORTED"
    assert nd(s=0) == "NC_ERR_INVALID" and nd(s=16) == "NC_ERR_INVALID"
    assert nd(B=0) == "NC_ERR_INVALID"
    assert nd(ws_bytes=8) == "NC_ERR_WORKSPACE"
    assert nd(x=A + 16) == "NC_ERR_ALIGN"
    assert nd(d=0) == "NC_OK"
    assert nd(status=A + 2) == "NC_ERR_ALIGN"
    assert st(lib.nd_norm_status(one, 1, 4, None, None)) == "NC_ERR_INVALID"
    assert st(lib.nd_norm_status(null, 1, 4, C.c_void_p(A), None)) == "NC_ERR_INVALID"
    assert st(lib.nd_norm_status(one, 1, 0, C.c_void_p(A), None)) == "NC_OK"      # B = 0: no launch
    raw = C.CDLL(nc.LIB_PATH)          # a separate handle: the binding's prototypes stay as set
    r = raw.nd_sparse_compress(C.c_void_p(A), C.c_size_t(64), C.c_uint64((1 << 32) + 1),
                               C.c_float(1.0), 0, 4, C.c_uint64(0), 0, C.c_void_p(A),
                               C.c_void_p(A), C.c_void_p(A), C.c_void_p(A), C.c_size_t(64),
                               C.c_void_p(A), C.c_size_t(1 << 20), None)
    assert st(r) == "NC_ERR_INVALID"
    del keep_alive


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_1905_10988_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text
                assert "liboracle" not in text and "natcomp_oracle" not in text
