"""ctypes binding of the CPU oracle (oracle/natcomp_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg; never by the package.  Arrays are numpy, host side.
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())

_u8p = C.POINTER(C.c_uint8)
_u32p = C.POINTER(C.c_uint32)
_i32p = C.POINTER(C.c_int32)
_u64p = C.POINTER(C.c_uint64)
_f32p = C.POINTER(C.c_float)
_f64p = C.POINTER(C.c_double)

P_INF = 0  # encoding of p = infinity


def _sig(name, restype, *argtypes):
    fn = getattr(_lib, name)
    fn.restype = restype
    fn.argtypes = list(argtypes)
    return fn


_set_threads = _sig("orc_set_threads", None, C.c_int)
_max_threads = _sig("orc_max_threads", C.c_int)
_philox = _sig("orc_philox4x32_10", None, _u32p, _u32p, _u32p)
_stream_words = _sig("orc_stream_words", None, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64,
                     C.c_uint64, _u32p)
_cnat_values = _sig("orc_cnat_values", None, _f32p, _u32p, C.c_uint64, _f64p)
_cnat_codes = _sig("orc_cnat_codes", None, _f32p, _u32p, C.c_uint64, _u8p, _u8p)
_cnat_decode = _sig("orc_cnat_decode", None, _u8p, _u8p, C.c_uint64, _f32p)
_nc_compress = _sig("orc_nc_compress", None, _f32p, C.c_uint64, C.c_uint64, C.c_uint64,
                    C.c_uint32, _u8p, _u32p)
_nc_decode_accumulate = _sig("orc_nc_decode_accumulate", None, _u8p, _u32p, C.c_uint64, _f32p)
_nc_aggregate = _sig("orc_nc_aggregate", None, C.POINTER(_u8p), C.POINTER(_u32p), C.c_int,
                     C.c_uint64, _f32p)
_sum_fp32 = _sig("orc_sum_fp32", None, C.POINTER(_f32p), C.c_int, C.c_uint64, _f32p)
_norms = _sig("orc_norms", None, _f32p, _u64p, C.c_int, C.c_int, _f32p)
_nd_level_codes = _sig("orc_nd_level_codes", None, _f64p, _u32p, C.c_uint64, C.c_int, _i32p)
_nd_compress = _sig("orc_nd_compress", None, _f32p, C.c_uint64, C.c_uint64, _u64p, C.c_int,
                    C.c_int, C.c_int, C.c_uint64, C.c_uint32, C.c_uint32, C.c_int, _f32p, _u8p,
                    _u32p)
_nd_decode_accumulate = _sig("orc_nd_decode_accumulate", None, _f32p, _u8p, _u32p, C.c_uint64,
                             _u64p, C.c_int, C.c_int, _f32p)
_nd_aggregate = _sig("orc_nd_aggregate", None, C.POINTER(_f32p), C.POINTER(_u8p),
                     C.POINTER(_u32p), C.c_int, C.c_uint64, _u64p, C.c_int, C.c_int, _f32p)
_sparse_compress = _sig("orc_sparse_compress", C.c_uint64, _f32p, C.c_uint64, C.c_uint64,
                        C.c_float, C.c_int, C.c_int, C.c_uint64, C.c_uint32, _u32p, _u8p,
                        C.c_uint64, _f32p, _f32p)
_sparse_decode_accumulate = _sig("orc_sparse_decode_accumulate", None, _u32p, _u8p, C.c_uint64,
                                 C.c_float, C.c_int, _f32p)


def _arr(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _p(a, ptype):
    return a.ctypes.data_as(ptype)


def _ptr_array(arrays, ptype):
    return (ptype * len(arrays))(*[_p(a, ptype) for a in arrays])


def set_threads(t: int) -> None:
    _set_threads(int(t))


def max_threads() -> int:
    return int(_max_threads())


def philox4x32_10(ctr, key) -> np.ndarray:
    ctr = _arr(ctr, np.uint32)
    key = _arr(key, np.uint32)
    assert ctr.shape == (4,) and key.shape == (2,)
    out = np.empty(4, np.uint32)
    _philox(_p(ctr, _u32p), _p(key, _u32p), _p(out, _u32p))
    return out


def stream_words(seed: int, worker: int, domain: int, j0: int, count: int) -> np.ndarray:
    out = np.empty(count, np.uint32)
    _stream_words(seed, worker, domain, j0, count, _p(out, _u32p))
    return out


def cnat_values(t, r23) -> np.ndarray:
    t = _arr(t, np.float32)
    r23 = _arr(r23, np.uint32)
    assert t.shape == r23.shape
    out = np.empty(t.shape, np.float64)
    _cnat_values(_p(t, _f32p), _p(r23, _u32p), t.size, _p(out, _f64p))
    return out


def cnat_codes(t, r23):
    t = _arr(t, np.float32)
    r23 = _arr(r23, np.uint32)
    assert t.shape == r23.shape
    e = np.empty(t.shape, np.uint8)
    s = np.empty(t.shape, np.uint8)
    _cnat_codes(_p(t, _f32p), _p(r23, _u32p), t.size, _p(e, _u8p), _p(s, _u8p))
    return e, s


def cnat_decode(exp_bytes, sign_bits) -> np.ndarray:
    e = _arr(exp_bytes, np.uint8)
    s = _arr(sign_bits, np.uint8)
    out = np.empty(e.shape, np.float32)
    _cnat_decode(_p(e, _u8p), _p(s, _u8p), e.size, _p(out, _f32p))
    return out


def nc_compress(x, seed: int, worker: int, j0: int = 0):
    """C_nat of one worker's vector (or of the slice starting at element j0)."""
    x = _arr(x, np.float32)
    assert j0 % 32 == 0
    d = x.size
    e = np.zeros(d, np.uint8)
    s = np.zeros((d + 31) // 32, np.uint32)
    _nc_compress(_p(x, _f32p), d, j0, seed, worker, _p(e, _u8p), _p(s, _u32p))
    return e, s


def nc_decode_accumulate(exp, sign, acc) -> None:
    exp = _arr(exp, np.uint8)
    sign = _arr(sign, np.uint32)
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    _nc_decode_accumulate(_p(exp, _u8p), _p(sign, _u32p), acc.size, _p(acc, _f32p))


def nc_aggregate(exps, signs, d: int) -> np.ndarray:
    exps = [_arr(a, np.uint8) for a in exps]
    signs = [_arr(a, np.uint32) for a in signs]
    out = np.empty(d, np.float32)
    _nc_aggregate(_ptr_array(exps, _u8p), _ptr_array(signs, _u32p), len(exps), d, _p(out, _f32p))
    return out


def sum_fp32(xs) -> np.ndarray:
    xs = [_arr(a, np.float32) for a in xs]
    d = xs[0].size
    out = np.empty(d, np.float32)
    _sum_fp32(_ptr_array(xs, _f32p), len(xs), d, _p(out, _f32p))
    return out


def norms(x, bucket_off, p: int) -> np.ndarray:
    x = _arr(x, np.float32)
    off = _arr(bucket_off, np.uint64)
    out = np.empty(off.size - 1, np.float32)
    _norms(_p(x, _f32p), _p(off, _u64p), off.size - 1, p, _p(out, _f32p))
    return out


def nd_level_codes(y, r23, s: int) -> np.ndarray:
    y = _arr(y, np.float64)
    r23 = _arr(r23, np.uint32)
    assert y.shape == r23.shape
    out = np.empty(y.shape, np.int32)
    _nd_level_codes(_p(y, _f64p), _p(r23, _u32p), y.size, s, _p(out, _i32p))
    return out


def nd_compress(x, bucket_off, p: int, s: int, seed: int, worker: int, *, given_norms=None,
                domain: int = 1, j0: int = 0):
    """D_nat^{p,s}; definition mode unless given_norms is passed (given-norm mode)."""
    x = _arr(x, np.float32)
    off = _arr(bucket_off, np.uint64)
    assert j0 % 32 == 0 and 1 <= s <= 15
    d = x.size
    B = off.size - 1
    if given_norms is None:
        nrm = np.zeros(B, np.float32)
        mode = 0
    else:
        nrm = np.array(given_norms, dtype=np.float32, copy=True)
        assert nrm.size == B
        mode = 1
    level = np.zeros((d + 1) // 2, np.uint8)
    sign = np.zeros((d + 31) // 32, np.uint32)
    _nd_compress(_p(x, _f32p), d, j0, _p(off, _u64p), B, p, s, seed, worker, domain, mode,
                 _p(nrm, _f32p), _p(level, _u8p), _p(sign, _u32p))
    return nrm, level, sign


def nd_decode_accumulate(nrm, level, sign, bucket_off, s: int, acc) -> None:
    nrm = _arr(nrm, np.float32)
    level = _arr(level, np.uint8)
    sign = _arr(sign, np.uint32)
    off = _arr(bucket_off, np.uint64)
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    _nd_decode_accumulate(_p(nrm, _f32p), _p(level, _u8p), _p(sign, _u32p), acc.size,
                          _p(off, _u64p), off.size - 1, s, _p(acc, _f32p))


def nd_aggregate(nrms, levels, signs, bucket_off, s: int, d: int) -> np.ndarray:
    nrms = [_arr(a, np.float32) for a in nrms]
    levels = [_arr(a, np.uint8) for a in levels]
    signs = [_arr(a, np.uint32) for a in signs]
    off = _arr(bucket_off, np.uint64)
    out = np.zeros(d, np.float32)
    _nd_aggregate(_ptr_array(nrms, _f32p), _ptr_array(levels, _u8p), _ptr_array(signs, _u32p),
                  len(nrms), d, _p(off, _u64p), off.size - 1, s, _p(out, _f32p))
    return out


def sparse_compress(x, keep_threshold: int, scale: float, p: int, s: int, seed: int, worker: int,
                    cap=None, given_norm=None):
    """S (Bernoulli keep, threshold / 2^32) then D_nat^{p,s}; returns idx, codes, count, norm.
    given_norm replaces the oracle's own norm of the kept entries (given-norm mode)."""
    x = _arr(x, np.float32)
    assert 1 <= s <= 7
    d = x.size
    if cap is None:
        cap = d
    idx = np.zeros(cap, np.uint32)
    codes = np.zeros((cap + 1) // 2, np.uint8)
    nrm = C.c_float(0.0)
    gn = None if given_norm is None else C.byref(C.c_float(float(given_norm)))
    count = _sparse_compress(_p(x, _f32p), d, keep_threshold, scale, p, s, seed, worker,
                             _p(idx, _u32p), _p(codes, _u8p), cap, C.byref(nrm),
                             C.cast(gn, _f32p) if gn is not None else None)
    stored = min(int(count), cap)
    return idx[:stored], codes[:(stored + 1) // 2], int(count), np.float32(nrm.value)


def sparse_decode_accumulate(idx, codes, count: int, nrm, s: int, acc) -> None:
    idx = _arr(idx, np.uint32)
    codes = _arr(codes, np.uint8)
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    _sparse_decode_accumulate(_p(idx, _u32p), _p(codes, _u8p), count, float(nrm), s,
                              _p(acc, _f32p))


_dsta_level_index = _sig("orc_dsta_level_index", None, _f64p, _u32p, C.c_uint64, C.c_int, _i32p)
_dsta_apply = _sig("orc_dsta_apply", None, _f32p, C.c_uint64, C.c_int, C.c_int, C.c_uint64,
                   C.c_uint32, _f64p)


def dsta_level_index(y, r23, u: int) -> np.ndarray:
    """Standard-dithering level index (0..u) of y for explicit thresholds."""
    y = _arr(y, np.float64)
    r23 = _arr(r23, np.uint32)
    assert y.shape == r23.shape
    out = np.empty(y.shape, np.int32)
    _dsta_level_index(_p(y, _f64p), _p(r23, _u32p), y.size, u, _p(out, _i32p))
    return out


def dsta_apply(x, p: int, u: int, seed: int, worker: int) -> np.ndarray:
    """D_sta^{p,u}(x) decoded, one bucket (oracle-side comparison operator)."""
    x = _arr(x, np.float32)
    out = np.empty(x.size, np.float64)
    _dsta_apply(_p(x, _f32p), x.size, p, u, seed, worker, _p(out, _f64p))
    return out


_nc_compress_nearest = _sig("orc_nc_compress_nearest", None, _f32p, C.c_uint64, _u8p, _u32p)


def nc_compress_nearest(x):
    """Codes of x rounded to the nearest power of two (the deterministic control variant)."""
    x = _arr(x, np.float32)
    d = x.size
    e = np.zeros(d, np.uint8)
    s = np.zeros((d + 31) // 32, np.uint32)
    _nc_compress_nearest(_p(x, _f32p), d, _p(e, _u8p), _p(s, _u32p))
    return e, s


_sparse_compact_compress = _sig("orc_sparse_compact_compress", C.c_uint64, _f32p, C.c_uint64,
                                C.c_uint64, C.c_float, C.c_int, C.c_int, C.c_uint64, C.c_uint32,
                                _u32p, _u32p, C.c_uint64, _f32p)
_sparse_compact_decode_accumulate = _sig("orc_sparse_compact_decode_accumulate", None, _u32p,
                                         _u32p, C.c_uint64, C.c_float, C.c_int, _f32p)


def code_bits(s: int) -> int:
    """Bits per code of the compact sparse format: sign + ceil(log2 s)."""
    nb = 0
    while (1 << nb) < s:
        nb += 1
    return nb + 1


def sparse_compact_compress(x, keep_threshold: int, scale: float, p: int, s: int, seed: int,
                            worker: int, cap=None):
    """Sparsifier + D_nat with zero-level entries dropped; returns idx, planes, count, norm."""
    x = _arr(x, np.float32)
    d = x.size
    if cap is None:
        cap = d
    idx = np.zeros(cap, np.uint32)
    planes = np.zeros(((cap + 31) // 32) * code_bits(s), np.uint32)
    nrm = C.c_float(0.0)
    count = _sparse_compact_compress(_p(x, _f32p), d, keep_threshold, scale, p, s, seed, worker,
                                     _p(idx, _u32p), _p(planes, _u32p), cap, C.byref(nrm))
    stored = min(int(count), cap)
    return idx[:stored], planes, int(count), np.float32(nrm.value)


def sparse_compact_decode_accumulate(idx, planes, count: int, nrm, s: int, acc) -> None:
    idx = _arr(idx, np.uint32)
    planes = _arr(planes, np.uint32)
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    _sparse_compact_decode_accumulate(_p(idx, _u32p), _p(planes, _u32p), count, float(nrm), s,
                                      _p(acc, _f32p))


_i64p = C.POINTER(C.c_int64)
_nc8_compress = _sig("orc_nc8_compress", None, _f32p, C.c_uint64, C.c_uint64, C.c_uint64,
                     C.c_uint32, _u8p)
_nc8_decode = _sig("orc_nc8_decode", None, _u8p, C.c_uint64, _f32p)
_nc8_aggregate = _sig("orc_nc8_aggregate", None, C.POINTER(_u8p), C.c_int, C.c_uint64, _f32p,
                      _i64p)
_nc8_aggregate_compress = _sig("orc_nc8_aggregate_compress", None, C.POINTER(_u8p), C.c_int,
                               C.c_uint64, C.c_uint64, C.c_uint32, _u8p)


def nc8_compress(x, seed: int, worker: int, j0: int = 0) -> np.ndarray:
    """C_nat followed by the paper's 8-bit code (sign, zero flag, exponent clipped to -50..10)."""
    x = _arr(x, np.float32)
    out = np.zeros(x.size, np.uint8)
    _nc8_compress(_p(x, _f32p), x.size, j0, seed, worker, _p(out, _u8p))
    return out


def nc8_decode(code) -> np.ndarray:
    code = _arr(code, np.uint8)
    out = np.empty(code.size, np.float32)
    _nc8_decode(_p(code, _u8p), code.size, _p(out, _f32p))
    return out


def nc8_aggregate(codes, d: int):
    """Integer aggregation; returns (fp32 result, exact int64 sums)."""
    codes = [_arr(c, np.uint8) for c in codes]
    out = np.empty(d, np.float32)
    sums = np.empty(d, np.int64)
    _nc8_aggregate(_ptr_array(codes, _u8p), len(codes), d, _p(out, _f32p), _p(sums, _i64p))
    return out, sums


def nc8_aggregate_compress(codes, d: int, seed: int, master: int) -> np.ndarray:
    codes = [_arr(c, np.uint8) for c in codes]
    out = np.zeros(d, np.uint8)
    _nc8_aggregate_compress(_ptr_array(codes, _u8p), len(codes), d, seed, master, _p(out, _u8p))
    return out


_select_smallest = _sig("orc_select_smallest", None, _u32p, C.c_uint64, C.c_uint64, _u8p)
_sparse_exact_compress = _sig("orc_sparse_exact_compress", C.c_uint64, _f32p, C.c_uint64,
                              C.c_uint64, C.c_float, C.c_int, C.c_int, C.c_uint64, C.c_uint32,
                              _u32p, _u32p, C.c_uint64, _f32p, _f32p)
_topk_compress = _sig("orc_topk_compress", None, _f32p, C.c_uint64, C.c_uint64, C.c_uint64,
                      C.c_uint32, _u32p, _u8p, _u32p)
_topk_decode_accumulate = _sig("orc_topk_decode_accumulate", None, _u32p, _u8p, _u32p, C.c_uint64,
                               _f32p)


def select_smallest(keys, q: int) -> np.ndarray:
    """mask of the q smallest keys, ties to the lower index."""
    keys = _arr(keys, np.uint32)
    mask = np.zeros(keys.size, np.uint8)
    _select_smallest(_p(keys, _u32p), keys.size, q, _p(mask, _u8p))
    return mask


def sparse_exact_compress(x, q: int, scale: float, p: int, s: int, seed: int, worker: int,
                          cap=None, given_norm=None):
    """S^q with exactly q kept coordinates, then D_nat, compact form."""
    x = _arr(x, np.float32)
    d = x.size
    if cap is None:
        cap = d
    idx = np.zeros(cap, np.uint32)
    planes = np.zeros(((cap + 31) // 32) * code_bits(s), np.uint32)
    nrm = C.c_float(0.0)
    gn = None if given_norm is None else C.byref(C.c_float(float(given_norm)))
    count = _sparse_exact_compress(_p(x, _f32p), d, q, scale, p, s, seed, worker, _p(idx, _u32p),
                                   _p(planes, _u32p), cap, C.byref(nrm), gn)
    return idx[:min(int(count), cap)], planes, int(count), np.float32(nrm.value)


def topk_compress(x, K: int, seed: int, worker: int):
    """TopK by magnitude then C_nat: ascending indices, exponent bytes, sign words."""
    x = _arr(x, np.float32)
    listed = min(K, x.size)
    idx = np.zeros(listed, np.uint32)
    exp = np.zeros(listed, np.uint8)
    sign = np.zeros((listed + 31) // 32, np.uint32)
    _topk_compress(_p(x, _f32p), x.size, K, seed, worker, _p(idx, _u32p), _p(exp, _u8p),
                   _p(sign, _u32p))
    return idx, exp, sign


def topk_decode_accumulate(idx, exp, sign, acc) -> None:
    idx = _arr(idx, np.uint32)
    exp = _arr(exp, np.uint8)
    sign = _arr(sign, np.uint32)
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    _topk_decode_accumulate(_p(idx, _u32p), _p(exp, _u8p), _p(sign, _u32p), idx.size,
                            _p(acc, _f32p))


_u16p = C.POINTER(C.c_uint16)
_nc_compress_typed = _sig("orc_nc_compress_typed", None, _u16p, C.c_int, C.c_uint64, C.c_uint64,
                          C.c_uint32, _u8p, _u32p)
_values_of_16bit = _sig("orc_values_of_16bit", None, _u16p, C.c_int, C.c_uint64, _f32p)
DTYPE_BF16, DTYPE_F16 = 1, 2


def nc_compress_typed(x16, dtype: int, seed: int, worker: int):
    """C_nat of bfloat16 (dtype 1) or binary16 (dtype 2) bit patterns: exponent bytes, sign words."""
    x16 = _arr(x16, np.uint16)
    exp = np.zeros(x16.size, np.uint8)
    sign = np.zeros((x16.size + 31) // 32, np.uint32)
    _nc_compress_typed(_p(x16, _u16p), dtype, x16.size, seed, worker, _p(exp, _u8p),
                       _p(sign, _u32p))
    return exp, sign


_nc_compress_bf16_r8 = _sig("orc_nc_compress_bf16_r8", None, _u16p, C.c_uint64, C.c_uint64,
                            C.c_uint32, _u8p, _u32p)


def nc_compress_bf16_r8(x16, seed: int, worker: int):
    """C_nat of bfloat16 bit patterns with 7-bit thresholds drawn from one stream byte per entry
    (domain 4): exponent bytes, sign words."""
    x16 = _arr(x16, np.uint16)
    exp = np.zeros(x16.size, np.uint8)
    sign = np.zeros((x16.size + 31) // 32, np.uint32)
    _nc_compress_bf16_r8(_p(x16, _u16p), x16.size, seed, worker, _p(exp, _u8p), _p(sign, _u32p))
    return exp, sign


_nc_compress_f16_r16 = _sig("orc_nc_compress_f16_r16", None, _u16p, C.c_uint64, C.c_uint64,
                            C.c_uint32, _u8p, _u32p)


def nc_compress_f16_r16(x16, seed: int, worker: int):
    """C_nat of binary16 bit patterns with 10-bit thresholds drawn from one stream half-word per
    entry (domain 5): exponent bytes, sign words."""
    x16 = _arr(x16, np.uint16)
    exp = np.zeros(x16.size, np.uint8)
    sign = np.zeros((x16.size + 31) // 32, np.uint32)
    _nc_compress_f16_r16(_p(x16, _u16p), x16.size, seed, worker, _p(exp, _u8p), _p(sign, _u32p))
    return exp, sign


def values_of_16bit(x16, dtype: int) -> np.ndarray:
    x16 = _arr(x16, np.uint16)
    out = np.zeros(x16.size, np.float32)
    _values_of_16bit(_p(x16, _u16p), dtype, x16.size, _p(out, _f32p))
    return out


_u64p = C.POINTER(C.c_uint64)
_nc64_compress = _sig("orc_nc64_compress", None, _f64p, C.c_uint64, C.c_uint64, C.c_uint32, _u8p,
                      _u8p)
_nc64_aggregate = _sig("orc_nc64_aggregate", None, C.POINTER(_u8p), C.POINTER(_u8p), C.c_int,
                       C.c_uint64, _f64p)
_cnat64_values = _sig("orc_cnat64_values", None, _f64p, _u64p, C.c_uint64, _f64p)


def nc64_compress(x, seed: int, worker: int):
    """C_nat of a binary64 vector: low exponent bytes and the (sign, high exponent) nibble plane."""
    x = _arr(x, np.float64)
    exp_lo = np.zeros(x.size, np.uint8)
    hi = np.zeros((x.size + 1) // 2, np.uint8)
    _nc64_compress(_p(x, _f64p), x.size, seed, worker, _p(exp_lo, _u8p), _p(hi, _u8p))
    return exp_lo, hi


def nc64_aggregate(exp_los, his, d: int) -> np.ndarray:
    n = len(exp_los)
    exp_los = [_arr(e, np.uint8) for e in exp_los]
    his = [_arr(h, np.uint8) for h in his]
    ea = (_u8p * n)(*[_p(e, _u8p) for e in exp_los])
    ha = (_u8p * n)(*[_p(h, _u8p) for h in his])
    out = np.zeros(d, np.float64)
    _nc64_aggregate(ea, ha, n, d, _p(out, _f64p))
    return out


def cnat64_values(t, r52) -> np.ndarray:
    t = _arr(t, np.float64)
    r52 = _arr(r52, np.uint64)
    out = np.zeros(t.size, np.float64)
    _cnat64_values(_p(t, _f64p), _p(r52, _u64p), t.size, _p(out, _f64p))
    return out


_sparse_regen_decode_accumulate = _sig("orc_sparse_regen_decode_accumulate", None, _u8p,
                                       C.c_uint64, C.c_float, C.c_uint64, C.c_uint64, C.c_int,
                                       C.c_uint64, C.c_uint32, _f32p)


def sparse_regen_decode_accumulate(codes, count: int, nrm, keep_threshold: int, s: int, seed: int,
                                   worker: int, acc) -> None:
    """Apply the listed 4-bit codes to the kept coordinates regenerated from the seed."""
    codes = _arr(codes, np.uint8)
    assert acc.dtype == np.float32 and acc.flags.c_contiguous
    _sparse_regen_decode_accumulate(_p(codes, _u8p), count, float(nrm), acc.size, keep_threshold, s,
                                    seed, worker, _p(acc, _f32p))
