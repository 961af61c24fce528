"""Thin ctypes binding of libnatcomp.so: argument marshalling only.

Every function has the name and the argument order of its C entry point
(include/natcomp.h).  Tensors are torch CUDA tensors used as device memory; the
binding passes their pointers and the current CUDA stream and raises NatcompError
on a non-zero status.  There is no CPU fallback: without the built library the
import fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnatcomp.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libnatcomp.so is not built; run `python paper_1905_10988_b200/build.py` "
        "(needs nvcc; targets sm_100a).  There is no CPU fallback.")

lib = C.CDLL(LIB_PATH)

NC_MAX_WORKERS = 64
P_INF = 0

EXPORTS = (
    "nc_status_string", "nc_exp_bytes", "nc_sign_bytes", "nd_level_bytes", "nd_workspace_bytes",
    "nd_sparse_workspace_bytes", "nc_compress", "nc_compress_batch", "nc_decode_accumulate",
    "nc_aggregate", "nc_sum_fp32", "nd_compress", "nd_decode_accumulate", "nd_aggregate",
    "nd_sparse_compress", "nd_sparse_decode_accumulate", "nc_copy_to_device", "nc_copy_to_host",
    "nd_batch_workspace_bytes", "nd_compress_batch", "nd_sparse_batch_workspace_bytes",
    "nd_sparse_compress_batch", "nd_static_scratch_bytes", "nd_compress_static",
    "nc_aggregate_compress", "nc_compress_nearest", "nc_compress_nearest_batch",
    "nd_sparse_plane_bytes", "nd_sparse_compact_compress", "nd_sparse_compact_compress_batch",
    "nd_sparse_compact_decode_accumulate", "nc8_compress", "nc8_compress_batch", "nc8_aggregate",
    "nc8_aggregate_compress", "nc_select_workspace_bytes", "nd_sparse_exact_compress",
    "nc_topk_compress", "nc_topk_decode_accumulate", "nc_compress_typed",
    "nc_compress_typed_batch", "nc64_compress", "nc64_compress_batch", "nc64_aggregate",
    "nd_sparse_regen_workspace_bytes", "nd_sparse_regen_decode_accumulate",
    "nd_sparse_compact_aggregate", "nc_aggregate_compress_shard", "nc_compress_bf16_r8",
    "nc_compress_bf16_r8_batch", "nc_compress_f16_r16", "nc_compress_f16_r16_batch",
    "nd_norm_status", "nd_norms_batch", "nd_round_batch", "nc_debug_bounds_status",
    "nc_debug_bounds_selftest",
)


class NatcompError(RuntimeError):
    def __init__(self, fn: str, status: int):
        super().__init__("%s failed: %s (%d)" % (fn, status_string(status), status))
        self.status = status


_vp = C.c_void_p
_sz = C.c_size_t


def _sig(name, restype, *argtypes):
    fn = getattr(lib, name)
    fn.restype = restype
    fn.argtypes = list(argtypes)
    return fn


_status_string = _sig("nc_status_string", C.c_char_p, C.c_int)
_nc_exp_bytes = _sig("nc_exp_bytes", _sz, _sz)
_nc_sign_bytes = _sig("nc_sign_bytes", _sz, _sz)
_nd_level_bytes = _sig("nd_level_bytes", _sz, _sz)
_nd_workspace_bytes = _sig("nd_workspace_bytes", _sz, _sz, C.c_int)
_nd_sparse_workspace_bytes = _sig("nd_sparse_workspace_bytes", _sz, _sz, _sz)
_nc_compress = _sig("nc_compress", C.c_int, _vp, _sz, C.c_uint64, C.c_uint32, _vp, _vp, _vp)
_nc_compress_batch = _sig("nc_compress_batch", C.c_int, C.POINTER(_vp), _sz, C.c_uint64,
                          C.POINTER(C.c_uint32), C.POINTER(_vp), C.POINTER(_vp), C.c_int, _vp)
_nc_decode_accumulate = _sig("nc_decode_accumulate", C.c_int, _vp, _vp, _sz, _vp, _vp)
_nc_aggregate = _sig("nc_aggregate", C.c_int, C.POINTER(_vp), C.POINTER(_vp), C.c_int, _sz, _vp,
                     _vp)
_nc_sum_fp32 = _sig("nc_sum_fp32", C.c_int, C.POINTER(_vp), C.c_int, _sz, _vp, _vp)
_nd_compress = _sig("nd_compress", C.c_int, _vp, _sz, _vp, C.c_int, C.c_int, C.c_int, C.c_uint64,
                    C.c_uint32, _vp, _vp, _vp, _vp, _sz, _vp, _vp)
_nd_decode_accumulate = _sig("nd_decode_accumulate", C.c_int, _vp, _vp, _vp, _sz, _vp, C.c_int,
                             C.c_int, _vp, _vp)
_nd_aggregate = _sig("nd_aggregate", C.c_int, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp),
                     C.c_int, _sz, _vp, C.c_int, C.c_int, _vp, _vp)
_nd_sparse_compress = _sig("nd_sparse_compress", C.c_int, _vp, _sz, C.c_uint64, C.c_float,
                           C.c_int, C.c_int, C.c_uint64, C.c_uint32, _vp, _vp, _vp, _vp, _sz,
                           _vp, _sz, _vp)
_nd_sparse_decode_accumulate = _sig("nd_sparse_decode_accumulate", C.c_int, _vp, _vp, _vp, _vp,
                                    C.c_int, _sz, _sz, _vp, _vp)


_nd_batch_workspace_bytes = _sig("nd_batch_workspace_bytes", _sz, _sz, C.c_int, C.c_int)
_nd_compress_batch = _sig("nd_compress_batch", C.c_int, C.POINTER(_vp), _sz, _vp, C.c_int, C.c_int,
                          C.c_int, C.c_uint64, C.POINTER(C.c_uint32), C.POINTER(_vp),
                          C.POINTER(_vp), C.POINTER(_vp), C.c_int, _vp, _sz, _vp, _vp)
_nd_norm_status = _sig("nd_norm_status", C.c_int, C.POINTER(_vp), C.c_int, C.c_int, _vp, _vp)
_nd_sparse_batch_workspace_bytes = _sig("nd_sparse_batch_workspace_bytes", _sz, _sz, _sz, C.c_int)
_nd_sparse_compress_batch = _sig("nd_sparse_compress_batch", C.c_int, C.POINTER(_vp), _sz,
                                 C.c_uint64, C.c_float, C.c_int, C.c_int, C.c_uint64,
                                 C.POINTER(C.c_uint32), C.POINTER(_vp), C.POINTER(_vp),
                                 C.POINTER(_vp), C.POINTER(_vp), _sz, C.c_int, _vp, _sz, _vp)


def nd_batch_workspace_bytes(d: int, num_buckets: int, n: int) -> int:
    return int(_nd_batch_workspace_bytes(d, num_buckets, n))


def nd_compress_batch(xs, d, bucket_off, B, p, s, seed, workers, norms, levels, signs, n,
                      workspace, workspace_bytes, stream=None, status=None) -> None:
    """status (the C argument before the stream; optional): device uint32 that the call
    increments once per bucket whose norm is inf or NaN."""
    w = (C.c_uint32 * n)(*[int(v) for v in workers])
    _check("nd_compress_batch", _nd_compress_batch(_ptrs(xs), d, _ptr(bucket_off), B, p, s, seed,
                                                   w, _ptrs(norms), _ptrs(levels), _ptrs(signs),
                                                   n, _ptr(workspace), workspace_bytes,
                                                   _ptr(status), _stream(stream)))


_nd_norms_batch = _sig("nd_norms_batch", C.c_int, C.POINTER(_vp), _sz, _vp, C.c_int, C.c_int,
                       C.POINTER(_vp), C.c_int, _vp, _sz, _vp, _vp)
_nd_round_batch = _sig("nd_round_batch", C.c_int, C.POINTER(_vp), _sz, _vp, C.c_int, C.c_int,
                       C.c_uint64, C.POINTER(C.c_uint32), C.POINTER(_vp), C.POINTER(_vp),
                       C.POINTER(_vp), C.c_int, _vp)


def nd_norms_batch(xs, d, bucket_off, B, p, norms, n, workspace, workspace_bytes, stream=None,
                   status=None) -> None:
    _check("nd_norms_batch", _nd_norms_batch(_ptrs(xs), d, _ptr(bucket_off), B, p, _ptrs(norms), n,
                                             _ptr(workspace), workspace_bytes, _ptr(status),
                                             _stream(stream)))


def nd_round_batch(xs, d, bucket_off, B, s, seed, workers, norms, levels, signs, n,
                   stream=None) -> None:
    w = (C.c_uint32 * n)(*[int(v) for v in workers])
    _check("nd_round_batch", _nd_round_batch(_ptrs(xs), d, _ptr(bucket_off), B, s, seed, w,
                                             _ptrs(norms), _ptrs(levels), _ptrs(signs), n,
                                             _stream(stream)))


def nd_norm_status(norms, n, B, status, stream=None) -> None:
    _check("nd_norm_status", _nd_norm_status(_ptrs(norms), n, B, _ptr(status), _stream(stream)))


def nd_sparse_batch_workspace_bytes(d: int, cap: int, n: int) -> int:
    return int(_nd_sparse_batch_workspace_bytes(d, cap, n))


def nd_sparse_compress_batch(xs, d, keep_threshold, scale, p, s, seed, workers, idxs, codes,
                             counts, norms, cap, n, workspace, workspace_bytes,
                             stream=None) -> None:
    w = (C.c_uint32 * n)(*[int(v) for v in workers])
    _check("nd_sparse_compress_batch",
           _nd_sparse_compress_batch(_ptrs(xs), d, keep_threshold, scale, p, s, seed, w,
                                     _ptrs(idxs), _ptrs(codes), _ptrs(counts), _ptrs(norms), cap,
                                     n, _ptr(workspace), workspace_bytes, _stream(stream)))


_nc_aggregate_compress = _sig("nc_aggregate_compress", C.c_int, C.POINTER(_vp), C.POINTER(_vp),
                              C.c_int, _sz, C.c_uint64, C.c_uint32, _vp, _vp, _vp)


def nc_aggregate_compress(exps, signs, n, d, seed, master, out_exp, out_sign, stream=None) -> None:
    _check("nc_aggregate_compress",
           _nc_aggregate_compress(_ptrs(exps), _ptrs(signs), n, d, seed, master, _ptr(out_exp),
                                  _ptr(out_sign), _stream(stream)))


_nc_aggregate_compress_shard = _sig("nc_aggregate_compress_shard", C.c_int, C.POINTER(_vp),
                                    C.POINTER(_vp), C.c_int, _sz, C.c_uint64, C.c_uint64,
                                    C.c_uint32, _vp, _vp, _vp)


def nc_aggregate_compress_shard(exps, signs, n, d, first_index, seed, master, out_exp, out_sign,
                                stream=None) -> None:
    _check("nc_aggregate_compress_shard",
           _nc_aggregate_compress_shard(_ptrs(exps), _ptrs(signs), n, d, first_index, seed,
                                        master, _ptr(out_exp), _ptr(out_sign), _stream(stream)))


_nc_compress_bf16_r8 = _sig("nc_compress_bf16_r8", C.c_int, _vp, _sz, C.c_uint64, C.c_uint32, _vp,
                            _vp, _vp)
_nc_compress_bf16_r8_batch = _sig("nc_compress_bf16_r8_batch", C.c_int, C.POINTER(_vp), _sz,
                                  C.c_uint64, C.POINTER(C.c_uint32), C.POINTER(_vp),
                                  C.POINTER(_vp), C.c_int, _vp)


def nc_compress_bf16_r8(x, d, seed, worker, exp, sign, stream=None) -> None:
    _check("nc_compress_bf16_r8",
           _nc_compress_bf16_r8(_ptr(x), d, seed, worker, _ptr(exp), _ptr(sign), _stream(stream)))


def nc_compress_bf16_r8_batch(xs, d, seed, workers, exps, signs, n, stream=None) -> None:
    w = (C.c_uint32 * n)(*[int(v) for v in workers])
    _check("nc_compress_bf16_r8_batch",
           _nc_compress_bf16_r8_batch(_ptrs(xs), d, seed, w, _ptrs(exps), _ptrs(signs), n,
                                      _stream(stream)))


_nc_compress_f16_r16 = _sig("nc_compress_f16_r16", C.c_int, _vp, _sz, C.c_uint64, C.c_uint32, _vp,
                            _vp, _vp)
_nc_compress_f16_r16_batch = _sig("nc_compress_f16_r16_batch", C.c_int, C.POINTER(_vp), _sz,
                                  C.c_uint64, C.POINTER(C.c_uint32), C.POINTER(_vp),
                                  C.POINTER(_vp), C.c_int, _vp)


def nc_compress_f16_r16(x, d, seed, worker, exp, sign, stream=None) -> None:
    _check("nc_compress_f16_r16",
           _nc_compress_f16_r16(_ptr(x), d, seed, worker, _ptr(exp), _ptr(sign), _stream(stream)))


def nc_compress_f16_r16_batch(xs, d, seed, workers, exps, signs, n, stream=None) -> None:
    w = (C.c_uint32 * n)(*[int(v) for v in workers])
    _check("nc_compress_f16_r16_batch",
           _nc_compress_f16_r16_batch(_ptrs(xs), d, seed, w, _ptrs(exps), _ptrs(signs), n,
                                      _stream(stream)))


_nc_compress_nearest = _sig("nc_compress_nearest", C.c_int, _vp, _sz, _vp, _vp, _vp)
_nc_compress_nearest_batch = _sig("nc_compress_nearest_batch", C.c_int, C.POINTER(_vp), _sz,
                                  C.POINTER(_vp), C.POINTER(_vp), C.c_int, _vp)


def nc_compress_nearest(x, d, exp, sign, stream=None) -> None:
    _check("nc_compress_nearest", _nc_compress_nearest(_ptr(x), d, _ptr(exp), _ptr(sign),
                                                       _stream(stream)))


def nc_compress_nearest_batch(xs, d, exps, signs, n, stream=None) -> None:
    _check("nc_compress_nearest_batch",
           _nc_compress_nearest_batch(_ptrs(xs), d, _ptrs(exps), _ptrs(signs), n,
                                      _stream(stream)))


_nd_sparse_plane_bytes = _sig("nd_sparse_plane_bytes", _sz, _sz, C.c_int)
_nd_sparse_compact_compress = _sig("nd_sparse_compact_compress", C.c_int, _vp, _sz, C.c_uint64,
                                   C.c_float, C.c_int, C.c_int, C.c_uint64, C.c_uint32, _vp, _vp,
                                   _vp, _vp, _sz, _vp, _sz, _vp)
_nd_sparse_compact_compress_batch = _sig("nd_sparse_compact_compress_batch", C.c_int,
                                         C.POINTER(_vp), _sz, C.c_uint64, C.c_float, C.c_int,
                                         C.c_int, C.c_uint64, C.POINTER(C.c_uint32),
                                         C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp),
                                         C.POINTER(_vp), _sz, C.c_int, _vp, _sz, _vp)
_nd_sparse_compact_decode_accumulate = _sig("nd_sparse_compact_decode_accumulate", C.c_int, _vp,
                                            _vp, _vp, _vp, C.c_int, _sz, _sz, _vp, _vp)


def nd_sparse_plane_bytes(cap: int, s: int) -> int:
    return int(_nd_sparse_plane_bytes(cap, s))


def nd_sparse_compact_compress(x, d, keep_threshold, scale, p, s, seed, worker, idx, planes, count,
                               norm, cap, workspace, workspace_bytes, stream=None) -> None:
    _check("nd_sparse_compact_compress",
           _nd_sparse_compact_compress(_ptr(x), d, keep_threshold, scale, p, s, seed, worker,
                                       _ptr(idx), _ptr(planes), _ptr(count), _ptr(norm), cap,
                                       _ptr(workspace), workspace_bytes, _stream(stream)))


def nd_sparse_compact_compress_batch(xs, d, keep_threshold, scale, p, s, seed, workers, idxs,
                                     planes, counts, norms, cap, n, workspace, workspace_bytes,
                                     stream=None) -> None:
    w = (C.c_uint32 * n)(*[int(v) for v in workers])
    _check("nd_sparse_compact_compress_batch",
           _nd_sparse_compact_compress_batch(_ptrs(xs), d, keep_threshold, scale, p, s, seed, w,
                                             _ptrs(idxs), _ptrs(planes), _ptrs(counts),
                                             _ptrs(norms), cap, n, _ptr(workspace),
                                             workspace_bytes, _stream(stream)))


def nd_sparse_compact_decode_accumulate(idx, planes, count, norm, s, d, cap, acc,
                                        stream=None) -> None:
    _check("nd_sparse_compact_decode_accumulate",
           _nd_sparse_compact_decode_accumulate(_ptr(idx), _ptr(planes), _ptr(count), _ptr(norm),
                                                s, d, cap, _ptr(acc), _stream(stream)))


_nc8_compress = _sig("nc8_compress", C.c_int, _vp, _sz, C.c_uint64, C.c_uint32, _vp, _vp)
_nc8_compress_batch = _sig("nc8_compress_batch", C.c_int, C.POINTER(_vp), _sz, C.c_uint64,
                           C.POINTER(C.c_uint32), C.POINTER(_vp), C.c_int, _vp)
_nc8_aggregate = _sig("nc8_aggregate", C.c_int, C.POINTER(_vp), C.c_int, _sz, _vp, _vp)
_nc8_aggregate_compress = _sig("nc8_aggregate_compress", C.c_int, C.POINTER(_vp), C.c_int, _sz,
                               C.c_uint64, C.c_uint32, _vp, _vp)


def nc8_compress(x, d, seed, worker, code, stream=None) -> None:
    _check("nc8_compress", _nc8_compress(_ptr(x), d, seed, worker, _ptr(code), _stream(stream)))


def nc8_compress_batch(xs, d, seed, workers, codes, n, stream=None) -> None:
    w = (C.c_uint32 * n)(*[int(v) for v in workers])
    _check("nc8_compress_batch", _nc8_compress_batch(_ptrs(xs), d, seed, w, _ptrs(codes), n,
                                                     _stream(stream)))


def nc8_aggregate(codes, n, d, out, stream=None) -> None:
    _check("nc8_aggregate", _nc8_aggregate(_ptrs(codes), n, d, _ptr(out), _stream(stream)))


def nc8_aggregate_compress(codes, n, d, seed, master, out_code, stream=None) -> None:
    _check("nc8_aggregate_compress",
           _nc8_aggregate_compress(_ptrs(codes), n, d, seed, master, _ptr(out_code),
                                   _stream(stream)))


_nd_static_scratch_bytes = _sig("nd_static_scratch_bytes", _sz)
_nd_compress_static = _sig("nd_compress_static", C.c_int, _vp, _sz, _vp, C.c_int, C.c_int,
                           C.c_int, C.c_uint64, C.c_uint32, _vp, _vp, _vp, _vp, _vp)


def nd_static_scratch_bytes() -> int:
    return int(_nd_static_scratch_bytes())


def nd_compress_static(x, d, bucket_off, B, p, s, seed, worker, norms, level, sign,
                       stream=None, status=None) -> None:
    """nd_compress with the library's built-in scratch array instead of a workspace argument:
    for callers that may not allocate device memory.  Raises NatcompError(NC_ERR_TOO_LARGE) when
    nd_workspace_bytes(d, B) exceeds nd_static_scratch_bytes().  Calls on one device share the
    scratch, so they must not overlap on the GPU."""
    _check("nd_compress_static", _nd_compress_static(_ptr(x), d, _ptr(bucket_off), B, p, s, seed,
                                                     worker, _ptr(norms), _ptr(level), _ptr(sign),
                                                     _ptr(status), _stream(stream)))


_nc_debug_bounds_status = _sig("nc_debug_bounds_status", C.c_int, C.POINTER(C.c_uint64),
                               C.POINTER(C.c_uint64), C.c_int)
_nc_debug_bounds_selftest = _sig("nc_debug_bounds_selftest", C.c_int, _vp, _vp)


def nc_debug_bounds_status(reset: bool = False):
    """(violations, first_address) of the debug build; the regular library raises
    NatcompError(NC_ERR_UNSUPPORTED)."""
    v, a = C.c_uint64(0), C.c_uint64(0)
    _check("nc_debug_bounds_status", _nc_debug_bounds_status(C.byref(v), C.byref(a), int(reset)))
    return int(v.value), int(a.value)


def nc_debug_bounds_selftest(scratch, stream=None) -> None:
    _check("nc_debug_bounds_selftest", _nc_debug_bounds_selftest(_ptr(scratch), _stream(stream)))


_nc_copy_to_device = _sig("nc_copy_to_device", C.c_int, _vp, _vp, _sz, _vp)
_nc_copy_to_host = _sig("nc_copy_to_host", C.c_int, _vp, _vp, _sz, _vp)


def nc_copy_to_device(dst_device, src_host, nbytes, stream=None) -> None:
    _check("nc_copy_to_device", _nc_copy_to_device(_ptr(dst_device), _ptr(src_host), nbytes,
                                                   _stream(stream)))


def nc_copy_to_host(dst_host, src_device, nbytes, stream=None) -> None:
    _check("nc_copy_to_host", _nc_copy_to_host(_ptr(dst_host), _ptr(src_device), nbytes,
                                               _stream(stream)))


def status_string(status: int) -> str:
    return _status_string(int(status)).decode()


def _ptr(t) -> int:
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _ptrs(ts: Sequence):
    return (_vp * len(ts))(*[_ptr(t) for t in ts])


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(fn: str, status: int) -> None:
    if status != 0:
        raise NatcompError(fn, status)


# ---- sizes ---------------------------------------------------------------------------
def nc_exp_bytes(d: int) -> int:
    return int(_nc_exp_bytes(d))


def nc_sign_bytes(d: int) -> int:
    return int(_nc_sign_bytes(d))


def nd_level_bytes(d: int) -> int:
    return int(_nd_level_bytes(d))


def nd_workspace_bytes(d: int, num_buckets: int) -> int:
    return int(_nd_workspace_bytes(d, num_buckets))


def nd_sparse_workspace_bytes(d: int, cap: int) -> int:
    return int(_nd_sparse_workspace_bytes(d, cap))


# ---- C_nat ---------------------------------------------------------------------------
def nc_compress(x, d, seed, worker, exp, sign, stream=None) -> None:
    _check("nc_compress", _nc_compress(_ptr(x), d, seed, worker, _ptr(exp), _ptr(sign),
                                       _stream(stream)))


def nc_compress_batch(xs, d, seed, workers, exps, signs, n, stream=None) -> None:
    w = (C.c_uint32 * n)(*[int(v) for v in workers])
    _check("nc_compress_batch", _nc_compress_batch(_ptrs(xs), d, seed, w, _ptrs(exps),
                                                   _ptrs(signs), n, _stream(stream)))


def nc_decode_accumulate(exp, sign, d, acc, stream=None) -> None:
    _check("nc_decode_accumulate", _nc_decode_accumulate(_ptr(exp), _ptr(sign), d, _ptr(acc),
                                                         _stream(stream)))


def nc_aggregate(exps, signs, n, d, out, stream=None) -> None:
    _check("nc_aggregate", _nc_aggregate(_ptrs(exps), _ptrs(signs), n, d, _ptr(out),
                                         _stream(stream)))


def nc_sum_fp32(xs, n, d, out, stream=None) -> None:
    _check("nc_sum_fp32", _nc_sum_fp32(_ptrs(xs), n, d, _ptr(out), _stream(stream)))


# ---- D_nat ---------------------------------------------------------------------------
def nd_compress(x, d, bucket_off, B, p, s, seed, worker, norms, level, sign, workspace,
                workspace_bytes, stream=None, status=None) -> None:
    _check("nd_compress", _nd_compress(_ptr(x), d, _ptr(bucket_off), B, p, s, seed, worker,
                                       _ptr(norms), _ptr(level), _ptr(sign), _ptr(workspace),
                                       workspace_bytes, _ptr(status), _stream(stream)))


def nd_decode_accumulate(norms, level, sign, d, bucket_off, B, s, acc, stream=None) -> None:
    _check("nd_decode_accumulate", _nd_decode_accumulate(_ptr(norms), _ptr(level), _ptr(sign), d,
                                                         _ptr(bucket_off), B, s, _ptr(acc),
                                                         _stream(stream)))


def nd_aggregate(norms, levels, signs, n, d, bucket_off, B, s, out, stream=None) -> None:
    _check("nd_aggregate", _nd_aggregate(_ptrs(norms), _ptrs(levels), _ptrs(signs), n, d,
                                         _ptr(bucket_off), B, s, _ptr(out), _stream(stream)))


# ---- sparsifier composed with D_nat ----------------------------------------------------
def nd_sparse_compress(x, d, keep_threshold, scale, p, s, seed, worker, idx, codes, count, norm,
                       cap, workspace, workspace_bytes, stream=None) -> None:
    _check("nd_sparse_compress", _nd_sparse_compress(_ptr(x), d, keep_threshold, scale, p, s,
                                                     seed, worker, _ptr(idx), _ptr(codes),
                                                     _ptr(count), _ptr(norm), cap,
                                                     _ptr(workspace), workspace_bytes,
                                                     _stream(stream)))


def nd_sparse_decode_accumulate(idx, codes, count, norm, s, d, cap, acc, stream=None) -> None:
    _check("nd_sparse_decode_accumulate",
           _nd_sparse_decode_accumulate(_ptr(idx), _ptr(codes), _ptr(count), _ptr(norm), s, d,
                                        cap, _ptr(acc), _stream(stream)))


# ---- exactly q kept coordinates (S^q then D_nat) and TopK then C_nat ----------------------
_nc_select_workspace_bytes = _sig("nc_select_workspace_bytes", _sz, _sz, _sz)
_nd_sparse_exact_compress = _sig("nd_sparse_exact_compress", C.c_int, _vp, _sz, C.c_uint64,
                                 C.c_float, C.c_int, C.c_int, C.c_uint64, C.c_uint32, _vp, _vp,
                                 _vp, _vp, _sz, _vp, _sz, _vp)
_nc_topk_compress = _sig("nc_topk_compress", C.c_int, _vp, _sz, C.c_uint64, C.c_uint64,
                         C.c_uint32, _vp, _vp, _vp, _vp, _sz, _vp)
_nc_topk_decode_accumulate = _sig("nc_topk_decode_accumulate", C.c_int, _vp, _vp, _vp, _sz, _sz,
                                  _vp, _vp)


def nc_select_workspace_bytes(d: int, cap: int) -> int:
    return int(_nc_select_workspace_bytes(d, cap))


def nd_sparse_exact_compress(x, d, q, scale, p, s, seed, worker, idx, planes, count, norm, cap,
                             workspace, workspace_bytes, stream=None) -> None:
    _check("nd_sparse_exact_compress",
           _nd_sparse_exact_compress(_ptr(x), d, q, scale, p, s, seed, worker, _ptr(idx),
                                     _ptr(planes), _ptr(count), _ptr(norm), cap, _ptr(workspace),
                                     workspace_bytes, _stream(stream)))


def nc_topk_compress(x, d, K, seed, worker, idx, exp, sign, workspace, workspace_bytes,
                     stream=None) -> None:
    _check("nc_topk_compress",
           _nc_topk_compress(_ptr(x), d, K, seed, worker, _ptr(idx), _ptr(exp), _ptr(sign),
                             _ptr(workspace), workspace_bytes, _stream(stream)))


def nc_topk_decode_accumulate(idx, exp, sign, count, d, acc, stream=None) -> None:
    _check("nc_topk_decode_accumulate",
           _nc_topk_decode_accumulate(_ptr(idx), _ptr(exp), _ptr(sign), count, d, _ptr(acc),
                                      _stream(stream)))


# ---- 16-bit inputs ----------------------------------------------------------------------------
DTYPE_F32, DTYPE_BF16, DTYPE_F16 = 0, 1, 2
_nc_compress_typed = _sig("nc_compress_typed", C.c_int, _vp, C.c_int, _sz, C.c_uint64, C.c_uint32,
                          _vp, _vp, _vp)
_nc_compress_typed_batch = _sig("nc_compress_typed_batch", C.c_int, C.POINTER(_vp), C.c_int, _sz,
                                C.c_uint64, C.POINTER(C.c_uint32), C.POINTER(_vp), C.POINTER(_vp),
                                C.c_int, _vp)


def nc_compress_typed(x, dtype, d, seed, worker, exp, sign, stream=None) -> None:
    _check("nc_compress_typed", _nc_compress_typed(_ptr(x), dtype, d, seed, worker, _ptr(exp),
                                                   _ptr(sign), _stream(stream)))


def nc_compress_typed_batch(xs, dtype, d, seed, workers, exps, signs, n, stream=None) -> None:
    w = (C.c_uint32 * n)(*[int(v) for v in workers])
    _check("nc_compress_typed_batch",
           _nc_compress_typed_batch(_ptrs(xs), dtype, d, seed, w, _ptrs(exps), _ptrs(signs), n,
                                    _stream(stream)))


# ---- binary64 inputs: 12-bit codes ------------------------------------------------------------
_nc64_compress = _sig("nc64_compress", C.c_int, _vp, _sz, C.c_uint64, C.c_uint32, _vp, _vp, _vp)
_nc64_compress_batch = _sig("nc64_compress_batch", C.c_int, C.POINTER(_vp), _sz, C.c_uint64,
                            C.POINTER(C.c_uint32), C.POINTER(_vp), C.POINTER(_vp), C.c_int, _vp)
_nc64_aggregate = _sig("nc64_aggregate", C.c_int, C.POINTER(_vp), C.POINTER(_vp), C.c_int, _sz,
                       _vp, _vp)


def nc64_compress(x, d, seed, worker, exp_lo, hi, stream=None) -> None:
    _check("nc64_compress", _nc64_compress(_ptr(x), d, seed, worker, _ptr(exp_lo), _ptr(hi),
                                           _stream(stream)))


def nc64_compress_batch(xs, d, seed, workers, exp_los, his, n, stream=None) -> None:
    w = (C.c_uint32 * n)(*[int(v) for v in workers])
    _check("nc64_compress_batch",
           _nc64_compress_batch(_ptrs(xs), d, seed, w, _ptrs(exp_los), _ptrs(his), n,
                                _stream(stream)))


def nc64_aggregate(exp_los, his, n, d, out, stream=None) -> None:
    _check("nc64_aggregate", _nc64_aggregate(_ptrs(exp_los), _ptrs(his), n, d, _ptr(out),
                                             _stream(stream)))


# ---- sparse update without an index list (kept set regenerated from the seed) -----------------
_nd_sparse_regen_workspace_bytes = _sig("nd_sparse_regen_workspace_bytes", _sz, _sz)
_nd_sparse_regen_decode_accumulate = _sig("nd_sparse_regen_decode_accumulate", C.c_int, _vp, _vp,
                                          _vp, _sz, C.c_uint64, C.c_int, C.c_uint64, C.c_uint32,
                                          _sz, _vp, _vp, _sz, _vp)


def nd_sparse_regen_workspace_bytes(d: int) -> int:
    return int(_nd_sparse_regen_workspace_bytes(d))


def nd_sparse_regen_decode_accumulate(codes, count, norm, d, keep_threshold, s, seed, worker, cap,
                                      acc, workspace, workspace_bytes, stream=None) -> None:
    _check("nd_sparse_regen_decode_accumulate",
           _nd_sparse_regen_decode_accumulate(_ptr(codes), _ptr(count), _ptr(norm), d,
                                              keep_threshold, s, seed, worker, cap, _ptr(acc),
                                              _ptr(workspace), workspace_bytes, _stream(stream)))


_nd_sparse_compact_aggregate = _sig("nd_sparse_compact_aggregate", C.c_int, C.POINTER(_vp),
                                    C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp), C.c_int,
                                    C.c_int, _sz, _sz, _vp, _vp)


def nd_sparse_compact_aggregate(idxs, planes, counts, norms, n, s, d, cap, out,
                                stream=None) -> None:
    _check("nd_sparse_compact_aggregate",
           _nd_sparse_compact_aggregate(_ptrs(idxs), _ptrs(planes), _ptrs(counts), _ptrs(norms),
                                        n, s, d, cap, _ptr(out), _stream(stream)))
