"""Thin ctypes binding of libnuq.so: argument marshalling only.

Every function has the name and the argument order of its C counterpart in
include/nuq.h; tensors are passed as raw device pointers and the current torch
CUDA stream is used unless one is given.  There is no CPU path: importing this
module fails if the CUDA library cannot be built or loaded.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

NUQ_OK, ERR_INVALID_ARG, ERR_CAPACITY, ERR_BAD_STREAM, ERR_CUDA, ERR_TIMEOUT, ERR_INTERNAL = 0, -1, -2, -3, -4, -5, -6
WARN_NONFINITE = 1
NORM_L2, NORM_LINF = 0, 1
LEVELS_EXP, LEVELS_UNIFORM, LEVELS_TABLE = 0 << 8, 1 << 8, 2 << 8
MODE_ERC, MODE_FIXED, MODE_CODED = 0 << 16, 1 << 16, 2 << 16
TEST_NORMS = 1 << 24
TEST_SHORT_PATIENCE = 1 << 25
HEADER_WORDS = 16
STATIC_SCRATCH_BYTES = 512 * 1024


class NuqError(RuntimeError):
    def __init__(self, where, code):
        super().__init__(f"{where} failed with status {code}")
        self.code = code


class _Info(C.Structure):
    _fields_ = [("d", C.c_uint64), ("bucket", C.c_uint32), ("s", C.c_uint32), ("flags", C.c_uint32),
                ("sub_block", C.c_uint32), ("nblk", C.c_uint64), ("container_bits", C.c_uint64),
                ("code_bits", C.c_uint64), ("nnz", C.c_uint64)]


def _load():
    path = _build.LIB
    if not os.path.exists(path):
        _build.build()
    lib = C.CDLL(path)
    lib.nuq_encode.restype = C.c_int
    lib.nuq_encode.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint64, C.c_uint64,
                               C.c_void_p, C.c_void_p, C.c_void_p]
    lib.nuq_encode_static.restype = C.c_int
    lib.nuq_encode_static.argtypes = lib.nuq_encode.argtypes
    lib.nuq_decode_accumulate.restype = C.c_int
    lib.nuq_decode_accumulate.argtypes = [C.POINTER(C.c_void_p), C.c_uint32, C.c_uint64, C.c_uint32, C.c_uint32,
                                          C.c_void_p, C.c_void_p]
    lib.nuq_decode_update.restype = C.c_int
    lib.nuq_decode_update.argtypes = [C.POINTER(C.c_void_p), C.c_uint32, C.c_uint64, C.c_uint32, C.c_uint32,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_float, C.c_float, C.c_void_p]
    lib.nuq_encode_bound.restype = C.c_uint64
    lib.nuq_encode_bound.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32]
    lib.nuq_set_level_table.restype = C.c_int
    lib.nuq_set_level_table.argtypes = [C.POINTER(C.c_float), C.c_uint32]
    lib.nuq_level_histogram.restype = C.c_int
    lib.nuq_level_histogram.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint64,
                                        C.c_uint64, C.c_void_p, C.c_void_p]
    lib.nuq_fit_level_code.restype = C.c_int
    lib.nuq_fit_level_code.argtypes = [C.POINTER(C.c_uint64), C.c_uint32, C.POINTER(C.c_uint8)]
    lib.nuq_set_level_code.restype = C.c_int
    lib.nuq_set_level_code.argtypes = [C.POINTER(C.c_uint8), C.c_uint32]
    lib.nuq_set_test_norms.restype = C.c_int
    lib.nuq_set_test_norms.argtypes = [C.c_void_p]
    lib.nuq_last_status.restype = C.c_int
    lib.nuq_last_status.argtypes = [C.c_void_p]
    lib.nuq_stream_info.restype = C.c_int
    lib.nuq_stream_info.argtypes = [C.c_void_p, C.POINTER(_Info), C.c_void_p]
    lib.nuq_shutdown.restype = None
    lib.nuq_shutdown.argtypes = []
    lib.nuq_version.restype = C.c_char_p
    lib.nuq_version.argtypes = []
    return lib


_lib = _load()
LIBRARY_PATH = _build.LIB


def _stream(stream):
    if stream is None:
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, torch.cuda.Stream):
        return C.c_void_p(stream.cuda_stream)
    return C.c_void_p(int(stream))


def version() -> str:
    return _lib.nuq_version().decode()


def encode_bound(d, bucket, s, norm_kind=0) -> int:
    return int(_lib.nuq_encode_bound(d, bucket, s, norm_kind))


def set_level_table(interior_levels):
    """interior levels l_1 < ... < l_s of the level sequence (0, l_1, ..., l_s, 1) used with LEVELS_TABLE"""
    vals = [float(x) for x in interior_levels]
    arr = (C.c_float * len(vals))(*vals)
    rc = _lib.nuq_set_level_table(arr, len(vals))
    if rc != NUQ_OK:
        raise NuqError("nuq_set_level_table", rc)


def level_histogram(g: torch.Tensor, bucket, s, norm_kind=0, seed=0, offset=0, hist=None, stream=None):
    """how often each level index 0..s+1 comes out of the quantizer for g: int64 CUDA tensor of s + 2 counters"""
    assert g.is_cuda and g.dtype == torch.float32 and g.is_contiguous()
    if hist is None:
        hist = torch.empty(s + 2, dtype=torch.int64, device=g.device)
    rc = _lib.nuq_level_histogram(C.c_void_p(g.data_ptr()), g.numel(), bucket, s, norm_kind, seed, offset,
                                  C.c_void_p(hist.data_ptr()), _stream(stream))
    if rc != NUQ_OK:
        raise NuqError("nuq_level_histogram", rc)
    return hist


def fit_level_code(hist, s):
    """code lengths of the level indices 1..s+1 (Huffman) from the s + 2 counts of level_histogram (host values)"""
    vals = [int(x) for x in hist]
    assert len(vals) == s + 2
    arr = (C.c_uint64 * len(vals))(*vals)
    out = (C.c_uint8 * (s + 1))()
    rc = _lib.nuq_fit_level_code(arr, s, out)
    if rc != NUQ_OK:
        raise NuqError("nuq_fit_level_code", rc)
    return list(out)


def set_level_code(lengths):
    """code lengths of the level indices 1..s+1 that MODE_CODED calls use from now on"""
    vals = [int(x) for x in lengths]
    arr = (C.c_uint8 * len(vals))(*vals)
    rc = _lib.nuq_set_level_code(arr, len(vals) - 1)
    if rc != NUQ_OK:
        raise NuqError("nuq_set_level_code", rc)


def set_test_norms(norms: torch.Tensor | None):
    """norms: CUDA float32 tensor of ceil(d/bucket) bucket norms (kept by reference), or None."""
    rc = _lib.nuq_set_test_norms(C.c_void_p(norms.data_ptr()) if norms is not None else None)
    if rc != NUQ_OK:
        raise NuqError("nuq_set_test_norms", rc)


def encode(g: torch.Tensor, bucket, s, norm_kind=0, seed=0, offset=0, out=None, out_bits=None, stream=None):
    """c <- ENCODE(g).  Returns (out, out_bits): the container as an int32 CUDA tensor of
    nuq_encode_bound bytes and a one-element int64 CUDA tensor that receives container_bits."""
    assert g.is_cuda and g.dtype == torch.float32 and g.is_contiguous()
    d = g.numel()
    if out is None:
        nbytes = encode_bound(d, bucket, s, norm_kind)
        if nbytes == 0:
            raise NuqError("nuq_encode_bound", ERR_INVALID_ARG)
        out = torch.empty(nbytes // 4, dtype=torch.int32, device=g.device)
    if out_bits is None:
        out_bits = torch.empty(1, dtype=torch.int64, device=g.device)
    rc = _lib.nuq_encode(C.c_void_p(g.data_ptr()), d, bucket, s, norm_kind, seed, offset, C.c_void_p(out.data_ptr()),
                         C.c_void_p(out_bits.data_ptr()), _stream(stream))
    if rc != NUQ_OK:
        raise NuqError("nuq_encode", rc)
    return out, out_bits


def encode_static(g: torch.Tensor, bucket, s, norm_kind=0, seed=0, offset=0, *, out, out_bits, stream=None):
    """nuq_encode_static: the encoder for callers that may not allocate device memory.  Its
    scan state lives in a fixed array inside the library instead of a cudaMalloc'ed workspace,
    so `out` (encode_bound bytes) and `out_bits` (one int64) must be passed in and nothing is
    allocated here either.  Raises NuqError(ERR_CAPACITY) when d is too long for that array.
    Calls that could overlap on the GPU must be serialised by the caller."""
    assert g.is_cuda and g.dtype == torch.float32 and g.is_contiguous()
    rc = _lib.nuq_encode_static(C.c_void_p(g.data_ptr()), g.numel(), bucket, s, norm_kind, seed, offset,
                                C.c_void_p(out.data_ptr()), C.c_void_p(out_bits.data_ptr()), _stream(stream))
    if rc != NUQ_OK:
        raise NuqError("nuq_encode_static", rc)
    return out, out_bits


def decode_accumulate(streams, d, bucket, s, acc=None, stream=None):
    """acc <- sum_k DECODE(streams[k]); acc is overwritten."""
    if acc is None:
        acc = torch.empty(d, dtype=torch.float32, device=streams[0].device)
    ptrs = (C.c_void_p * len(streams))(*[C.c_void_p(t.data_ptr()) for t in streams])
    rc = _lib.nuq_decode_accumulate(ptrs, len(streams), d, bucket, s, C.c_void_p(acc.data_ptr()), _stream(stream))
    if rc != NUQ_OK:
        raise NuqError("nuq_decode_accumulate", rc)
    return acc


def decode_update(streams, d, bucket, s, w, yl=None, alpha=1.0, mu=0.0, l=0.0, acc=None, stream=None):
    """w <- w - (alpha / K) sum_k DECODE(streams[k]), or the momentum rule with yl when mu != 0; in place."""
    ptrs = (C.c_void_p * len(streams))(*[C.c_void_p(t.data_ptr()) for t in streams])
    rc = _lib.nuq_decode_update(ptrs, len(streams), d, bucket, s, C.c_void_p(acc.data_ptr() if acc is not None else None),
                                C.c_void_p(w.data_ptr()), C.c_void_p(yl.data_ptr() if yl is not None else None),
                                C.c_float(alpha), C.c_float(mu), C.c_float(l), _stream(stream))
    if rc != NUQ_OK:
        raise NuqError("nuq_decode_update", rc)
    return w


def last_status(stream=None) -> int:
    return int(_lib.nuq_last_status(_stream(stream)))


def stream_info(out: torch.Tensor, stream=None) -> dict:
    info = _Info()
    rc = _lib.nuq_stream_info(C.c_void_p(out.data_ptr()), C.byref(info), _stream(stream))
    if rc != NUQ_OK:
        raise NuqError("nuq_stream_info", rc)
    return {k: int(getattr(info, k)) for k, _ in _Info._fields_}


def shutdown():
    _lib.nuq_shutdown()
