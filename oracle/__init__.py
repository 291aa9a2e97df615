"""FastSGD oracle: TEST INFRASTRUCTURE, not the product.

A thin ctypes view of ``fastsgd_oracle.c`` (plain single-threaded C written from
the paper's Sec. 3.1-3.3, Eq. 2-4 and Algorithms 1-2).  Only the tests, the smoke
check and the CPU-baseline leg of the benchmark may import this package; the CUDA
library never does, and nothing here imports the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fastsgd_oracle.c")
_HDR = os.path.join(_HERE, "fastsgd_oracle.h")
_LIB = os.path.join(_HERE, "libfastsgd_oracle.so")

GCC_FLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c99", "-shared", "-fPIC"]

OK, ERR_NONFINITE, ERR_CAPACITY, ERR_TIMEOUT = 0, 1, 2, 3
DEC_BAD_MAGIC, DEC_BAD_VERSION, DEC_BAD_STATUS, DEC_N_MISMATCH = 16, 17, 18, 19
DEC_PARAM_MISMATCH, DEC_TRUNCATED, DEC_BAD_DIRECTORY, DEC_BAD_KEY, DEC_BAD_CODE = 20, 21, 22, 23, 24
BAD_PARAM = -3


def build(force: bool = False) -> str:
    """Compile the C oracle next to its source (gcc, no fast-math, no FMA contraction)."""
    stale = (not os.path.exists(_LIB)) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB) for s in (_SRC, _HDR))
    if force or stale:
        subprocess.check_call(["gcc", *GCC_FLAGS, "-o", _LIB, _SRC, "-lm"])
    return _LIB


class Params(C.Structure):
    _fields_ = [("base", C.c_double), ("tau", C.c_uint32), ("flag_bits", C.c_uint32),
                ("group_log2", C.c_uint32), ("reserved", C.c_uint32)]


class Adam(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float)]


def params(base: float, tau: int = 128, flag_bits: int = 2, group_log2: int = 14) -> Params:
    return Params(float(base), int(tau), int(flag_bits), int(group_log2), 0)


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        f32p, u64p, i32p, u8p, f64p = (C.POINTER(t) for t in (C.c_float, C.c_uint64, C.c_int32, C.c_uint8, C.c_double))
        u32p = C.POINTER(C.c_uint32)
        PP = C.POINTER(Params)
        L.fsgo_abs_sum.restype = C.c_double
        L.fsgo_abs_sum.argtypes = [f32p, C.c_uint64]
        L.fsgo_tables.restype = C.c_int
        L.fsgo_tables.argtypes = [C.c_double, C.c_double, C.c_uint32, f64p, f64p]
        L.fsgo_quantise.restype = C.c_uint32
        L.fsgo_quantise.argtypes = [C.c_double, f64p, C.c_uint32]
        L.fsgo_value_encode.restype = C.c_int
        L.fsgo_value_encode.argtypes = [f32p, C.c_uint64, C.c_double, C.c_uint32, u64p, i32p, u64p, f64p]
        L.fsgo_code_byte.restype = C.c_uint8
        L.fsgo_code_byte.argtypes = [C.c_int32]
        L.fsgo_code_from_byte.restype = C.c_int32
        L.fsgo_code_from_byte.argtypes = [C.c_uint8]
        L.fsgo_bitlen.restype = C.c_uint32
        L.fsgo_bitlen.argtypes = [C.c_uint64]
        L.fsgo_widths.restype = None
        L.fsgo_widths.argtypes = [C.c_uint32, C.c_uint32, u32p]
        L.fsgo_length_flag.restype = C.c_uint32
        L.fsgo_length_flag.argtypes = [C.c_uint64, u32p, C.c_uint32]
        L.fsgo_key_encode_paper.restype = C.c_int64
        L.fsgo_key_encode_paper.argtypes = [u64p, C.c_uint64, C.c_uint32, C.c_char_p, C.c_uint64, u32p]
        L.fsgo_compress_bound.restype = C.c_uint64
        L.fsgo_compress_bound.argtypes = [C.c_uint64, PP]
        L.fsgo_compress.restype = C.c_int
        L.fsgo_compress.argtypes = [f32p, C.c_uint64, PP, u8p, C.c_uint64, u64p]
        L.fsgo_write_stream.restype = C.c_int
        L.fsgo_write_stream.argtypes = [u64p, i32p, C.c_uint64, C.c_uint64, C.c_double, PP, u8p, C.c_uint64, u64p]
        L.fsgo_parse.restype = C.c_int
        L.fsgo_parse.argtypes = [u8p, C.c_uint64, C.c_uint64, PP, u64p, i32p, u64p, f64p]
        L.fsgo_decompress_accumulate.restype = C.c_int
        L.fsgo_decompress_accumulate.argtypes = [u8p, C.c_uint64, C.c_uint64, PP, f32p]
        L.fsgo_compress_kv.restype = C.c_int
        L.fsgo_compress_kv.argtypes = [u64p, f32p, C.c_uint64, C.c_uint64, PP, u8p, C.c_uint64, u64p]
        L.fsgo_sparse_adam_update.restype = C.c_int
        L.fsgo_sparse_adam_update.argtypes = [C.POINTER(u8p), u64p, C.c_uint32, C.c_uint64, PP, C.POINTER(Adam), f32p, f32p, f32p]
        _lib = L
    return _lib


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def _f32(v) -> np.ndarray:
    return np.ascontiguousarray(v, dtype=np.float32)


def abs_sum(v) -> float:
    v = _f32(v)
    return lib().fsgo_abs_sum(_ptr(v, C.c_float), v.size)


def tables(s: float, base: float, tau: int):
    P = np.zeros(129, np.float64)
    B = np.zeros(129, np.float64)
    rc = lib().fsgo_tables(s, base, tau, _ptr(P, C.c_double), _ptr(B, C.c_double))
    if rc:
        raise ValueError("bad parameters")
    return P[:tau + 1].copy(), B[:tau + 1].copy()


def quantise(a: float, B: np.ndarray, tau: int) -> int:
    B = np.ascontiguousarray(B, np.float64)
    return lib().fsgo_quantise(float(a), _ptr(B, C.c_double), tau)


def value_encode(v, base: float, tau: int):
    """Algorithm 1 -> (status, keys, signed codes, sum)."""
    v = _f32(v)
    keys = np.zeros(max(v.size, 1), np.uint64)
    codes = np.zeros(max(v.size, 1), np.int32)
    d = C.c_uint64(0)
    s = C.c_double(0.0)
    rc = lib().fsgo_value_encode(_ptr(v, C.c_float), v.size, base, tau, _ptr(keys, C.c_uint64),
                                 _ptr(codes, C.c_int32), C.byref(d), C.byref(s))
    return rc, keys[:d.value].copy(), codes[:d.value].copy(), s.value


def code_byte(q: int) -> int:
    return lib().fsgo_code_byte(q)


def code_from_byte(c: int) -> int:
    return lib().fsgo_code_from_byte(c)


def bitlen(x: int) -> int:
    return lib().fsgo_bitlen(x)


def widths(M: int, l: int):
    w = np.zeros(32, np.uint32)
    lib().fsgo_widths(M, l, _ptr(w, C.c_uint32))
    return [int(x) for x in w[:1 << l]]


def length_flag(delta: int, w, l: int) -> int:
    wa = np.zeros(32, np.uint32)
    wa[:len(w)] = w
    return lib().fsgo_length_flag(delta, _ptr(wa, C.c_uint32), l)


def key_encode_paper(keys, l: int):
    """Algorithm 2 as printed -> (BK as a '0'/'1' string, M)."""
    k = np.ascontiguousarray(keys, np.uint64)
    cap = int(k.size) * (l + 64) + 8
    buf = C.create_string_buffer(cap)
    M = C.c_uint32(0)
    nb = lib().fsgo_key_encode_paper(_ptr(k, C.c_uint64), k.size, l, buf, cap, C.byref(M))
    assert nb >= 0
    return buf.value.decode("ascii"), M.value


def compress_bound(n: int, p: Params) -> int:
    return lib().fsgo_compress_bound(n, C.byref(p))


def compress(v, p: Params, cap: int | None = None):
    """Encoder -> (status, stream bytes as uint8 array)."""
    v = _f32(v)
    if cap is None:
        cap = compress_bound(v.size, p)
    out = np.zeros(max(cap, 64), np.uint8)
    total = C.c_uint64(0)
    rc = lib().fsgo_compress(_ptr(v, C.c_float), v.size, C.byref(p), _ptr(out, C.c_uint8), cap, C.byref(total))
    return rc, out[:total.value].copy()


def write_stream(keys, codes, n: int, s: float, p: Params, cap: int | None = None):
    k = np.ascontiguousarray(keys, np.uint64)
    c = np.ascontiguousarray(codes, np.int32)
    if cap is None:
        cap = compress_bound(n, p)
    out = np.zeros(max(cap, 64), np.uint8)
    total = C.c_uint64(0)
    rc = lib().fsgo_write_stream(_ptr(k, C.c_uint64), _ptr(c, C.c_int32), k.size, n, s, C.byref(p),
                                 _ptr(out, C.c_uint8), cap, C.byref(total))
    return rc, out[:total.value].copy()


def parse(stream, n: int, p: Params, nbytes: int | None = None):
    """Decoder phases 1-2 -> (status, keys, signed codes, sum)."""
    s = np.ascontiguousarray(stream, np.uint8)
    nbytes = s.size if nbytes is None else nbytes
    dmax = int(np.frombuffer(s[24:32].tobytes(), np.uint64)[0]) if s.size >= 64 else 0
    dmax = min(dmax, n)
    keys = np.zeros(max(dmax, 1), np.uint64)
    codes = np.zeros(max(dmax, 1), np.int32)
    d = C.c_uint64(0)
    sm = C.c_double(0.0)
    rc = lib().fsgo_parse(_ptr(s, C.c_uint8), nbytes, n, C.byref(p), _ptr(keys, C.c_uint64),
                          _ptr(codes, C.c_int32), C.byref(d), C.byref(sm))
    return rc, keys[:d.value].copy(), codes[:d.value].copy(), sm.value


def decompress_accumulate(stream, n: int, p: Params, dense: np.ndarray, nbytes: int | None = None) -> int:
    """Decoder phases 1-4 + aggregation, in place on `dense` (float32, n entries)."""
    s = np.ascontiguousarray(stream, np.uint8)
    nbytes = s.size if nbytes is None else nbytes
    assert dense.dtype == np.float32 and dense.flags.c_contiguous and dense.size == n
    return lib().fsgo_decompress_accumulate(_ptr(s, C.c_uint8), nbytes, n, C.byref(p), _ptr(dense, C.c_float))


def sparse_adam_update(streams, n: int, p: Params, lr: float, beta1: float, beta2: float, eps: float,
                       theta: np.ndarray, m: np.ndarray, v: np.ndarray) -> int:
    """Adam (the experimental set-up's equations, no bias correction) on the coordinates where the sum of
    the decoded streams is non-zero; in place on theta, m, v (float32, n entries each)."""
    ss = [np.ascontiguousarray(s, np.uint8) for s in streams]
    for a in (theta, m, v):
        assert a.dtype == np.float32 and a.flags.c_contiguous and a.size == n
    u8p = C.POINTER(C.c_uint8)
    ptrs = (u8p * len(ss))(*[_ptr(s, C.c_uint8) for s in ss])
    sizes = (C.c_uint64 * len(ss))(*[s.size for s in ss])
    h = Adam(lr, beta1, beta2, eps)
    return lib().fsgo_sparse_adam_update(ptrs, sizes, len(ss), n, C.byref(p), C.byref(h),
                                         _ptr(theta, C.c_float), _ptr(m, C.c_float), _ptr(v, C.c_float))


def compress_kv(keys, values, n: int, p: Params, cap: int | None = None):
    """Encoder on key-value pairs -> (status, stream bytes as uint8 array)."""
    k = np.ascontiguousarray(keys, np.uint64)
    v = _f32(values)
    assert k.size == v.size
    if cap is None:
        cap = compress_bound(n, p)
    out = np.zeros(max(cap, 64), np.uint8)
    total = C.c_uint64(0)
    rc = lib().fsgo_compress_kv(_ptr(k, C.c_uint64), _ptr(v, C.c_float), k.size, n, C.byref(p), _ptr(out, C.c_uint8), cap, C.byref(total))
    return rc, out[:total.value].copy()
