"""ctypes front end of the CPU oracle (test infrastructure only).

The arithmetic lives in ``bq_oracle.cpp``; this module only compiles it, loads it and
marshals numpy arrays.  Nothing under ``oracle/`` is imported by the CUDA library or its
Python binding: the tests, the smoke check and the CPU-baseline leg of the benchmark are
the only callers.

Element types are passed as numpy arrays: ``float32`` for fp32, and ``uint16`` holding the
raw bit patterns for fp16 / bf16 (numpy has no bf16).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

F32, F16, BF16 = 0, 1, 2
_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bq_oracle.cpp")
_HDR = os.path.join(_HERE, "bq_oracle.h")
_LIB = os.path.join(_HERE, "libbq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle into ``oracle/libbq_oracle.so`` (skipped when up to date)."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= newest:
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-Wall", "-Wextra", "-o", tmp, _SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        L.bq_oracle_make_codebook.argtypes = [vp]
        L.bq_oracle_quantize.argtypes = [vp, i32, sz, i32, vp, vp, vp]
        L.bq_oracle_dequantize.argtypes = [vp, vp, sz, i32, vp, vp, i32]
        L.bq_oracle_roundtrip.argtypes = [vp, i32, sz, i32, vp, vp, i32, vp, vp]
        L.bq_oracle_widen.argtypes = [ctypes.c_uint16, i32]
        L.bq_oracle_widen.restype = ctypes.c_float
        L.bq_oracle_narrow.argtypes = [ctypes.c_float, i32]
        L.bq_oracle_narrow.restype = ctypes.c_uint16
        L.bq_oracle_nearest.argtypes = [ctypes.c_float, vp]
        _lib = L
    return _lib


def _np_dtype(dt: int):
    if dt not in (F32, F16, BF16):
        raise ValueError(f"unknown element type {dt}")
    return np.float32 if dt == F32 else np.uint16


def _ptr(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check_in(a: np.ndarray, dt: int) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != _np_dtype(dt):
        raise TypeError(f"dtype {dt} wants a {_np_dtype(dt).__name__} array, got {a.dtype}")
    return a.reshape(-1)


def make_codebook() -> np.ndarray:
    cb = np.empty(256, np.float32)
    rc = lib().bq_oracle_make_codebook(_ptr(cb))
    assert rc == 0
    return cb


def nearest(xhat: float, cb: np.ndarray) -> int:
    return int(lib().bq_oracle_nearest(ctypes.c_float(float(xhat)), _ptr(cb)))


def widen(bits: int, dt: int) -> float:
    return float(lib().bq_oracle_widen(int(bits), dt))


def narrow(v: float, dt: int) -> int:
    return int(lib().bq_oracle_narrow(ctypes.c_float(v), dt))


def quantize(x: np.ndarray, xdt: int, block: int, cb: np.ndarray):
    x = _check_in(x, xdt)
    n = x.size
    nb = (n + block - 1) // block if block >= 1 else 0
    codes = np.empty(n, np.uint8)
    absmax = np.empty(nb, np.float32)
    rc = lib().bq_oracle_quantize(_ptr(x), xdt, n, block, _ptr(cb), _ptr(codes), _ptr(absmax))
    if rc:
        raise ValueError("bq_oracle_quantize: bad argument")
    return codes, absmax


def dequantize(codes: np.ndarray, absmax: np.ndarray, block: int, cb: np.ndarray, ydt: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, np.uint8).reshape(-1)
    absmax = np.ascontiguousarray(absmax, np.float32).reshape(-1)
    y = np.empty(codes.size, _np_dtype(ydt))
    rc = lib().bq_oracle_dequantize(_ptr(codes), _ptr(absmax), codes.size, block, _ptr(cb), _ptr(y), ydt)
    if rc:
        raise ValueError("bq_oracle_dequantize: bad argument")
    return y


def roundtrip(x: np.ndarray, xdt: int, block: int, cb: np.ndarray, ydt: int, side: bool = False):
    x = _check_in(x, xdt)
    n = x.size
    nb = (n + block - 1) // block if block >= 1 else 0
    y = np.empty(n, _np_dtype(ydt))
    codes = np.empty(n, np.uint8) if side else None
    absmax = np.empty(nb, np.float32) if side else None
    rc = lib().bq_oracle_roundtrip(_ptr(x), xdt, n, block, _ptr(cb), _ptr(y), ydt, _ptr(codes), _ptr(absmax))
    if rc:
        raise ValueError("bq_oracle_roundtrip: bad argument")
    return (y, codes, absmax) if side else y


def _shard_ranges(n: int, block: int, threads: int):
    nb = (n + block - 1) // block
    threads = max(1, min(threads, nb))
    per = (nb + threads - 1) // threads
    out = []
    for t in range(threads):
        b0, b1 = t * per, min(nb, (t + 1) * per)
        if b0 < b1:
            out.append((b0, b1, b0 * block, min(n, b1 * block)))
    return nb, out


def _run_sharded(work, ranges, threads: int, what: str) -> None:
    with ThreadPoolExecutor(max(1, threads)) as ex:
        rcs = list(ex.map(work, ranges))
    if any(rcs):
        raise ValueError(f"{what}: bad argument")


# The three *_sharded helpers run the unchanged single-threaded oracle on contiguous ranges
# of whole blocks, one range per host thread.  Blocks are independent, so the bytes are the
# same as one call over everything; the threading is here, outside the oracle's functions.

def quantize_sharded(x: np.ndarray, xdt: int, block: int, cb: np.ndarray, threads: int):
    x = _check_in(x, xdt)
    n = x.size
    nb, ranges = _shard_ranges(n, block, threads)
    codes = np.empty(n, np.uint8)
    absmax = np.empty(nb, np.float32)
    L = lib()

    def work(r):
        b0, b1, e0, e1 = r
        return L.bq_oracle_quantize(_ptr(x[e0:e1]), xdt, e1 - e0, block, _ptr(cb), _ptr(codes[e0:e1]), _ptr(absmax[b0:b1]))

    _run_sharded(work, ranges, threads, "bq_oracle_quantize")
    return codes, absmax


def dequantize_sharded(codes: np.ndarray, absmax: np.ndarray, block: int, cb: np.ndarray, ydt: int, threads: int):
    codes = np.ascontiguousarray(codes, np.uint8).reshape(-1)
    absmax = np.ascontiguousarray(absmax, np.float32).reshape(-1)
    n = codes.size
    _, ranges = _shard_ranges(n, block, threads)
    y = np.empty(n, _np_dtype(ydt))
    L = lib()

    def work(r):
        b0, b1, e0, e1 = r
        return L.bq_oracle_dequantize(_ptr(codes[e0:e1]), _ptr(absmax[b0:b1]), e1 - e0, block, _ptr(cb), _ptr(y[e0:e1]), ydt)

    _run_sharded(work, ranges, threads, "bq_oracle_dequantize")
    return y


def roundtrip_sharded(x: np.ndarray, xdt: int, block: int, cb: np.ndarray, ydt: int, threads: int):
    """Returns (y, codes, absmax)."""
    x = _check_in(x, xdt)
    n = x.size
    nb, ranges = _shard_ranges(n, block, threads)
    y = np.empty(n, _np_dtype(ydt))
    codes = np.empty(n, np.uint8)
    absmax = np.empty(nb, np.float32)
    L = lib()

    def work(r):
        b0, b1, e0, e1 = r
        return L.bq_oracle_roundtrip(_ptr(x[e0:e1]), xdt, e1 - e0, block, _ptr(cb), _ptr(y[e0:e1]), ydt,
                                     _ptr(codes[e0:e1]), _ptr(absmax[b0:b1]))

    _run_sharded(work, ranges, threads, "bq_oracle_roundtrip")
    return y, codes, absmax
