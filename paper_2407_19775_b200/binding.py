"""ctypes binding of ``libbq.so``: the same calls as ``include/bq.h``, taking torch tensors.

Argument marshalling only.  Every step of the method runs in the library's CUDA kernels;
there is no CPU path, and a missing or unbuilt library is an error.
"""
from __future__ import annotations

import ctypes
import os

import torch

F32, F16, BF16 = 0, 1, 2
DYNAMIC_TREE, USER = 0, 1
_DT = {torch.float32: F32, torch.float16: F16, torch.bfloat16: BF16}
_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("BQ_LIB", os.path.join(_HERE, "libbq.so"))    # BQ_LIB: load another build of the library
_lib = None

SYMBOLS = ("bq_make_codebook", "bq_free_codebook", "bq_quantize", "bq_dequantize", "bq_roundtrip",
           "bq_status_string", "bq_last_cuda_error", "bq_codebook_is_folded", "bq_debug_build",
           "bq_host_pipe_create", "bq_host_pipe_destroy", "bq_quantize_host", "bq_dequantize_host", "bq_roundtrip_host",
           "bq_host_pipe_wait", "bq_host_pipe_wait_on_stream", "bq_set_staging", "bq_kernel_status")


class BqError(RuntimeError):
    pass


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise BqError(f"{LIB_PATH} is missing: build it with `python -m paper_2407_19775_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        L.bq_make_codebook.argtypes = [i32, vp, vp, ctypes.POINTER(vp)]
        L.bq_free_codebook.argtypes = [vp]
        L.bq_quantize.argtypes = [vp, i32, sz, i32, vp, vp, vp, vp]
        L.bq_dequantize.argtypes = [vp, vp, sz, i32, vp, vp, i32, vp]
        L.bq_roundtrip.argtypes = [vp, i32, sz, i32, vp, vp, i32, vp, vp, vp]
        L.bq_status_string.argtypes = [i32]
        L.bq_status_string.restype = ctypes.c_char_p
        L.bq_last_cuda_error.restype = ctypes.c_char_p
        L.bq_codebook_is_folded.argtypes = [vp]
        L.bq_host_pipe_create.argtypes = [vp, sz, i32, i32, i32, ctypes.POINTER(vp)]
        L.bq_host_pipe_destroy.argtypes = [vp]
        L.bq_quantize_host.argtypes = [vp, vp, i32, sz, i32, vp, vp]
        L.bq_dequantize_host.argtypes = [vp, vp, vp, sz, i32, vp, i32]
        L.bq_roundtrip_host.argtypes = [vp, vp, i32, sz, i32, vp, i32]
        L.bq_host_pipe_wait.argtypes = [vp]
        L.bq_host_pipe_wait_on_stream.argtypes = [vp, vp]
        L.bq_set_staging.argtypes = [i32]
        L.bq_kernel_status.argtypes = [vp, ctypes.POINTER(i32)]
        _lib = L
    return _lib


def _check(rc: int, what: str) -> None:
    if rc != 0:
        L = lib()
        msg = L.bq_status_string(rc).decode()
        if rc in (6, 10, 11):                                     # CUDA errors, the static limit and debug assertions leave a text
            msg += ": " + L.bq_last_cuda_error().decode()
        raise BqError(f"{what} failed with status {rc} ({msg})")


def _stream(x: torch.Tensor) -> int:
    return torch.cuda.current_stream(x.device).cuda_stream


def _dev(t: torch.Tensor, name: str) -> torch.Tensor:
    if not t.is_cuda:
        raise BqError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise BqError(f"{name} must be contiguous")
    return t


class Codebook:
    """Handle of a 256-entry codebook and its device tables (``bq_make_codebook``)."""

    def __init__(self, kind: int = DYNAMIC_TREE, user_values=None, device=None):
        import numpy as np
        self._h = ctypes.c_void_p()
        self.values = np.empty(256, np.float32)
        user = None
        if user_values is not None:
            user = np.ascontiguousarray(user_values, np.float32)
            if user.size != 256:
                raise BqError("a user codebook has 256 values")
        dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        with torch.cuda.device(dev):
            rc = lib().bq_make_codebook(kind, None if user is None else user.ctypes.data, self.values.ctypes.data,
                                        ctypes.byref(self._h))
        _check(rc, "bq_make_codebook")
        self.device = dev

    @property
    def handle(self) -> ctypes.c_void_p:
        return self._h

    @property
    def folded(self) -> bool:
        return bool(lib().bq_codebook_is_folded(self._h))

    def close(self) -> None:
        if self._h:
            lib().bq_free_codebook(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def set_staging(on: bool) -> bool:
    """``bq_set_staging``: blocks of 2048 / 4096 through the shared-memory-staged kernel; returns the previous setting."""
    return bool(lib().bq_set_staging(int(bool(on))))


def debug_build() -> bool:
    """``bq_debug_build``: whether the loaded library carries its host-side assertions."""
    return bool(lib().bq_debug_build())


def kernel_status(cb: "Codebook") -> int:
    """``bq_kernel_status``: non-zero when a kernel of this codebook gave up on a bounded wait (reads and clears)."""
    st = ctypes.c_int(0)
    with torch.cuda.device(cb.device):
        _check(lib().bq_kernel_status(cb.handle, ctypes.byref(st)), "bq_kernel_status")
    return int(st.value)


def n_blocks(n: int, block: int) -> int:
    return (n + block - 1) // block


def bq_quantize(x: torch.Tensor, block: int, cb: Codebook, codes_out: torch.Tensor | None = None,
                absmax_out: torch.Tensor | None = None):
    """``bq_quantize``: returns (codes uint8[n], absmax float32[ceil(n / block)])."""
    _dev(x, "x")
    n = x.numel()
    if codes_out is None:
        codes_out = torch.empty(n, dtype=torch.uint8, device=x.device)
    if absmax_out is None:
        absmax_out = torch.empty(n_blocks(n, max(block, 1)), dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        rc = lib().bq_quantize(x.data_ptr(), _DT[x.dtype], n, block, cb.handle, _dev(codes_out, "codes_out").data_ptr(),
                               _dev(absmax_out, "absmax_out").data_ptr(), _stream(x))
    _check(rc, "bq_quantize")
    return codes_out, absmax_out


def bq_dequantize(codes: torch.Tensor, absmax: torch.Tensor, block: int, cb: Codebook, dtype: torch.dtype,
                  y_out: torch.Tensor | None = None) -> torch.Tensor:
    """``bq_dequantize``: returns y of ``dtype`` with ``codes.numel()`` elements."""
    _dev(codes, "codes")
    _dev(absmax, "absmax")
    n = codes.numel()
    if y_out is None:
        y_out = torch.empty(n, dtype=dtype, device=codes.device)
    with torch.cuda.device(codes.device):
        rc = lib().bq_dequantize(codes.data_ptr(), absmax.data_ptr(), n, block, cb.handle, _dev(y_out, "y_out").data_ptr(),
                                 _DT[y_out.dtype], _stream(codes))
    _check(rc, "bq_dequantize")
    return y_out


def bq_roundtrip(x: torch.Tensor, block: int, cb: Codebook, dtype: torch.dtype | None = None, y_out: torch.Tensor | None = None,
                 codes_out: torch.Tensor | None = None, absmax_out: torch.Tensor | None = None) -> torch.Tensor:
    """``bq_roundtrip``: dequantize(quantize(x)) in one kernel; side outputs are optional."""
    _dev(x, "x")
    n = x.numel()
    if y_out is None:
        y_out = torch.empty(x.shape, dtype=dtype or x.dtype, device=x.device)
    c = None if codes_out is None else _dev(codes_out, "codes_out").data_ptr()
    a = None if absmax_out is None else _dev(absmax_out, "absmax_out").data_ptr()
    with torch.cuda.device(x.device):
        rc = lib().bq_roundtrip(x.data_ptr(), _DT[x.dtype], n, block, cb.handle, _dev(y_out, "y_out").data_ptr(), _DT[y_out.dtype], c, a,
                                _stream(x))
    _check(rc, "bq_roundtrip")
    return y_out
