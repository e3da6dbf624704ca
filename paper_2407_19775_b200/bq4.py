"""ctypes binding of the 4-bit calls of ``libbq.so`` (``include/bq4.h``), taking torch tensors.
Argument marshalling only: every step runs in the library's kernels."""
from __future__ import annotations

import ctypes

import numpy as np
import torch

from .binding import _DT, DYNAMIC_TREE, BqError, _check, _dev, _stream, lib

SYMBOLS = ("bq4_make_codebook", "bq4_free_codebook", "bq4_quantize", "bq4_dequantize", "bq4_quantize_s16", "bq4_dequantize_s16")
_typed = False


def _lib() -> ctypes.CDLL:
    global _typed
    L = lib()
    if not _typed:
        vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        L.bq4_make_codebook.argtypes = [i32, vp, vp, ctypes.POINTER(vp)]
        L.bq4_free_codebook.argtypes = [vp]
        L.bq4_quantize.argtypes = [vp, i32, sz, i32, vp, vp, vp, vp]
        L.bq4_dequantize.argtypes = [vp, vp, sz, i32, vp, vp, i32, vp]
        L.bq4_quantize_s16.argtypes = [vp, i32, sz, i32, vp, vp, vp, vp]
        L.bq4_dequantize_s16.argtypes = [vp, vp, sz, i32, vp, vp, i32, vp]
        _typed = True
    return L


class Codebook4:
    """Handle of a 16-entry codebook (``bq4_make_codebook``)."""

    def __init__(self, kind: int = DYNAMIC_TREE, user_values=None):
        self._h = ctypes.c_void_p()
        self.values = np.empty(16, np.float32)
        user = None
        if user_values is not None:
            user = np.ascontiguousarray(user_values, np.float32)
            if user.size != 16:
                raise BqError("a 4-bit user codebook has 16 values")
        rc = _lib().bq4_make_codebook(kind, None if user is None else user.ctypes.data, self.values.ctypes.data, ctypes.byref(self._h))
        _check(rc, "bq4_make_codebook")

    @property
    def handle(self):
        return self._h

    def close(self) -> None:
        if self._h:
            _lib().bq4_free_codebook(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def bq4_quantize(x: torch.Tensor, block: int, cb: Codebook4, packed_out: torch.Tensor | None = None, absmax_out: torch.Tensor | None = None):
    """``bq4_quantize``: returns (packed uint8[ceil(n / 2)], absmax float32[ceil(n / block)])."""
    _dev(x, "x")
    n = x.numel()
    if packed_out is None:
        packed_out = torch.empty((n + 1) // 2, dtype=torch.uint8, device=x.device)
    if absmax_out is None:
        absmax_out = torch.empty((n + max(block, 1) - 1) // max(block, 1), dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        rc = _lib().bq4_quantize(x.data_ptr(), _DT[x.dtype], n, block, cb.handle, _dev(packed_out, "packed_out").data_ptr(),
                                 _dev(absmax_out, "absmax_out").data_ptr(), _stream(x))
    _check(rc, "bq4_quantize")
    return packed_out, absmax_out


def bq4_dequantize(packed: torch.Tensor, absmax: torch.Tensor, n: int, block: int, cb: Codebook4, dtype: torch.dtype,
                   y_out: torch.Tensor | None = None) -> torch.Tensor:
    """``bq4_dequantize``: returns y of ``dtype`` with n elements."""
    _dev(packed, "packed")
    _dev(absmax, "absmax")
    if y_out is None:
        y_out = torch.empty(n, dtype=dtype, device=packed.device)
    with torch.cuda.device(packed.device):
        rc = _lib().bq4_dequantize(packed.data_ptr(), absmax.data_ptr(), n, block, cb.handle, _dev(y_out, "y_out").data_ptr(), _DT[y_out.dtype],
                                   _stream(packed))
    _check(rc, "bq4_dequantize")
    return y_out


def bq4_quantize_s16(x: torch.Tensor, block: int, cb: Codebook4, packed_out: torch.Tensor | None = None, scale_out: torch.Tensor | None = None):
    """``bq4_quantize_s16``: returns (packed uint8[ceil(n / 2)], scale bfloat16[ceil(n / block)])."""
    _dev(x, "x")
    n = x.numel()
    if packed_out is None:
        packed_out = torch.empty((n + 1) // 2, dtype=torch.uint8, device=x.device)
    if scale_out is None:
        scale_out = torch.empty((n + max(block, 1) - 1) // max(block, 1), dtype=torch.bfloat16, device=x.device)
    if scale_out.dtype != torch.bfloat16:
        raise BqError("scale_out must be bfloat16")
    with torch.cuda.device(x.device):
        rc = _lib().bq4_quantize_s16(x.data_ptr(), _DT[x.dtype], n, block, cb.handle, _dev(packed_out, "packed_out").data_ptr(),
                                     _dev(scale_out, "scale_out").data_ptr(), _stream(x))
    _check(rc, "bq4_quantize_s16")
    return packed_out, scale_out


def bq4_dequantize_s16(packed: torch.Tensor, scale: torch.Tensor, n: int, block: int, cb: Codebook4, dtype: torch.dtype,
                       y_out: torch.Tensor | None = None) -> torch.Tensor:
    """``bq4_dequantize_s16``: returns y of ``dtype`` with n elements."""
    _dev(packed, "packed")
    _dev(scale, "scale")
    if scale.dtype != torch.bfloat16:
        raise BqError("scale must be bfloat16")
    if y_out is None:
        y_out = torch.empty(n, dtype=dtype, device=packed.device)
    with torch.cuda.device(packed.device):
        rc = _lib().bq4_dequantize_s16(packed.data_ptr(), scale.data_ptr(), n, block, cb.handle, _dev(y_out, "y_out").data_ptr(), _DT[y_out.dtype],
                                       _stream(packed))
    _check(rc, "bq4_dequantize_s16")
    return y_out
