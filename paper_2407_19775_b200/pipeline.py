"""Host-to-host calls: the tensor starts and ends in (pinned) host memory.

A shard that receives its activations over the network holds them in host buffers.
``HostBoundary`` wraps the library's host-buffer calls (``bq_host_pipe_create``,
``bq_quantize_host``, ``bq_dequantize_host``, ``bq_roundtrip_host``): the chunking, the three
streams and the events live in the library; this module only marshals torch tensors.
"""
from __future__ import annotations

import ctypes

import torch

from .binding import _DT, BqError, Codebook, _check, lib


def _host(t: torch.Tensor, name: str) -> torch.Tensor:
    if t.is_cuda:
        raise BqError(f"{name} must be a host tensor")
    if not t.is_contiguous():
        raise BqError(f"{name} must be contiguous")
    return t


class HostBoundary:
    """Chunked quantize / dequantize / roundtrip between host tensors (pinned for overlap).

    ``chunk`` is the number of elements per piece, ``slots`` pieces are in flight at once,
    ``min_block`` is the smallest block size the calls will use.  Device staging buffers are
    allocated once, here, by the library.  Calls enqueue and return; ``wait()`` blocks until the
    results are in the host tensors, ``wait_on_current_stream()`` orders the current CUDA stream
    behind them without blocking the host.
    """

    def __init__(self, cb: Codebook, dtype: torch.dtype, chunk: int = 1 << 25, slots: int = 3, min_block: int = 64):
        self.cb, self.dtype, self.chunk, self.slots = cb, dtype, int(chunk), int(slots)
        self.dev = cb.device
        self._h = ctypes.c_void_p()
        with torch.cuda.device(self.dev):
            rc = lib().bq_host_pipe_create(cb.handle, self.chunk, int(min_block), _DT[dtype], self.slots, ctypes.byref(self._h))
        _check(rc, "bq_host_pipe_create")

    def quantize(self, x_host: torch.Tensor, block: int, codes_host: torch.Tensor, absmax_host: torch.Tensor) -> None:
        _host(x_host, "x_host"); _host(codes_host, "codes_host"); _host(absmax_host, "absmax_host")
        with torch.cuda.device(self.dev):
            rc = lib().bq_quantize_host(self._h, x_host.data_ptr(), _DT[x_host.dtype], x_host.numel(), block, codes_host.data_ptr(),
                                        absmax_host.data_ptr())
        _check(rc, "bq_quantize_host")

    def dequantize(self, codes_host: torch.Tensor, absmax_host: torch.Tensor, block: int, y_host: torch.Tensor) -> None:
        _host(codes_host, "codes_host"); _host(absmax_host, "absmax_host"); _host(y_host, "y_host")
        with torch.cuda.device(self.dev):
            rc = lib().bq_dequantize_host(self._h, codes_host.data_ptr(), absmax_host.data_ptr(), codes_host.numel(), block,
                                          y_host.data_ptr(), _DT[y_host.dtype])
        _check(rc, "bq_dequantize_host")

    def roundtrip(self, x_host: torch.Tensor, block: int, y_host: torch.Tensor) -> None:
        _host(x_host, "x_host"); _host(y_host, "y_host")
        with torch.cuda.device(self.dev):
            rc = lib().bq_roundtrip_host(self._h, x_host.data_ptr(), _DT[x_host.dtype], x_host.numel(), block, y_host.data_ptr(),
                                         _DT[y_host.dtype])
        _check(rc, "bq_roundtrip_host")

    def wait(self) -> None:
        _check(lib().bq_host_pipe_wait(self._h), "bq_host_pipe_wait")

    def wait_on_current_stream(self) -> None:
        with torch.cuda.device(self.dev):
            _check(lib().bq_host_pipe_wait_on_stream(self._h, torch.cuda.current_stream(self.dev).cuda_stream), "bq_host_pipe_wait_on_stream")

    def close(self) -> None:
        if self._h:
            lib().bq_host_pipe_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
