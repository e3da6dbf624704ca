"""ctypes binding of the order-slicing calls (``include/mtpp.h``): argument marshalling only."""
from __future__ import annotations

import ctypes

import numpy as np
import torch

from .binding import BqError, _check, lib

MAX_NODES, MAX_BLOCKS = 1024, 16
SYMBOLS = ("mtpp_graph_create", "mtpp_graph_free", "mtpp_decode_orders", "mtpp_slice_orders")
_ready = False


def _lib():
    global _ready
    L = lib()
    if not _ready:
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
        L.mtpp_graph_create.argtypes = [i32, i32, vp, vp, vp, vp, ctypes.POINTER(vp)]
        L.mtpp_graph_free.argtypes = [vp]
        L.mtpp_decode_orders.argtypes = [vp, vp, i32, vp, vp]
        L.mtpp_slice_orders.argtypes = [vp, vp, i32, i32, i64, i64, vp, vp, vp, vp, vp]
        _ready = True
    return L


class SliceGraph:
    """Device copy of a computation graph (``mtpp_graph_create``).  ``edges`` is an [m, 2] integer array of
    (producer, consumer) pairs; work / sizeparam / sizeout are integer arrays of length n."""

    def __init__(self, n: int, edges, work, sizeparam, sizeout, device=None):
        self.n = int(n)
        e = np.ascontiguousarray(np.asarray(edges, np.int32).reshape(-1, 2))
        w, sp, so = (np.ascontiguousarray(np.asarray(a, np.int64)) for a in (work, sizeparam, sizeout))
        if not (w.size == sp.size == so.size == self.n):
            raise BqError("work, sizeparam and sizeout have one entry per node")
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self._h = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            rc = _lib().mtpp_graph_create(self.n, e.shape[0], e.ctypes.data if e.size else None, w.ctypes.data, sp.ctypes.data, so.ctypes.data,
                                          ctypes.byref(self._h))
        _check(rc, "mtpp_graph_create")

    def decode_orders(self, keys: torch.Tensor, orders_out: torch.Tensor | None = None) -> torch.Tensor:
        """``mtpp_decode_orders``: keys [P, n] float32 on the device -> orders [P, n] int32."""
        if not (keys.is_cuda and keys.is_contiguous() and keys.dtype == torch.float32 and keys.dim() == 2 and keys.shape[1] == self.n):
            raise BqError("keys must be a contiguous CUDA float32 tensor [P, n]")
        P = keys.shape[0]
        if orders_out is None:
            orders_out = torch.empty((P, self.n), dtype=torch.int32, device=keys.device)
        with torch.cuda.device(self.device):
            rc = _lib().mtpp_decode_orders(self._h, keys.data_ptr(), P, orders_out.data_ptr(), torch.cuda.current_stream(self.device).cuda_stream)
        _check(rc, "mtpp_decode_orders")
        return orders_out

    def slice_orders(self, orders: torch.Tensor, k: int, B: int, M: int, out=None):
        """``mtpp_slice_orders``: returns (cost int64 [P], blocks int32 [P], cuts int32 [P, k], status int32 [P])."""
        if not (orders.is_cuda and orders.is_contiguous() and orders.dtype == torch.int32 and orders.dim() == 2 and orders.shape[1] == self.n):
            raise BqError("orders must be a contiguous CUDA int32 tensor [P, n]")
        P = orders.shape[0]
        if out is None:
            dev = orders.device
            out = (torch.empty(P, dtype=torch.int64, device=dev), torch.empty(P, dtype=torch.int32, device=dev),
                   torch.empty((P, max(k, 1)), dtype=torch.int32, device=dev), torch.empty(P, dtype=torch.int32, device=dev))
        cost, blocks, cuts, status = out
        with torch.cuda.device(self.device):
            rc = _lib().mtpp_slice_orders(self._h, orders.data_ptr(), P, k, B, M, cost.data_ptr(), blocks.data_ptr(), cuts.data_ptr(),
                                          status.data_ptr(), torch.cuda.current_stream(self.device).cuda_stream)
        _check(rc, "mtpp_slice_orders")
        return out

    def close(self) -> None:
        if self._h:
            _lib().mtpp_graph_free(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
