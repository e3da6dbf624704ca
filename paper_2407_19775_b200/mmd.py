"""ctypes binding of the mixed-matrix-decomposition calls of ``libbq.so`` (``include/mmd.h``),
taking torch tensors.  Argument marshalling only: every step runs in the library's kernels.
"""
from __future__ import annotations

import ctypes

import numpy as np
import torch

from .binding import _DT, BqError, _check, _dev, _stream, lib

PATH_AUTO, PATH_GENERAL, PATH_TENSOR, PATH_TENSOR_TILE, PATH_TENSOR_SOLO, PATH_TENSOR_STREAMK = 0, 1, 2, 3, 4, 5
_TORCH_OF = {0: torch.float32, 1: torch.float16, 2: torch.bfloat16}

SYMBOLS = ("mmd_side_columns", "mmd_select_features", "mmd_rowquant", "mmd_decompose", "mmd_free", "mmd_weights_view",
           "mmd_workspace_layout", "mmd_linear", "mmd_linear_static", "mmd_kernel_status", "mmd_selftest_bounded_wait", "mmd_workspace_bytes_streamk")
SELFTEST_CODE = 77
STATIC_SCRATCH_BYTES = 4 << 20
_typed = False


def _lib() -> ctypes.CDLL:
    global _typed
    L = lib()
    if not _typed:
        vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        L.mmd_side_columns.argtypes = [i32]
        L.mmd_select_features.argtypes = [vp, i32, ctypes.c_float, vp, ctypes.POINTER(i32)]
        L.mmd_rowquant.argtypes = [vp, i32, i32, i32, vp, i32, vp, vp, vp, vp]
        L.mmd_decompose.argtypes = [vp, i32, i32, i32, vp, i32, vp, ctypes.POINTER(vp)]
        L.mmd_free.argtypes = [vp]
        L.mmd_weights_view.argtypes = [vp] + [ctypes.POINTER(vp)] * 4 + [ctypes.POINTER(i32)] * 4
        L.mmd_workspace_layout.argtypes = [vp, i32, ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.mmd_workspace_bytes_streamk.argtypes = [vp, i32, ctypes.POINTER(sz)]
        L.mmd_linear.argtypes = [vp, vp, i32, vp, i32, vp, sz, i32, vp]
        L.mmd_linear_static.argtypes = [vp, vp, i32, vp, i32, i32, vp]
        L.mmd_kernel_status.argtypes = [vp, ctypes.POINTER(i32)]
        L.mmd_selftest_bounded_wait.argtypes = [vp, ctypes.c_uint, ctypes.POINTER(i32), vp]
        _typed = True
    return L


def mmd_side_columns(n_features: int) -> int:
    return int(_lib().mmd_side_columns(n_features))


def mmd_select_features(feature_absmax, tau: float) -> np.ndarray:
    """``mmd_select_features`` on a host array of per-feature calibration magnitudes."""
    a = np.ascontiguousarray(feature_absmax, np.float32)
    idx = np.empty(a.size, np.int32)
    count = ctypes.c_int(0)
    _check(_lib().mmd_select_features(a.ctypes.data, a.size, float(tau), idx.ctypes.data, ctypes.byref(count)), "mmd_select_features")
    return idx[:count.value].copy()


def mmd_rowquant(v: torch.Tensor, idx: torch.Tensor | None):
    """``mmd_rowquant``: returns (q int8 [R, K], scale float32 [R], side [R, side columns])."""
    _dev(v, "v")
    R, K = v.shape
    ko = 0 if idx is None else idx.numel()
    q = torch.empty((R, K), dtype=torch.int8, device=v.device)
    scale = torch.empty(R, dtype=torch.float32, device=v.device)
    side = torch.empty((R, mmd_side_columns(ko)), dtype=v.dtype, device=v.device)
    with torch.cuda.device(v.device):
        rc = _lib().mmd_rowquant(v.data_ptr(), _DT[v.dtype], R, K, None if ko == 0 else _dev(idx, "idx").data_ptr(), ko, q.data_ptr(),
                                 scale.data_ptr(), side.data_ptr() if ko else None, _stream(v))
    _check(rc, "mmd_rowquant")
    return q, scale, side


def rowquant_into(v: torch.Tensor, idx: torch.Tensor | None, q: torch.Tensor, scale: torch.Tensor, side: torch.Tensor) -> None:
    """``mmd_rowquant`` into caller-provided outputs."""
    R, K = v.shape
    ko = 0 if idx is None else idx.numel()
    with torch.cuda.device(v.device):
        rc = _lib().mmd_rowquant(_dev(v, "v").data_ptr(), _DT[v.dtype], R, K, None if ko == 0 else idx.data_ptr(), ko, q.data_ptr(),
                                 scale.data_ptr(), side.data_ptr() if ko else None, _stream(v))
    _check(rc, "mmd_rowquant")


class DecomposedLinear:
    """Handle of one decomposed weight matrix (``mmd_decompose``) and its linear layer."""

    def __init__(self, W: torch.Tensor, features):
        _dev(W, "W")
        idx = np.ascontiguousarray(features, np.int32)
        self._h = ctypes.c_void_p()
        self.N, self.K = W.shape
        self.dtype = W.dtype
        self.device = W.device
        with torch.cuda.device(W.device):
            rc = _lib().mmd_decompose(W.data_ptr(), _DT[W.dtype], self.N, self.K, idx.ctypes.data if idx.size else None, idx.size,
                                      _stream(W), ctypes.byref(self._h))
        _check(rc, "mmd_decompose")
        self.n_features = int(idx.size)
        self._ws = None

    @property
    def handle(self):
        return self._h

    def view(self):
        """(q, scale, side, idx) as torch tensors aliasing the handle's device memory."""
        ptr = [ctypes.c_void_p() for _ in range(4)]
        ints = [ctypes.c_int() for _ in range(4)]
        _check(_lib().mmd_weights_view(self._h, *[ctypes.byref(p) for p in ptr], *[ctypes.byref(i) for i in ints]), "mmd_weights_view")
        N, K, ko, _ = (i.value for i in ints)
        sc = mmd_side_columns(ko)

        def alias(p, shape, dtype):
            n = int(np.prod(shape))
            if n == 0:
                return torch.empty(shape, dtype=dtype, device=self.device)
            nbytes = n * torch.empty((), dtype=dtype).element_size()
            iface = {"shape": (nbytes,), "typestr": "|u1", "data": (p.value, False), "version": 3}
            holder = type("DevMem", (), {"__cuda_array_interface__": iface})()
            return torch.as_tensor(holder, device=self.device).view(dtype).view(shape)

        return (alias(ptr[0], (N, K), torch.int8), alias(ptr[1], (N,), torch.float32), alias(ptr[2], (N, sc), self.dtype),
                alias(ptr[3], (ko,), torch.int32))

    def workspace_layout(self, M: int):
        offs = (ctypes.c_size_t * 3)()
        total = ctypes.c_size_t()
        _check(_lib().mmd_workspace_layout(self._h, M, offs, ctypes.byref(total)), "mmd_workspace_layout")
        return tuple(int(o) for o in offs), int(total.value)

    def workspace_bytes(self, M: int) -> int:
        """``mmd_workspace_bytes_streamk``: the workspace size that lets decode-size calls take the stream-K kernel."""
        total = ctypes.c_size_t()
        _check(_lib().mmd_workspace_bytes_streamk(self._h, M, ctypes.byref(total)), "mmd_workspace_bytes_streamk")
        return int(total.value)

    def workspace(self, M: int, streamk: bool = False) -> torch.Tensor:
        """A workspace for M rows (cached); with ``streamk`` also the room the stream-K kernel's slots need."""
        total = self.workspace_bytes(M) if streamk else self.workspace_layout(M)[1]
        if self._ws is None or self._ws.numel() < total:
            self._ws = torch.empty(total + 256, dtype=torch.uint8, device=self.device)
        off = (-self._ws.data_ptr()) % 256
        return self._ws[off:off + total]

    def linear(self, X: torch.Tensor, out_dtype: torch.dtype | None = None, path: int = PATH_AUTO, y_out: torch.Tensor | None = None,
               workspace: torch.Tensor | None = None) -> torch.Tensor:
        """``mmd_linear``: Y = X W^T through the decomposition."""
        _dev(X, "X")
        if X.dtype != self.dtype or X.dim() != 2 or X.shape[1] != self.K:
            raise BqError("X must be [M, K] of the weights' element type")
        M = X.shape[0]
        ws = self.workspace(M, streamk=(path == PATH_TENSOR_STREAMK)) if workspace is None else workspace
        if y_out is None:
            y_out = torch.empty((M, self.N), dtype=out_dtype or X.dtype, device=X.device)
        with torch.cuda.device(X.device):
            rc = _lib().mmd_linear(self._h, X.data_ptr(), M, _dev(y_out, "y_out").data_ptr(), _DT[y_out.dtype], ws.data_ptr(), ws.numel(),
                                   path, _stream(X))
        _check(rc, "mmd_linear")
        return y_out

    def linear_static(self, X: torch.Tensor, out_dtype: torch.dtype | None = None, path: int = PATH_AUTO,
                      y_out: torch.Tensor | None = None) -> torch.Tensor:
        """``mmd_linear_static``: the same layer with the library's built-in scratch array (small M only); the call
        itself allocates nothing when ``y_out`` is given."""
        _dev(X, "X")
        if X.dtype != self.dtype or X.dim() != 2 or X.shape[1] != self.K:
            raise BqError("X must be [M, K] of the weights' element type")
        M = X.shape[0]
        if y_out is None:
            y_out = torch.empty((M, self.N), dtype=out_dtype or X.dtype, device=X.device)
        with torch.cuda.device(X.device):
            rc = _lib().mmd_linear_static(self._h, X.data_ptr(), M, _dev(y_out, "y_out").data_ptr(), _DT[y_out.dtype], path, _stream(X))
        if rc == 10:
            raise BqError("mmd_linear_static failed with status 10: " + _lib().bq_last_cuda_error().decode())
        _check(rc, "mmd_linear_static")
        return y_out

    def workspace_parts(self, M: int, workspace: torch.Tensor | None = None):
        """(qx, scalex, sidex) views of the workspace after a call with M rows."""
        ws = self.workspace(M) if workspace is None else workspace
        (oq, osc, osd), _ = self.workspace_layout(M)
        sc = mmd_side_columns(self.n_features)
        qx = ws[oq:oq + M * self.K].view(torch.int8).view(M, self.K)
        sx = ws[osc:osc + 4 * M].view(torch.float32)
        sd = ws[osd:osd + 2 * M * sc].view(self.dtype).view(M, sc)
        return qx, sx, sd

    def kernel_status(self) -> int:
        st = ctypes.c_int(0)
        with torch.cuda.device(self.device):
            _check(_lib().mmd_kernel_status(self._h, ctypes.byref(st)), "mmd_kernel_status")
        return int(st.value)

    def selftest_bounded_wait(self, limit_us: int = 2000) -> int:
        """``mmd_selftest_bounded_wait``: lets a bounded wait of the tensor-core kernels run out on purpose (short
        limit, a barrier nothing arms); returns how many threads left through the give-up path."""
        left = ctypes.c_int(-1)
        with torch.cuda.device(self.device):
            _check(_lib().mmd_selftest_bounded_wait(self._h, limit_us, ctypes.byref(left), torch.cuda.current_stream(self.device).cuda_stream),
                   "mmd_selftest_bounded_wait")
        return int(left.value)

    def close(self) -> None:
        if self._h:
            _lib().mmd_free(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
