"""ctypes binding of the block-size selection calls of ``libbq.so`` (``include/bq_tune.h``), taking
torch tensors.  Argument marshalling only."""
from __future__ import annotations

import ctypes

import numpy as np
import torch

from .binding import BqError, Codebook, _DT, _check, _stream, lib

SYMBOLS = ("bqt_workspace_bytes", "bqt_block_errors", "bqt_pick_block")
MAX_CANDIDATES = 16
_typed = False


def _lib() -> ctypes.CDLL:
    global _typed
    L = lib()
    if not _typed:
        vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        L.bqt_workspace_bytes.argtypes = [i32, sz]
        L.bqt_workspace_bytes.restype = sz
        L.bqt_block_errors.argtypes = [vp, i32, sz, vp, vp, i32, vp, sz, vp, vp]
        L.bqt_pick_block.argtypes = [vp, vp, i32, ctypes.c_double, ctypes.POINTER(i32)]
        _typed = True
    return L


def workspace_bytes(dtype: torch.dtype, n: int) -> int:
    return int(_lib().bqt_workspace_bytes(_DT[dtype], n))


def block_errors(x: torch.Tensor, blocks, cb: Codebook, workspace: torch.Tensor | None = None, sums_out: torch.Tensor | None = None) -> torch.Tensor:
    """``bqt_block_errors``: returns the device tensor of len(blocks) + 1 doubles (err2 per candidate, then norm2)."""
    if not x.is_cuda or not x.is_contiguous():
        raise BqError("x must be a contiguous CUDA tensor")
    cand = np.ascontiguousarray(blocks, np.int32)
    n = x.numel()
    if workspace is None:
        workspace = torch.empty(max(workspace_bytes(x.dtype, n), 256), dtype=torch.uint8, device=x.device)
    if sums_out is None:
        sums_out = torch.empty(cand.size + 1, dtype=torch.float64, device=x.device)
    with torch.cuda.device(x.device):
        rc = _lib().bqt_block_errors(x.data_ptr(), _DT[x.dtype], n, cb.handle, cand.ctypes.data, cand.size, workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size(), sums_out.data_ptr(), _stream(x))
    _check(rc, "bqt_block_errors")
    return sums_out


def pick_block(blocks, sums, max_rel_rms: float) -> int:
    """``bqt_pick_block`` on host values (sums: len(blocks) + 1 doubles)."""
    cand = np.ascontiguousarray(blocks, np.int32)
    s = np.ascontiguousarray(sums, np.float64)
    if s.size != cand.size + 1:
        raise BqError("sums must hold one value per candidate and the squared norm")
    out = ctypes.c_int(0)
    _check(_lib().bqt_pick_block(cand.ctypes.data, s.ctypes.data, cand.size, float(max_rel_rms), ctypes.byref(out)), "bqt_pick_block")
    return int(out.value)


def autotune_block(x: torch.Tensor, blocks, cb: Codebook, max_rel_rms: float, workspace: torch.Tensor | None = None):
    """Measures the candidates on x and picks: returns (block, relative rms error per candidate).  Synchronises (the
    sums are read on the host)."""
    sums = block_errors(x, blocks, cb, workspace).cpu().numpy()
    rel = np.sqrt(sums[:-1] / sums[-1]) if sums[-1] > 0 else np.zeros(len(sums) - 1)
    return pick_block(blocks, sums, max_rel_rms), rel
