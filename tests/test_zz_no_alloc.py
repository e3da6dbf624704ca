"""mmd_linear_static: the decomposed linear layer with the library's built-in scratch array,
for callers that cannot obtain device memory when they call (their own pool holds the whole
GPU, or an allocation's device-wide synchronisation is not acceptable in their loop).

Its results are checked against mmd_linear (the entry point that takes a caller's workspace)
on two calls in a row with different activations, so that anything the first call left in the
shared array would show in the second.  Both entry points run the same kernels, and the test
holds them to the tolerance of the other GPU tests of this layer: one rounding of the result
plus one per accumulated side product, 2^-23 |y| + (side columns + 2) 2^-22 sum_j |x_j w_j|.
Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2407_19775_b200 import workloads

pytestmark = pytest.mark.gpu


def tolerance(lin, X, y_ref):
    _, _, wside, idx = lin.view()
    side_cols = wside.shape[1]
    if side_cols == 0:
        return torch.zeros_like(y_ref, dtype=torch.float32)
    xs = X[:, idx.long()].float().abs()
    sabs = xs @ wside[:, :idx.numel()].float().abs().T
    return 2.0 ** -23 * y_ref.float().abs() + (side_cols + 2) * 2.0 ** -22 * sabs


def test_static_scratch_matches_caller_workspace_twice_in_a_row(bq):
    X, W, idx = workloads.make_linear("mmd_decode70b", out_features=1024)      # 64 x 8192 fp16 activations, a decode step
    X, W = X.cuda(), W.cuda()
    lin = bq.DecomposedLinear(W, idx)
    X2 = torch.roll(X, shifts=3, dims=0) * 0.5                                   # other rows, other row scales
    for path in (bq.mmd.PATH_AUTO, bq.mmd.PATH_GENERAL):
        for x in (X, X2):
            y = torch.empty((x.shape[0], lin.N), dtype=torch.float32, device=x.device)
            lin.linear_static(x, path=path, y_out=y)
            assert lin.kernel_status() == 0
            y_ref = lin.linear(x, torch.float32, path=path)
            assert lin.kernel_status() == 0
            assert torch.all((y - y_ref).abs() <= tolerance(lin, x, y_ref))
            assert y_ref.abs().max() > 0
    # 16-bit output, fewer rows than the call before it
    y16 = lin.linear_static(X[:5])
    assert torch.all((y16.float() - lin.linear(X[:5]).float()).abs() <= tolerance(lin, X[:5], y16) + 2.0 ** -10 * y16.float().abs())
    lin.close()


def test_static_scratch_rejects_what_does_not_fit(bq):
    X, W, idx = workloads.make_linear("mmd_decode70b", out_features=64)
    lin = bq.DecomposedLinear(W.cuda(), idx)
    _, need = lin.workspace_layout(600)
    assert need > bq.mmd.STATIC_SCRATCH_BYTES
    big = torch.zeros((600, lin.K), dtype=W.dtype, device="cuda")
    with pytest.raises(bq.BqError, match="static array holds"):
        lin.linear_static(big)
    _, fits = lin.workspace_layout(64)
    assert fits <= bq.mmd.STATIC_SCRATCH_BYTES
    lin.close()


def test_static_entry_answers_bad_arguments_like_the_workspace_entry(bq):
    """Bad element type, bad path and zero rows: the two entry points return the same status, before any launch,
    whether or not the row count would fit the built-in array."""
    from paper_2407_19775_b200.mmd import _lib
    X, W, idx = workloads.make_linear("mmd_decode70b", out_features=64)
    lin = bq.DecomposedLinear(W.cuda(), idx)
    L = _lib()
    x = X.cuda()
    y = torch.empty((x.shape[0], lin.N), dtype=torch.float32, device="cuda")
    ws = lin.workspace(x.shape[0])
    stream = torch.cuda.current_stream().cuda_stream
    BF16, F32 = 2, 0                                                             # the weights are fp16: bf16 output is refused
    for M in (0, x.shape[0], 600):                                               # 600 rows do not fit the built-in array
        for ydt, path in ((BF16, 0), (F32, 99), (F32, -1), (BF16, 99)):
            a = L.mmd_linear(lin.handle, x.data_ptr(), M, y.data_ptr(), ydt, ws.data_ptr(), ws.numel(), path, stream)
            b = L.mmd_linear_static(lin.handle, x.data_ptr(), M, y.data_ptr(), ydt, path, stream)
            assert a == b and a != 0, (M, ydt, path, a, b)
    assert L.mmd_linear_static(lin.handle, x.data_ptr(), 0, y.data_ptr(), F32, 0, stream) == 0
    assert L.mmd_linear_static(None, x.data_ptr(), 4, y.data_ptr(), F32, 0, stream) == L.mmd_linear(None, x.data_ptr(), 4, y.data_ptr(), F32, ws.data_ptr(), ws.numel(), 0, stream)
    lin.close()
