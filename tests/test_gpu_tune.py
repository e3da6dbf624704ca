"""GPU parity of the block-size selection against its CPU oracle, through the C ABI.  The error sums are fp64 sums
in a different order on the two sides: they must agree to 1e-11 relative (the GPU's sequential share per thread is at
most n / 262144 terms, each addition within 2^-53 relative of a sum of non-negative terms); the choice is an integer
decided on both sides by the same fp64 comparison, and must be equal for bounds that do not sit on a candidate's error."""
import numpy as np
import pytest
import torch

import oracle
from oracle import tune_oracle as to
from paper_2407_19775_b200 import workloads

pytestmark = pytest.mark.gpu
F32, F16, BF16 = 0, 1, 2
DT = {torch.float32: F32, torch.float16: F16, torch.bfloat16: BF16}
RTOL = 1e-11


def bits(t: torch.Tensor) -> np.ndarray:
    return workloads.as_numpy_bits(t.cpu())


def check(bq, x: torch.Tensor, blocks):
    cb = bq.Codebook()
    cb_ref = oracle.make_codebook()
    flat = x.reshape(-1).contiguous()
    err_ref, norm_ref = to.block_errors(bits(flat), DT[flat.dtype], blocks, cb_ref)
    sums = bq.tune.block_errors(flat.cuda(), blocks, cb).cpu().numpy()
    assert sums.shape == (len(blocks) + 1,)
    assert np.allclose(sums[:-1], err_ref, rtol=RTOL, atol=0) and np.isclose(sums[-1], norm_ref, rtol=RTOL, atol=0)
    again = bq.tune.block_errors(flat.cuda(), blocks, cb).cpu().numpy()
    assert np.array_equal(sums.view(np.uint64), again.view(np.uint64))      # a fixed summation order: the same bits every time
    rel = np.sqrt(np.array(err_ref) / norm_ref) if norm_ref > 0 else np.zeros(len(blocks))
    # bounds between the candidates' errors (never on one), below all of them and above all of them
    srt = np.sort(np.unique(rel))
    bounds = [srt[0] * 0.5, srt[-1] * 2 + 1e-3] + [float(np.sqrt(a * b)) for a, b in zip(srt[:-1], srt[1:]) if b > a * (1 + 1e-6)]
    for tol in bounds:
        assert bq.tune.pick_block(blocks, sums, tol) == to.pick_block(blocks, err_ref, norm_ref, tol)
    return sums


@pytest.mark.parametrize("name,rows,blocks", [("tiny", None, [64, 256, 1024]), ("prefill7b", 48, [64, 256, 1024, 4096]),
                                              ("decode70b", 64, [32, 64, 4096]), ("moe_prefill", 24, [2048, 64]), ("sweep1g", 24, [64, 256, 1024, 4096])])
def test_workloads(bq, name, rows, blocks):
    sums = check(bq, workloads.make(name, rows=rows), blocks)
    assert sums[-1] > 0 and np.all(sums[:-1] > 0)


@pytest.mark.parametrize("tdt", [torch.float32, torch.bfloat16, torch.float16])
def test_ragged_unaligned_and_degenerate(bq, tdt):
    g = torch.Generator().manual_seed(31)
    x = (torch.randn(70000, generator=g) * 2).to(tdt)
    x[1000] = 90.0
    for n in (69999, 4097, 7, 1):
        check(bq, x[:n].clone(), [64, 100, 4096])
    cb = bq.Codebook()
    cb_ref = oracle.make_codebook()
    xd = x.cuda()[3:3 + 5000]                                     # not 16-byte aligned: the scalar path of the sums
    err_ref, norm_ref = to.block_errors(bits(x[3:3 + 5000]), DT[tdt], [64, 512], cb_ref)
    sums = bq.tune.block_errors(xd, [64, 512], cb).cpu().numpy()
    assert np.allclose(sums[:-1], err_ref, rtol=RTOL, atol=0) and np.isclose(sums[-1], norm_ref, rtol=RTOL, atol=0)
    z = torch.zeros(4096, dtype=tdt)
    zs = bq.tune.block_errors(z.cuda(), [64, 256], cb).cpu().numpy()
    assert np.array_equal(zs, np.zeros(3)) and bq.tune.pick_block([64, 256], zs, 0.0) == 256
    empty = bq.tune.block_errors(z.cuda()[:0], [64, 256], cb).cpu().numpy()
    assert np.array_equal(empty, np.zeros(3))


def test_autotune_on_a_large_tensor_by_properties(bq):
    """At a size the oracle does not reach: the sums equal torch's fp64 sums over the library's own roundtrip (whose
    parity is tested elsewhere), errors grow with the block size on this outlier-channel tensor, and the pick follows."""
    cb = bq.Codebook()
    x = workloads.make("sweep1g", rows=2048).reshape(-1).cuda()
    blocks = [64, 256, 1024, 4096]
    sums = bq.tune.block_errors(x, blocks, cb).cpu().numpy()
    xd = x.double()
    assert np.isclose(sums[-1], float((xd * xd).sum().item()), rtol=RTOL, atol=0)
    for c, b in enumerate(blocks):
        y = bq.bq_roundtrip(x, b, cb)
        d = xd - y.double()
        assert np.isclose(sums[c], float((d * d).sum().item()), rtol=RTOL, atol=0)
    assert np.all(np.diff(sums[:-1]) > 0)
    block, rel = bq.autotune_block(x, blocks, cb, max_rel_rms=float(np.sqrt(sums[2] / sums[-1]) * 1.01))
    assert block == 1024 and np.allclose(rel, np.sqrt(sums[:-1] / sums[-1]))
    assert bq.autotune_block(x, blocks, cb, max_rel_rms=1e-6)[0] == 64
