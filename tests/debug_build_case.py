"""Run as a script by tests/test_gpu_debug_build.py with BQ_LIB pointing at libbq_debug.so: the debug build gives the same
bits as the oracle on ragged tensors, takes the documented in-place roundtrip, and refuses overlapping buffers with
BQ_ERR_ASSERT before anything is launched."""
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

import oracle  # noqa: E402
import paper_2407_19775_b200 as bq  # noqa: E402
from oracle import bq4_oracle  # noqa: E402
from paper_2407_19775_b200 import workloads  # noqa: E402


def main() -> None:
    assert bq.debug_build(), "this script wants the debug build of the library"
    dev = torch.device("cuda:0")
    cb = bq.Codebook(device=dev)
    ref = oracle.make_codebook()
    for rows, cut, block in ((8, 0, 256), (3, 777, 64), (2, 4095, 4096), (1, 8100, 100)):
        x = workloads.make("prefill7b", rows=rows).view(-1)
        x = x[: x.numel() - cut].contiguous()
        xd = x.to(dev)
        codes, absmax = bq.bq_quantize(xd, block, cb)
        y = bq.bq_dequantize(codes, absmax, block, cb, torch.bfloat16)
        inplace = xd.clone()
        bq.bq_roundtrip(inplace, block, cb, y_out=inplace)                   # the documented in-place form passes the assertions
        torch.cuda.synchronize()
        yr, cr, ar = oracle.roundtrip(workloads.as_numpy_bits(x), oracle.BF16, block, ref, oracle.BF16, side=True)
        assert np.array_equal(codes.cpu().numpy(), cr) and np.array_equal(absmax.cpu().numpy().view(np.uint32), ar.view(np.uint32))
        assert np.array_equal(workloads.as_numpy_bits(y.cpu()), yr) and np.array_equal(workloads.as_numpy_bits(inplace.cpu()), yr)
        # 4 bits through the same build
        cb4 = bq.Codebook4()
        packed, am4 = bq.bq4_quantize(xd, block, cb4)
        torch.cuda.synchronize()
        pr, ar4 = bq4_oracle.quantize(workloads.as_numpy_bits(x), bq4_oracle.BF16, block, bq4_oracle.make_codebook())
        assert np.array_equal(packed.cpu().numpy(), pr) and np.array_equal(am4.cpu().numpy().view(np.uint32), ar4.view(np.uint32))

    # overlapping buffers: refused with status 11, nothing written
    n, block = 4096, 64
    buf = torch.zeros(4 * n, dtype=torch.uint8, device=dev)
    x = buf[: 2 * n].view(torch.bfloat16)
    x.copy_(workloads.make("prefill7b", rows=1).view(-1)[:n])
    before = buf.clone()
    absmax = torch.empty(n // block, dtype=torch.float32, device=dev)

    def refused(fn):
        try:
            fn()
        except bq.BqError as e:
            assert "status 11" in str(e) and "debug assertion failed" in str(e), str(e)
            return True
        return False

    assert refused(lambda: bq.bq_quantize(x, block, cb, buf[n: 2 * n], absmax))                      # codes over the second half of x
    assert refused(lambda: bq.bq_roundtrip(x, block, cb, y_out=buf[16: 16 + 2 * n].view(torch.bfloat16)))   # y shifted by 16 bytes over x
    codes = buf[2 * n: 3 * n]
    assert refused(lambda: bq.bq_dequantize(codes, absmax, block, cb, torch.bfloat16, buf[2 * n - 64: 4 * n - 64].view(torch.bfloat16)))
    assert refused(lambda: bq.bq4_quantize(x, block, bq.Codebook4(), buf[2 * n - 8: 2 * n - 8 + n // 2], absmax))
    torch.cuda.synchronize()
    assert torch.equal(buf, before)
    print("debug build ok")


if __name__ == "__main__":
    main()
