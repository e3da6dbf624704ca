"""Every fp32 bit pattern of a normalised value xhat in [-1, 1] through the tuned kernels' folded
single-lookup search, against the general kernels' 8-step search over the round-down midpoints,
on the device; a strided sample of whole blocks of every chunk also goes to the CPU oracle.

The patterns are laid out as fp32 blocks of 64 whose first element is 1.0, so that the block's
absmax is 1 and xhat = x / 1 is the pattern itself.  There are 1,065,353,217 patterns from +0.0
to +1.0 and as many from -0.0 to -1.0; 63 per block, 2^22 blocks (1 GiB) per chunk, generated on
the device.  The tuned kernel takes the aligned tensor (the persistent flavour on the whole
chunk, the small-tensor flavour on 8 Mi-element slices of it); a copy of the tensor that starts
one element off a 16-byte boundary takes the general kernel.
"""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu

ONE = 0x3F800000
BLOCKS_PER_CHUNK = 1 << 22
PER_BLOCK = 63


def _chunk(first_pattern: int, negative: bool, dev) -> torch.Tensor:
    """2^22 blocks of [1.0, 63 consecutive patterns]; patterns past 1.0 repeat 1.0."""
    blk = torch.arange(BLOCKS_PER_CHUNK, device=dev, dtype=torch.int32)[:, None]
    pos = torch.arange(64, device=dev, dtype=torch.int32)[None, :]
    pat = (blk * PER_BLOCK + (pos - 1) + first_pattern).clamp_(max=ONE)
    if negative:
        pat |= torch.iinfo(torch.int32).min
    pat[:, 0] = ONE
    return pat.view(torch.float32).view(-1)


def test_every_pattern_of_xhat_tuned_search_equals_general_search(bq, cb):
    dev = torch.device("cuda:0")
    gcb = bq.Codebook(device=dev)
    assert gcb.folded
    n = BLOCKS_PER_CHUNK * 64
    nb = BLOCKS_PER_CHUNK
    holder = torch.empty(n + 1, dtype=torch.float32, device=dev)
    shifted = holder[1:]                                          # 4 bytes off the allocation base: general kernels
    codes_t = torch.empty(n, dtype=torch.uint8, device=dev)
    codes_g = torch.empty(n, dtype=torch.uint8, device=dev)
    codes_l = torch.empty(n, dtype=torch.uint8, device=dev)
    am_t = torch.empty(nb, dtype=torch.float32, device=dev)
    am_g = torch.empty(nb, dtype=torch.float32, device=dev)
    am_l = torch.empty(nb, dtype=torch.float32, device=dev)
    y_t = torch.empty(n, dtype=torch.float32, device=dev)
    y_g = torch.empty(n, dtype=torch.float32, device=dev)
    lite = 1 << 23                                                # elements per slice of the small-tensor flavour
    sample_blocks = torch.arange(0, nb, 1021, device=dev)
    covered = 0
    for negative in (False, True):
        for first in range(0, ONE + 1, BLOCKS_PER_CHUNK * PER_BLOCK):
            x = _chunk(first, negative, dev)
            shifted.copy_(x)
            bq.bq_quantize(x, 64, gcb, codes_t, am_t)                                  # persistent tuned kernel
            bq.bq_quantize(shifted, 64, gcb, codes_g, am_g)                            # general kernel
            for s in range(0, n, lite):                                               # small-tensor tuned kernel
                bq.bq_quantize(x[s:s + lite], 64, gcb, codes_l[s:s + lite], am_l[s // 64:(s + lite) // 64])
            bq.bq_roundtrip(x, 64, gcb, y_out=y_t)
            bq.bq_roundtrip(shifted, 64, gcb, y_out=y_g)
            where = f"patterns from {first:#x}, {'negative' if negative else 'positive'}"
            assert torch.equal(codes_t, codes_g), "persistent kernel, " + where
            assert torch.equal(codes_l, codes_g), "small-tensor kernel, " + where
            assert torch.equal(y_t.view(torch.int32), y_g.view(torch.int32)), "fused roundtrip, " + where
            assert bool((am_t == 1.0).all()) and bool((am_g == 1.0).all()) and bool((am_l == 1.0).all())
            # a strided sample of whole blocks against the oracle (codes, absmax and the dequantised values)
            xs = x.view(nb, 64)[sample_blocks].reshape(-1).cpu().numpy()
            yr, cr, ar = oracle.roundtrip(xs, oracle.F32, 64, cb, oracle.F32, side=True)
            assert np.array_equal(codes_t.view(nb, 64)[sample_blocks].reshape(-1).cpu().numpy(), cr), "oracle, " + where
            assert np.array_equal(y_t.view(nb, 64)[sample_blocks].reshape(-1).cpu().numpy().view(np.uint32), yr.view(np.uint32))
            assert np.all(ar == 1.0)
            covered += min(ONE + 1 - first, BLOCKS_PER_CHUNK * PER_BLOCK)
            del x
    assert covered == 2 * (ONE + 1)
