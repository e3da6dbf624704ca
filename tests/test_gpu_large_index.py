"""GPU parity past 2^32 elements: every element offset, byte offset and block number of the kernels is a 64-bit
quantity, and this is the test that would show a 32-bit one.

The tensor is a seeded 64 Mi-element pattern (the first 8192 rows of `sweep1g`) repeated 66 times and a bit, each
repetition scaled by a power of two (exact in bf16) that cycles with period five, so that repetition r holds the
same values as repetition r - 5.  The oracle computes the five distinct repetitions (whole, on all host cores) and
the ragged tail; every repetition of the device's output is then compared with its oracle image on the device,
so the WHOLE tensor is checked against the oracle, including the 128 Mi elements that lie past element 2^32."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2407_19775_b200 import workloads

pytestmark = pytest.mark.gpu

THREADS = max(1, (os.cpu_count() or 2))
BLOCK = 256
SCALES = [0.25, 0.5, 1.0, 2.0, 4.0]


def _bits(t):
    return workloads.as_numpy_bits(t)


def test_whole_tensor_of_more_than_2_32_elements(bq):
    dev = torch.device("cuda:0")
    cb = bq.Codebook(device=dev)
    ref = oracle.make_codebook()
    pat = workloads.make("sweep1g", rows=8192).view(-1)                     # 2^26 bf16 elements
    L = pat.numel()
    assert L == 1 << 26
    n = (1 << 32) + (1 << 27) + 100                                         # 66 whole repetitions and a ragged block of 100
    reps = (n + L - 1) // L

    # the oracle's image of each distinct repetition
    want = []
    for s in SCALES:
        xs = (pat.float() * s).to(torch.bfloat16)
        assert torch.equal(xs.float(), pat.float() * s)                      # the scaling is exact
        y, codes, absmax = oracle.roundtrip_sharded(_bits(xs), oracle.BF16, BLOCK, ref, oracle.BF16, THREADS)
        want.append((torch.from_numpy(codes).to(dev), torch.from_numpy(absmax).to(dev),
                     workloads.from_numpy_bits(y, torch.bfloat16).to(dev)))

    pd = pat.to(dev)
    x = torch.empty(n, dtype=torch.bfloat16, device=dev)
    for r in range(reps):
        m = min(L, n - r * L)
        x[r * L: r * L + m] = (pd[:m].float() * SCALES[r % 5]).to(torch.bfloat16)
    nb = (n + BLOCK - 1) // BLOCK
    codes = torch.empty(n, dtype=torch.uint8, device=dev)
    absmax = torch.empty(nb, dtype=torch.float32, device=dev)
    y = torch.empty_like(x)
    bq.bq_quantize(x, BLOCK, cb, codes, absmax)
    bq.bq_dequantize(codes, absmax, BLOCK, cb, torch.bfloat16, y)
    torch.cuda.synchronize()

    def check(tag, codes_d, absmax_d, y_d):
        for r in range(reps):
            m = min(L, n - r * L)
            whole = (m // BLOCK) * BLOCK                                     # the ragged block of the last repetition is checked below
            wc, wa, wy = want[r % 5]
            if codes_d is not None:
                assert torch.equal(codes_d[r * L: r * L + whole], wc[:whole]), (tag, "codes", r)
                b0 = r * (L // BLOCK)
                assert torch.equal(absmax_d[b0: b0 + whole // BLOCK].view(torch.int32), wa[: whole // BLOCK].view(torch.int32)), (tag, "absmax", r)
            assert torch.equal(y_d[r * L: r * L + whole].view(torch.int16), wy[:whole].view(torch.int16)), (tag, "y", r)

    check("separate calls", codes, absmax, y)

    # the ragged last block (100 elements, the very end of the tensor) against the oracle directly
    t0 = (n // BLOCK) * BLOCK
    tail = x[t0:].cpu()
    ty, tc, ta = oracle.roundtrip(_bits(tail), oracle.BF16, BLOCK, ref, oracle.BF16, side=True)
    assert np.array_equal(codes[t0:].cpu().numpy(), tc)
    assert np.array_equal(absmax[nb - 1:].cpu().numpy().view(np.uint32), ta.view(np.uint32))
    assert np.array_equal(_bits(y[t0:].cpu()), ty)

    # the fused roundtrip with side outputs, into fresh buffers
    codes.fill_(0xA5)
    absmax.fill_(-1.0)
    y.fill_(0)
    bq.bq_roundtrip(x, BLOCK, cb, y_out=y, codes_out=codes, absmax_out=absmax)
    torch.cuda.synchronize()
    check("fused", codes, absmax, y)
    assert np.array_equal(codes[t0:].cpu().numpy(), tc) and np.array_equal(_bits(y[t0:].cpu()), ty)

    # in place, without side outputs
    bq.bq_roundtrip(x, BLOCK, cb, y_out=x)
    torch.cuda.synchronize()
    check("in place", None, None, x)
    assert np.array_equal(_bits(x[t0:].cpu()), ty)


def test_four_bit_codes_of_more_than_2_32_elements(bq):
    """The same tensor through the 4-bit calls.  The numpy oracle takes the first 2 Mi elements of each of the five distinct
    repetitions; every repetition of the device's output then has to equal, on the device, the repetition five before it
    (the same values), so the oracle's image of the low repetitions carries over the whole tensor, past byte 2^31 of the
    packed codes and past element 2^32 of the input."""
    from oracle import bq4_oracle
    dev = torch.device("cuda:0")
    cb4 = bq.Codebook4()
    ref4 = bq4_oracle.make_codebook()
    pat = workloads.make("sweep1g", rows=8192).view(-1)
    L = pat.numel()
    n = (1 << 32) + (1 << 27) + 100
    reps = (n + L - 1) // L
    pd = pat.to(dev)
    x = torch.empty(n, dtype=torch.bfloat16, device=dev)
    for r in range(reps):
        m = min(L, n - r * L)
        x[r * L: r * L + m] = (pd[:m].float() * SCALES[r % 5]).to(torch.bfloat16)
    nb = (n + BLOCK - 1) // BLOCK
    packed = torch.empty((n + 1) // 2, dtype=torch.uint8, device=dev)
    absmax = torch.empty(nb, dtype=torch.float32, device=dev)
    bq.bq4_quantize(x, BLOCK, cb4, packed, absmax)
    y = bq.bq4_dequantize(packed, absmax, n, BLOCK, cb4, torch.bfloat16)
    torch.cuda.synchronize()
    head = 1 << 21
    for r in range(5):
        xs = (pat[:head].float() * SCALES[r]).to(torch.bfloat16)
        wp, wa = bq4_oracle.quantize(_bits(xs), bq4_oracle.BF16, BLOCK, ref4)
        wy = bq4_oracle.dequantize(wp, wa, head, BLOCK, ref4, bq4_oracle.BF16)
        assert np.array_equal(packed[r * L // 2: (r * L + head) // 2].cpu().numpy(), wp), r
        assert np.array_equal(absmax[r * L // BLOCK: (r * L + head) // BLOCK].cpu().numpy().view(np.uint32), wa.view(np.uint32)), r
        assert np.array_equal(_bits(y[r * L: r * L + head].cpu()), wy), r
    for r in range(5, reps):
        m = min(L, n - r * L)
        whole = (m // BLOCK) * BLOCK
        a, b = r * L, (r - 5) * L
        assert torch.equal(packed[a // 2: (a + whole) // 2], packed[b // 2: (b + whole) // 2]), ("packed", r)
        assert torch.equal(absmax[a // BLOCK: (a + whole) // BLOCK].view(torch.int32), absmax[b // BLOCK: (b + whole) // BLOCK].view(torch.int32)), ("absmax", r)
        assert torch.equal(y[a: a + whole].view(torch.int16), y[b: b + whole].view(torch.int16)), ("y", r)
    # the ragged last block against the oracle directly
    t0 = (n // BLOCK) * BLOCK
    tail = x[t0:].cpu()
    wp, wa = bq4_oracle.quantize(_bits(tail), bq4_oracle.BF16, BLOCK, ref4)
    assert np.array_equal(packed[t0 // 2:].cpu().numpy(), wp)
    assert np.array_equal(absmax[nb - 1:].cpu().numpy().view(np.uint32), wa.view(np.uint32))
    assert np.array_equal(_bits(y[t0:].cpu()), bq4_oracle.dequantize(wp, wa, n - t0, BLOCK, ref4, bq4_oracle.BF16))


def test_boundary_transfer_of_more_than_2_32_elements(bq):
    """The same tensor handed across a (loop-back) shard boundary in 133 pieces of 32 Mi elements through three mailbox
    slots: what arrives is the oracle's roundtrip of every repetition, piece offsets past 2^32 included."""
    from paper_2407_19775_b200 import transport
    dev = torch.device("cuda:0")
    cb = bq.Codebook(device=dev)
    ref = oracle.make_codebook()
    pat = workloads.make("sweep1g", rows=8192).view(-1)
    L = pat.numel()
    n = (1 << 32) + (1 << 27) + 100
    reps = (n + L - 1) // L
    want = []
    for s in SCALES:
        xs = (pat.float() * s).to(torch.bfloat16)
        y, _, _ = oracle.roundtrip_sharded(_bits(xs), oracle.BF16, BLOCK, ref, oracle.BF16, THREADS)
        want.append(workloads.from_numpy_bits(y, torch.bfloat16).to(dev))
    pd = pat.to(dev)
    x = torch.empty(n, dtype=torch.bfloat16, device=dev)
    for r in range(reps):
        m = min(L, n - r * L)
        x[r * L: r * L + m] = (pd[:m].float() * SCALES[r % 5]).to(torch.bfloat16)
    y = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    chunk, slots = 1 << 25, 3
    rx = transport.Receiver(cb, chunk, min_block=BLOCK, slots=slots)
    tx = transport.Sender(cb, rx.export(), transport.STORE)
    s_send, s_recv = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    torch.cuda.synchronize()
    transport.transfer(tx, rx, x, BLOCK, y, s_send, s_recv)
    s_recv.synchronize()
    s_send.synchronize()
    assert len(transport.plan(n, BLOCK, chunk, slots)) == 133
    for r in range(reps):
        m = min(L, n - r * L)
        whole = (m // BLOCK) * BLOCK
        assert torch.equal(y[r * L: r * L + whole].view(torch.int16), want[r % 5][:whole].view(torch.int16)), r
    t0 = (n // BLOCK) * BLOCK
    ty = oracle.roundtrip(_bits(x[t0:].cpu()), oracle.BF16, BLOCK, ref, oracle.BF16)
    assert np.array_equal(_bits(y[t0:].cpu()), ty)
    tx.close()
    rx.close()
