"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded bytes.  Codes, absmax and dequantised output must be bit-identical."""
import os

import numpy as np
import pytest
import torch

import oracle
from helpers import midpoints, reciprocal_sensitive_pairs, round_down32
from paper_2407_19775_b200 import workloads

pytestmark = pytest.mark.gpu

ODT = {torch.float32: oracle.F32, torch.float16: oracle.F16, torch.bfloat16: oracle.BF16}
THREADS = max(1, (os.cpu_count() or 2))
CANARY = 0xA5


@pytest.fixture(scope="module")
def gcb(bq):
    return bq.Codebook(device="cuda:0")


def _bits(t):
    return workloads.as_numpy_bits(t)


def _padded(n, dtype, dev, pad=64, lead=0):
    """An output buffer of n elements that starts `lead` bytes into a (512-byte aligned) allocation,
    with canary bytes before and after it."""
    esz = torch.empty(0, dtype=dtype).element_size()
    assert lead % esz == 0
    raw = torch.full((lead + n * esz + pad,), CANARY, dtype=torch.uint8, device=dev)
    return (raw, lead), raw[lead: lead + n * esz].view(dtype)


def _canary_ok(raw_lead, nbytes):
    raw, lead = raw_lead
    return bool((raw[:lead] == CANARY).all().item()) and bool((raw[lead + nbytes:] == CANARY).all().item())


def check_all_ops(bq, gcb, cb, x_cpu: torch.Tensor, block: int, ydtypes=None, offset_elems: int = 0, out_lead=None):
    """quantize, dequantize, roundtrip (with and without side outputs) against the oracle.
    `out_lead` = bytes by which (y, codes, absmax) outputs are shifted off their allocation's base."""
    ylead, clead, alead = out_lead or (0, 0, 0)
    dev = torch.device("cuda:0")
    x_cpu = x_cpu.contiguous().view(-1)
    n = x_cpu.numel()
    nb = (n + block - 1) // block
    xdt = x_cpu.dtype
    if offset_elems:
        holder = torch.empty(n + offset_elems, dtype=xdt, device=dev)
        xd = holder[offset_elems:]
        xd.copy_(x_cpu)
    else:
        xd = x_cpu.to(dev)
    craw, codes = _padded(n, torch.uint8, dev, lead=clead)
    araw, absmax = _padded(nb, torch.float32, dev, lead=alead)
    bq.bq_quantize(xd, block, gcb, codes, absmax)
    ref_y, ref_c, ref_a = {}, None, None
    for ydt in (ydtypes or [xdt]):
        y, c, a = oracle.roundtrip_sharded(_bits(x_cpu), ODT[xdt], block, cb, ODT[ydt], THREADS)
        ref_y[ydt], ref_c, ref_a = y, c, a
    torch.cuda.synchronize()
    assert np.array_equal(codes.cpu().numpy(), ref_c), "codes"
    assert np.array_equal(absmax.cpu().numpy().view(np.uint32), ref_a.view(np.uint32)), "absmax"
    assert _canary_ok(craw, n) and _canary_ok(araw, nb * 4)
    for ydt, yref in ref_y.items():
        esz = torch.empty(0, dtype=ydt).element_size()
        ylead_e = ylead - ylead % esz
        yraw, y = _padded(n, ydt, dev, lead=ylead_e)
        bq.bq_dequantize(codes, absmax, block, gcb, ydt, y)
        y2raw, y2 = _padded(n, ydt, dev, lead=ylead_e)
        bq.bq_roundtrip(xd, block, gcb, y_out=y2)
        y3raw, y3 = _padded(n, ydt, dev, lead=ylead_e)
        c3raw, c3 = _padded(n, torch.uint8, dev, lead=clead)
        a3raw, a3 = _padded(nb, torch.float32, dev, lead=alead)
        bq.bq_roundtrip(xd, block, gcb, y_out=y3, codes_out=c3, absmax_out=a3)
        torch.cuda.synchronize()
        assert np.array_equal(_bits(y.cpu()), yref), f"dequantize {ydt}"
        assert np.array_equal(_bits(y2.cpu()), yref), f"roundtrip {ydt}"
        assert np.array_equal(_bits(y3.cpu()), yref), f"roundtrip+side {ydt}"
        assert np.array_equal(c3.cpu().numpy(), ref_c) and np.array_equal(a3.cpu().numpy().view(np.uint32), ref_a.view(np.uint32))
        for raw, nbytes in ((yraw, n * esz), (y2raw, n * esz), (y3raw, n * esz), (c3raw, n), (a3raw, nb * 4)):
            assert _canary_ok(raw, nbytes)


# ------------------------------------------------------------------------------- the configs

def test_codebook_matches_oracle(bq, gcb, cb):
    assert np.array_equal(gcb.values.view(np.uint32), cb.view(np.uint32))
    assert gcb.folded


def test_config_tiny(bq, gcb, cb):
    check_all_ops(bq, gcb, cb, workloads.make("tiny"), 64, ydtypes=[torch.float32, torch.bfloat16, torch.float16])


def test_config_prefill7b(bq, gcb, cb):
    check_all_ops(bq, gcb, cb, workloads.make("prefill7b"), 256)


def test_config_decode70b(bq, gcb, cb):
    check_all_ops(bq, gcb, cb, workloads.make("decode70b"), 64)


def _whole_tensor(bq, gcb, cb, name, blocks, chunk=1 << 26):
    """Full-size run in the launch configuration the benchmark times.  EVERY code, every absmax and
    every output element of quantize, dequantize, the fused roundtrip and the roundtrip with side
    outputs is compared with the oracle, which runs on all host cores over contiguous ranges of
    whole blocks, 64 Mi elements at a time so that host memory stays bounded.  Device-side
    properties (textbook absmax, the error bound) are checked on every element as well."""
    dev = torch.device("cuda:0")
    x_cpu = workloads.make(name).view(-1)
    n = x_cpu.numel()
    xd = x_cpu.to(dev)
    xb = _bits(x_cpu)
    odt = ODT[x_cpu.dtype]
    for block in blocks:
        assert n % block == 0 and chunk % block == 0
        nb = n // block
        codes, absmax = bq.bq_quantize(xd, block, gcb)
        y = bq.bq_dequantize(codes, absmax, block, gcb, x_cpu.dtype)
        y2 = bq.bq_roundtrip(xd, block, gcb).view(-1)
        y3 = torch.empty_like(y)
        c3, a3 = torch.empty_like(codes), torch.empty_like(absmax)
        bq.bq_roundtrip(xd, block, gcb, y_out=y3, codes_out=c3, absmax_out=a3)
        torch.cuda.synchronize()
        ref_absmax = xd.view(nb, block).abs().amax(dim=1).float()
        assert torch.equal(absmax.view(torch.int32), ref_absmax.view(torch.int32))
        for s in range(0, n, chunk):
            e = min(n, s + chunk)
            b0, b1 = s // block, e // block
            a_el = absmax[b0:b1].repeat_interleave(block)
            err = (xd[s:e].float() - y[s:e].float()).abs()
            bound = a_el * (0.00703125 + 2.0 ** -22) + (y[s:e].float().abs() * 2.0 ** -8)    # code gap + bf16 rounding of y
            assert bool((err <= bound).all().item())
            del a_el, err, bound
            yr, cr, ar = oracle.roundtrip_sharded(xb[s:e], odt, block, cb, odt, THREADS)
            where = f"{name} block {block} elements [{s}, {e})"
            assert np.array_equal(codes[s:e].cpu().numpy(), cr), "quantize codes, " + where
            assert np.array_equal(c3[s:e].cpu().numpy(), cr), "roundtrip side codes, " + where
            assert np.array_equal(absmax[b0:b1].cpu().numpy().view(np.uint32), ar.view(np.uint32)), "absmax, " + where
            assert np.array_equal(a3[b0:b1].cpu().numpy().view(np.uint32), ar.view(np.uint32)), "side absmax, " + where
            assert np.array_equal(_bits(y[s:e].cpu()), yr), "dequantize, " + where
            assert np.array_equal(_bits(y2[s:e].cpu()), yr), "roundtrip, " + where
            assert np.array_equal(_bits(y3[s:e].cpu()), yr), "roundtrip with side outputs, " + where
        del codes, absmax, y, y2, y3, c3, a3


def test_config_moe_prefill_full_size(bq, gcb, cb):
    _whole_tensor(bq, gcb, cb, "moe_prefill", [2048])


def test_config_sweep1g_full_size(bq, gcb, cb):
    _whole_tensor(bq, gcb, cb, "sweep1g", [64, 256, 1024, 4096])


# ------------------------------------------------------------------------------- blocks staged through shared memory

@pytest.fixture
def staging(bq):
    """Blocks of 2048 / 4096 elements go through the kernel that stages them in shared memory with bulk
    asynchronous copies; the default is restored afterwards."""
    before = bq.set_staging(True)
    try:
        yield
    finally:
        bq.set_staging(before)


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16])
@pytest.mark.parametrize("block", [2048, 4096])
@pytest.mark.parametrize("size", ["few", "medium", "large"])
def test_staged_blocks_against_the_oracle(bq, gcb, cb, staging, dtype, block, size):
    """A handful of blocks (fewer than teams), about a thousand, and enough for every ring to wrap many
    times; a short last block that the general kernel takes; fp32 blocks of 4096 have no staged kernel
    and must come out the same through the register kernel."""
    g = torch.Generator().manual_seed(block + 3)
    n = {"few": 2 * block, "medium": 1000 * block, "large": (1 << 23) + 300 * block}[size] + 37
    x = (torch.randn(n, generator=g) * (1.0 + 30.0 * (torch.rand(n, generator=g) < 0.002))).to(dtype)
    x[block:2 * block] = 0                                         # a zero block
    check_all_ops(bq, gcb, cb, x, block)
    assert bq.kernel_status(gcb) == 0


def test_staged_config_moe_prefill_full_size(bq, gcb, cb, staging):
    _whole_tensor(bq, gcb, cb, "moe_prefill", [2048])
    assert bq.kernel_status(gcb) == 0


def test_staged_scales_outside_the_reciprocal_window_and_in_place(bq, gcb, cb, staging):
    g = torch.Generator().manual_seed(12)
    x = torch.randn(2048 * 40, generator=g)
    x[:2048 * 10] *= 1e-25                                        # absmax below 2^-64: the IEEE division
    x[2048 * 10:2048 * 20] *= 1e25
    check_all_ops(bq, gcb, cb, x.to(torch.bfloat16), 2048)
    xd = x.to(torch.bfloat16).to("cuda:0")
    bq.bq_roundtrip(xd, 2048, gcb, y_out=xd)                      # in place: a stage is read before its block's outputs are written
    torch.cuda.synchronize()
    assert np.array_equal(_bits(xd.cpu()), oracle.roundtrip(_bits(x.to(torch.bfloat16)), oracle.BF16, 2048, cb, oracle.BF16))


# ------------------------------------------------------------------------------- shapes, tails, alignment

@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16])
@pytest.mark.parametrize("block", [64, 128, 256, 512, 1024, 2048, 4096])
@pytest.mark.parametrize("size", ["small", "medium", "large"])
def test_tuned_blocks_many_tiles_and_ragged_tail(bq, gcb, cb, dtype, block, size):
    """Several tiles per warp, then blocks that do not fill a tile, then a short block.  "small" and
    "medium" (a thousand CTAs) stay below the 8 Mi-element switch of the forward kernels (tables read
    through L1), "large" is above it (persistent kernels with the tables in shared memory)."""
    g = torch.Generator().manual_seed(block + 17)
    n = {"small": 300_000, "medium": (1 << 22) + 150_000, "large": (1 << 23) + 150_000}[size]
    n = (n // block) * block + 3 * block + 37
    x = (torch.randn(n, generator=g) * (1.0 + 30.0 * (torch.rand(n, generator=g) < 0.002))).to(dtype)
    check_all_ops(bq, gcb, cb, x, block)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n,block", [(1, 64), (63, 64), (64, 64), (65, 64), (1000, 7), (257, 1), (4096, 100), (5000, 4096),
                                       (300, 3000), (2048 * 3 + 1, 2048)])
def test_small_and_odd_shapes(bq, gcb, cb, dtype, n, block):
    g = torch.Generator().manual_seed(n * 31 + block)
    x = torch.randn(n, generator=g).to(dtype)
    check_all_ops(bq, gcb, cb, x, block)


@pytest.mark.parametrize("dtype,offset", [(torch.bfloat16, 1), (torch.bfloat16, 4), (torch.float32, 1), (torch.float16, 3)])
def test_unaligned_input_pointer(bq, gcb, cb, dtype, offset):
    g = torch.Generator().manual_seed(5)
    x = torch.randn(64 * 300 + 11, generator=g).to(dtype)
    check_all_ops(bq, gcb, cb, x, 64, offset_elems=offset)


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16])
@pytest.mark.parametrize("lead", [(16, 16, 16), (16, 0, 0), (0, 8, 4), (2, 1, 4), (4, 3, 8), (48, 24, 12), (32, 16, 4)])
@pytest.mark.parametrize("n", [64 * 300 + 11, (1 << 23) + 64 * 40 + 5])
def test_unaligned_output_pointers(bq, gcb, cb, dtype, lead, n):
    if n > 100_000 and lead not in ((16, 16, 16), (2, 1, 4), (32, 16, 4)):
        pytest.skip("the large size runs three of the offsets")
    """Outputs that start off their allocation's base: y on a 16-byte but not 32-byte boundary (the wide
    stores of the dequantize kernel must not be used), on an element boundary only, codes on odd bytes,
    absmax on a 4-byte boundary; below and above the size where the persistent kernels take over."""
    g = torch.Generator().manual_seed(sum(lead) + n % 97)
    x = torch.randn(n, generator=g).to(dtype)
    check_all_ops(bq, gcb, cb, x, 64, out_lead=lead)
    if n < 100_000:
        check_all_ops(bq, gcb, cb, x, 4096, out_lead=lead)
        check_all_ops(bq, gcb, cb, x, 100, out_lead=lead)


def test_mixed_output_types(bq, gcb, cb):
    g = torch.Generator().manual_seed(8)
    x = (torch.randn(256 * 100 + 3, generator=g) * 200.0).to(torch.bfloat16)
    check_all_ops(bq, gcb, cb, x, 256, ydtypes=[torch.float32, torch.float16, torch.bfloat16])
    x = (torch.randn(64 * 100, generator=g) * 1e5).float()            # overflows fp16 on the way out
    check_all_ops(bq, gcb, cb, x, 64, ydtypes=[torch.float16, torch.bfloat16])


def test_in_place_roundtrip(bq, gcb, cb):
    x = workloads.make("prefill7b", rows=32).view(-1)
    xd = x.to("cuda:0")
    bq.bq_roundtrip(xd, 256, gcb, y_out=xd)
    torch.cuda.synchronize()
    yref = oracle.roundtrip(_bits(x), oracle.BF16, 256, cb, oracle.BF16)
    assert np.array_equal(_bits(xd.cpu()), yref)


def test_non_default_stream(bq, gcb, cb):
    x = workloads.make("decode70b", rows=8).view(-1)
    s = torch.cuda.Stream(device="cuda:0")
    with torch.cuda.stream(s):
        xd = x.to("cuda:0", non_blocking=False)
        y = bq.bq_roundtrip(xd, 64, gcb)
    s.synchronize()
    assert np.array_equal(_bits(y.cpu()), oracle.roundtrip(_bits(x), oracle.F16, 64, cb, oracle.F16))


@pytest.mark.parametrize("dtype,block,chunk", [(torch.bfloat16, 256, 256 * 300), (torch.float32, 64, 5000), (torch.float16, 4096, 4096 * 3 + 100)])
def test_host_to_host_calls(bq, gcb, cb, dtype, block, chunk):
    """bq_quantize_host / bq_dequantize_host / bq_roundtrip_host between pinned host tensors give the
    oracle's bytes; the pieces are small here so that slots are reused several times, a piece is not
    a multiple of the block (the library rounds it down) and the last piece and the last block are
    short.  Calls are enqueued back to back: the dequantize reads what the quantize before it wrote."""
    g = torch.Generator().manual_seed(block)
    n = chunk * 7 + block * 2 + 13
    x = (torch.randn(n, generator=g) * 3).to(dtype)
    nb = (n + block - 1) // block
    hb = bq.HostBoundary(gcb, dtype, chunk=chunk, slots=3, min_block=block)
    x_pin = x.pin_memory()
    c_pin = torch.full((n + 64,), CANARY, dtype=torch.uint8).pin_memory()
    a_pin = torch.empty(nb, dtype=torch.float32).pin_memory()
    y_pin = torch.empty(n, dtype=dtype).pin_memory()
    y2_pin = torch.empty(n, dtype=dtype).pin_memory()
    for _ in range(2):                                           # the second round reuses slots that are still draining
        hb.quantize(x_pin, block, c_pin[:n], a_pin)
        hb.dequantize(c_pin[:n], a_pin, block, y_pin)
        hb.roundtrip(x_pin, block, y2_pin)
    hb.wait()
    yr, cr, ar = oracle.roundtrip_sharded(_bits(x), ODT[dtype], block, cb, ODT[dtype], THREADS)
    assert np.array_equal(c_pin[:n].numpy(), cr) and bool((c_pin[n:] == CANARY).all())
    assert np.array_equal(a_pin.numpy().view(np.uint32), ar.view(np.uint32))
    assert np.array_equal(_bits(y_pin), yr) and np.array_equal(_bits(y2_pin), yr)
    # in place, and ordered behind the current stream's view of the pipe
    x2 = x_pin.clone().pin_memory()
    hb.roundtrip(x2, block, x2)
    hb.wait_on_current_stream()
    torch.cuda.current_stream().synchronize()
    assert np.array_equal(_bits(x2), yr)
    # what the pipe was not made for is refused before anything is enqueued
    with pytest.raises(bq.BqError):
        hb.roundtrip(x_pin, max(1, block // 2), y2_pin)           # below min_block
    if dtype != torch.float32:
        with pytest.raises(bq.BqError):
            hb.roundtrip(x_pin.float(), block, y2_pin.float())    # wider than the staging
    hb.close()


def test_host_to_host_calls_overlap_unless_one_reads_what_another_writes(bq, gcb, cb):
    """Calls on one pipe that do not depend on each other run into each other (three roundtrips of different tensors into
    different buffers, then all waited for at once); a call that reads a host range an unfinished call writes (the codes of a
    quantize, a tensor rounded twice in place) is held back.  Many calls in a row overflow the pipe's list of unfinished
    outputs, which must only cost a wait."""
    g = torch.Generator().manual_seed(77)
    n, block = 64 * 5000 + 19, 64
    hb = bq.HostBoundary(gcb, torch.bfloat16, chunk=64 * 700, slots=3, min_block=64)
    xs = [(torch.randn(n, generator=g) * (i + 1)).to(torch.bfloat16).pin_memory() for i in range(3)]
    ys = [torch.empty(n, dtype=torch.bfloat16).pin_memory() for _ in xs]
    for x, y in zip(xs, ys):
        hb.roundtrip(x, block, y)
    hb.wait()
    refs = [oracle.roundtrip(_bits(x), oracle.BF16, block, cb, oracle.BF16) for x in xs]
    for y, r in zip(ys, refs):
        assert np.array_equal(_bits(y), r)
    # a chain through host memory: quantize -> dequantize of the same buffers, then the result rounded again in place, twice
    c = torch.empty(n, dtype=torch.uint8).pin_memory()
    a = torch.empty((n + block - 1) // block, dtype=torch.float32).pin_memory()
    z = torch.empty(n, dtype=torch.bfloat16).pin_memory()
    hb.quantize(xs[1], block, c, a)
    hb.dequantize(c, a, block, z)
    hb.roundtrip(z, block, z)
    hb.roundtrip(z, block, z)
    hb.wait()
    twice = oracle.roundtrip(refs[1], oracle.BF16, block, cb, oracle.BF16)
    assert np.array_equal(_bits(z), oracle.roundtrip(twice, oracle.BF16, block, cb, oracle.BF16))
    # more unfinished calls than the pipe remembers outputs for
    outs = [torch.empty(n, dtype=torch.bfloat16).pin_memory() for _ in range(30)]
    for i, y in enumerate(outs):
        hb.roundtrip(xs[i % 3], block, y)
    hb.wait()
    for i, y in enumerate(outs):
        assert np.array_equal(_bits(y), refs[i % 3])
    hb.close()


def test_host_to_host_calls_from_pageable_memory(bq, gcb, cb):
    x = workloads.make("prefill7b", rows=40).view(-1)
    n, block = x.numel(), 256
    hb = bq.HostBoundary(gcb, torch.bfloat16, chunk=256 * 100, slots=2, min_block=256)
    y = torch.empty(n, dtype=torch.bfloat16)
    hb.roundtrip(x, block, y)
    hb.wait()
    assert np.array_equal(_bits(y), oracle.roundtrip(_bits(x), oracle.BF16, block, cb, oracle.BF16))
    hb.close()


def test_non_finite_inputs_stay_in_bounds(bq, gcb, cb):
    """NaN / Inf are outside the contract, but every code must be a byte written in bounds
    (canaries intact) and blocks without such values must still match the oracle."""
    g = torch.Generator().manual_seed(2)
    for dtype, block in ((torch.bfloat16, 64), (torch.float32, 256), (torch.float16, 4096)):
        n = block * 40
        x = torch.randn(n, generator=g).to(dtype)
        bad = [3 * block + 5, 3 * block + 6, 17 * block, 29 * block + block - 1]
        x[bad[0]] = float("nan"); x[bad[1]] = float("inf"); x[bad[2]] = float("-inf"); x[bad[3]] = float("nan")
        xd = x.to("cuda:0")
        craw, codes = _padded(n, torch.uint8, xd.device)
        araw, absmax = _padded(n // block, torch.float32, xd.device)
        yraw, y = _padded(n, dtype, xd.device)
        bq.bq_quantize(xd, block, gcb, codes, absmax)
        bq.bq_roundtrip(xd, block, gcb, y_out=y)
        torch.cuda.synchronize()
        esz = x.element_size()
        assert _canary_ok(craw, n) and _canary_ok(araw, (n // block) * 4) and _canary_ok(yraw, n * esz)
        clean = np.ones(n // block, bool)
        clean[[3, 17, 29]] = False
        yr, cr, ar = oracle.roundtrip(_bits(x), ODT[dtype], block, cb, ODT[dtype], side=True)
        keep = np.repeat(clean, block)
        assert np.array_equal(codes.cpu().numpy()[keep], cr[keep])
        assert np.array_equal(_bits(y.cpu())[keep], yr[keep])


# ------------------------------------------------------------------------------- degenerate values

def test_zero_blocks_negative_zero_and_sign_of_absmax(bq, gcb, cb):
    x = torch.zeros(64 * 8)
    x[5] = -0.0
    x[64] = -3.0                                      # absmax element negative -> xhat = -1 -> code 0
    x[65:128] = torch.linspace(-3.0, 3.0, 63)
    x[128:192] = 2.5                                  # all equal
    x[192:256] = -2.5
    x[256] = 1e-30; x[257] = -1e-38; x[258] = 1e-45   # tiny absmax, subnormals inside
    x[320] = 3e38; x[321] = -1e30                     # huge absmax
    x[384] = 1.0; x[385] = 2.7e-7; x[386] = -2.7e-7; x[387] = 2.8e-7; x[388] = -2.8e-7
    x[448] = -1.0; x[449] = -0.9965; x[450] = -0.99649; x[451] = -0.997; x[452] = 0.997; x[453] = 0.9964
    for dtype in (torch.float32, torch.bfloat16):
        check_all_ops(bq, gcb, cb, x.to(dtype), 64)


def test_every_breakpoint_exactly(bq, gcb, cb):
    """Blocks whose absmax is a power of two, so xhat is exactly the chosen pattern: the
    round-down midpoint of every code pair, its neighbours, and every code value."""
    pats = []
    for t in midpoints(cb):
        lo = round_down32(t)
        pats += [np.nextafter(lo, np.float32(-np.inf)), lo, np.nextafter(lo, np.float32(np.inf))]
    pats += list(cb)
    pats = np.array(pats, np.float32)
    for scale in (1.0, 2.0 ** -40, 2.0 ** 70):       # inside and outside the reciprocal window (irrelevant for fp32)
        rows = []
        for i in range(0, pats.size, 63):
            chunk = pats[i:i + 63]
            rows.append(np.concatenate([[1.0], chunk, np.zeros(63 - chunk.size, np.float32)]))
        x = torch.from_numpy((np.concatenate(rows) * np.float32(scale)).astype(np.float32))
        check_all_ops(bq, gcb, cb, x, 64)


def test_quotients_that_a_rounded_reciprocal_gets_wrong(bq, gcb, cb):
    """fp32 pairs where x / a lands exactly on a breakpoint but x * RN(1/a) lands one float
    off (or the reverse): blocks [a, x, 0, ...] through the tuned and the general kernels."""
    pairs = reciprocal_sensitive_pairs(cb)
    rows = np.zeros((len(pairs), 64), np.float32)
    rows[:, 0] = [p[1] for p in pairs]
    rows[:, 1] = [p[0] for p in pairs]
    check_all_ops(bq, gcb, cb, torch.from_numpy(rows.reshape(-1)), 64)
    check_all_ops(bq, gcb, cb, torch.from_numpy(rows[:, :2].reshape(-1).copy()), 2)


def test_random_shapes_types_and_offsets(bq, gcb, cb):
    """Seeded fuzz: random length, block (powers of two and not), input type, pointer offset,
    value scale; every call against the oracle."""
    rng = np.random.default_rng(2024)
    g = torch.Generator().manual_seed(2024)
    dtypes = [torch.float32, torch.float16, torch.bfloat16]
    for case in range(40):
        block = int(rng.choice([1, 3, 16, 48, 64, 100, 128, 256, 512, 1000, 1024, 2048, 4096, 5000]))
        n = int(rng.integers(1, 60_000))
        dtype = dtypes[int(rng.integers(0, 3))]
        scale = float(10.0 ** rng.uniform(-3, 3)) if dtype != torch.float16 else float(10.0 ** rng.uniform(-2, 2))
        x = (torch.randn(n, generator=g) * scale).to(dtype)
        if rng.random() < 0.3:
            x[:: max(1, n // 7)] = 0.0
        offset = int(rng.choice([0, 0, 0, 1, 2, 8]))
        lead = (int(rng.choice([0, 0, 4, 16, 32, 48])), int(rng.choice([0, 0, 1, 8, 16])), int(rng.choice([0, 0, 4, 16])))
        check_all_ops(bq, gcb, cb, x, block, offset_elems=offset, out_lead=lead)


@pytest.mark.parametrize("dtype,sig", [(torch.bfloat16, 8), (torch.float16, 11)])
def test_all_significand_pairs_of_16bit_inputs(bq, gcb, cb, dtype, sig):
    """Every (absmax significand, element significand) pair at a few exponent gaps: the
    tuned kernels' reciprocal-based quotient must land on the same code as the division."""
    half = 1 << (sig - 1)
    sigs = (half + np.arange(half)).astype(np.float64)
    gaps = (0, 1, 2, 3, 6, 10) if sig == 8 else (0, 1, 4)
    blocks = []
    for md in range(0, half, 1 if sig == 8 else 5):
        d = sigs[md]
        for gap in gaps:
            xs = sigs * 2.0 ** (-gap)
            xs = xs[xs <= d]
            xs = np.concatenate([xs, -xs])
            for i in range(0, xs.size, 63):
                chunk = xs[i:i + 63]
                blocks.append(np.concatenate([[d], chunk, np.zeros(63 - chunk.size)]))
    x = np.concatenate(blocks) * 2.0 ** (-(sig - 1) - 3)
    check_all_ops(bq, gcb, cb, torch.from_numpy(x.astype(np.float32)).to(dtype), 64)


def test_fp16_subnormals_and_extremes(bq, gcb, cb):
    bits = np.arange(65536, dtype=np.uint16)
    t = workloads.from_numpy_bits(bits, torch.float16)
    t = t[torch.isfinite(t.float())]
    t = t[: (t.numel() // 64) * 64]
    check_all_ops(bq, gcb, cb, t, 64)
    b = workloads.from_numpy_bits(bits, torch.bfloat16)
    b = b[torch.isfinite(b.float())]
    b = b[: (b.numel() // 256) * 256]
    check_all_ops(bq, gcb, cb, b, 256)                # blocks spanning 2^-133 .. 2^127: outside the reciprocal window


# ------------------------------------------------------------------------------- user codebooks

def test_user_codebook_general_path(bq, cb):
    import ctypes
    lin = np.concatenate([np.linspace(-1, 0, 128), np.linspace(0, 1, 129)[1:]]).astype(np.float32)
    ucb = bq.Codebook(kind=bq.USER, user_values=lin, device="cuda:0")
    assert not ucb.folded and np.array_equal(ucb.values, lin)
    g = torch.Generator().manual_seed(4)
    x = torch.randn(64 * 500 + 9, generator=g).to(torch.bfloat16)
    check_all_ops(bq, ucb, lin, x, 64)
    with pytest.raises(bq.BqError):
        bq.Codebook(kind=bq.USER, user_values=np.linspace(-1, 1, 256).astype(np.float32), device="cuda:0")
    mirrored = bq.Codebook(kind=bq.USER, user_values=cb.copy(), device="cuda:0")
    assert mirrored.folded
    check_all_ops(bq, mirrored, cb, x, 64)
