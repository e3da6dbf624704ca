"""GPU parity of the 4-bit variant against its CPU oracle, through the C ABI: packed codes,
absmax and dequantised output are compared bit for bit (integer and byte work; the floating
point that decides a code is the same correctly rounded fp32 quotient on both sides)."""
from fractions import Fraction

import numpy as np
import pytest
import torch

from helpers import frac_of, round_down32
from oracle import bq4_oracle as o4
from paper_2407_19775_b200 import workloads

pytestmark = pytest.mark.gpu
F32, F16, BF16 = 0, 1, 2
DT = {torch.float32: F32, torch.float16: F16, torch.bfloat16: BF16}


def bits(t: torch.Tensor) -> np.ndarray:
    return workloads.as_numpy_bits(t.cpu())


def check(bq, x: torch.Tensor, block: int, ydt=None):
    """x: a CPU tensor (any shape).  Quantize and dequantize on the GPU, compare with the oracle."""
    cb = bq.Codebook4()
    cb_ref = o4.make_codebook()
    flat = x.reshape(-1)
    dt = DT[flat.dtype]
    p_ref, a_ref = o4.quantize(bits(flat), dt, block, cb_ref)
    xd = flat.cuda()
    p, a = bq.bq4_quantize(xd, block, cb)
    torch.cuda.synchronize()
    assert np.array_equal(p.cpu().numpy(), p_ref)
    assert np.array_equal(a.cpu().numpy().view(np.uint32), a_ref.view(np.uint32))
    for out in ([flat.dtype, torch.float32] if ydt is None else [ydt]):
        y = bq.bq4_dequantize(p, a, flat.numel(), block, cb, out)
        y_ref = o4.dequantize(p_ref, a_ref, flat.numel(), block, cb_ref, DT[out])
        got = bits(y)
        assert np.array_equal(got.view(np.uint32 if out == torch.float32 else np.uint16), y_ref.view(np.uint32 if out == torch.float32 else np.uint16))
    return p_ref, a_ref


@pytest.mark.parametrize("name,rows,block", [("tiny", None, 64), ("prefill7b", 96, 256), ("decode70b", 64, 64), ("moe_prefill", 40, 2048),
                                             ("sweep1g", 24, 128), ("sweep1g", 24, 8), ("sweep1g", 16, 65536), ("prefill7b", 40, 16)])
def test_workloads(bq, name, rows, block):
    x = workloads.make(name, rows=rows)
    check(bq, x, block)


@pytest.mark.parametrize("tdt", [torch.float32, torch.bfloat16, torch.float16])
def test_ragged_and_general_cases(bq, tdt):
    g = torch.Generator().manual_seed(7)
    x = (torch.randn(5000, generator=g) * 1.5).to(tdt)
    x[100:164] = 0
    for n, block in [(4999, 64), (5000, 24), (37, 64), (1, 8), (2, 1), (777, 3), (4097, 4096), (513, 512), (1023, 32), (5000, 131072)]:
        check(bq, x[:n].clone(), block)


def test_unaligned_pointers(bq):
    cb = bq.Codebook4()
    cb_ref = o4.make_codebook()
    g = torch.Generator().manual_seed(9)
    base = (torch.randn(4096 + 8, generator=g)).to(torch.bfloat16)
    xd = base.cuda()[3:3 + 4096]                                 # 6 bytes off a 16-byte boundary
    p_ref, a_ref = o4.quantize(bits(base[3:3 + 4096]), BF16, 64, cb_ref)
    pbuf = torch.empty(2048 + 4, dtype=torch.uint8, device="cuda")
    p, a = bq.bq4_quantize(xd, 64, cb, packed_out=pbuf[1:2049])
    assert np.array_equal(p.cpu().numpy(), p_ref) and np.array_equal(a.cpu().numpy(), a_ref)
    ybuf = torch.empty(4096 + 8, dtype=torch.bfloat16, device="cuda")
    y = bq.bq4_dequantize(p, a, 4096, 64, cb, torch.bfloat16, y_out=ybuf[5:5 + 4096])
    assert np.array_equal(bits(y), o4.dequantize(p_ref, a_ref, 4096, 64, cb_ref, BF16))


def test_breakpoints_and_division(bq):
    """Values on both sides of every breakpoint, with absmax 1 (block of 2: the absmax element and the value), and pairs
    whose quotient a multiplication by the reciprocal would move across a breakpoint."""
    cb_ref = o4.make_codebook()
    xs = []
    for j in range(15):
        lo = round_down32((frac_of(cb_ref[j]) + frac_of(cb_ref[j + 1])) / 2)
        xs += [1.0, float(lo), 1.0, float(np.nextafter(lo, np.float32(np.inf)))]
    check(bq, torch.tensor(xs, dtype=torch.float32), 2)
    rng = np.random.default_rng(0)
    vals = []
    for j in range(15):
        lo = round_down32((frac_of(cb_ref[j]) + frac_of(cb_ref[j + 1])) / 2)
        a = (1.0 + rng.random(6000)).astype(np.float32)
        for target in (lo, np.nextafter(lo, np.float32(np.inf))):
            x = (target * a).astype(np.float32)
            differ = ((x / a).astype(np.float32) != (x * (np.float32(1) / a)).astype(np.float32)) & (np.abs(x) <= a)
            for i in np.flatnonzero(differ)[:3]:
                vals += [float(a[i]), float(x[i])]
    assert len(vals) > 40
    check(bq, torch.tensor(vals, dtype=torch.float32), 2)
    # 16-bit absmax significands through the reciprocal route: every bf16 significand as the divisor
    sig = torch.arange(128, 256, dtype=torch.float32) / 128.0
    rows = torch.cat([sig[:, None], sig[:, None] * torch.linspace(-1, 1, 63)[None, :]], dim=1).to(torch.bfloat16)
    check(bq, rows, 64)


def test_vectorised_search_on_and_around_every_breakpoint(bq):
    """The vectorised kernels find the code with one table lookup on the bits of xhat.  Blocks of 8 whose first element is
    1.0 (so xhat = x) carry, for every breakpoint and both signs, the 2049 floats around it; plus a dense sweep of [-1, 1]
    and the values next to zero and to the table's lower end."""
    cb_ref = o4.make_codebook()
    vals = []
    for j in range(15):
        lo = round_down32((frac_of(cb_ref[j]) + frac_of(cb_ref[j + 1])) / 2)
        u = np.float32(lo).view(np.uint32).astype(np.int64)
        vals.append((u + np.arange(-1024, 1025)).astype(np.uint32).view(np.float32))
    vals.append(np.linspace(-1, 1, 200001).astype(np.float32))
    vals.append((np.float32(2.0 ** -9).view(np.uint32).astype(np.int64) + np.arange(-64, 65)).astype(np.uint32).view(np.float32))
    vals.append(np.array([0.0, -0.0, 1e-45, -1e-45, 1e-30, -1e-30, 1.0, -1.0, 0.99999994, -0.99999994], np.float32))
    v = np.concatenate(vals)
    v = np.concatenate([v, -v])
    v = v[np.abs(v) <= 1]
    v = v[: (v.size // 7) * 7].reshape(-1, 7)
    x = np.concatenate([np.ones((v.shape[0], 1), np.float32), v], axis=1)       # [1.0, seven values] per block of 8
    check(bq, torch.from_numpy(x), 8, ydt=torch.float32)
    x16 = np.concatenate([np.ones((v.shape[0], 1), np.float32), v], axis=1).reshape(-1)
    x16 = x16[: (x16.size // 1024) * 1024]                                      # the same through the one-warp-per-block kernel
    x16.reshape(-1, 1024)[:, 0] = 1.0
    check(bq, torch.from_numpy(x16), 1024, ydt=torch.float32)


def test_scales_outside_the_reciprocal_window(bq):
    g = torch.Generator().manual_seed(11)
    x = torch.randn(8, 256, generator=g)
    x[0] *= 1e-30; x[1] *= 1e30; x[2] *= 2.0 ** -64; x[3] *= 2.0 ** 64; x[4] *= 2.0 ** -65; x[5] = 0
    check(bq, x.to(torch.bfloat16), 256)
    check(bq, x.to(torch.bfloat16), 1024)
    check(bq, x, 64)


def test_user_codebook(bq):
    lin = np.linspace(-1, 1, 16).astype(np.float32)              # a uniform map (no exact zero: allowed for user maps)
    cb = bq.Codebook4(bq.USER, lin)
    g = torch.Generator().manual_seed(13)
    x = torch.randn(4096, generator=g).to(torch.float16)
    p_ref, a_ref = o4.quantize(bits(x), F16, 128, lin)
    p, a = bq.bq4_quantize(x.cuda(), 128, cb)
    assert np.array_equal(p.cpu().numpy(), p_ref) and np.array_equal(a.cpu().numpy(), a_ref)
    y = bq.bq4_dequantize(p, a, 4096, 128, cb, torch.float16)
    assert np.array_equal(bits(y), o4.dequantize(p_ref, a_ref, 4096, 128, lin, F16))
    with pytest.raises(bq.BqError):
        bq.Codebook4(bq.USER, lin[::-1].copy())


def test_kv_cache_shaped_tensor(bq):
    """The other large activation-like tensor of the paper's system is the KV cache (2 x head_dim x heads x layers values
    per token): the same calls with one block per head vector."""
    g = torch.Generator().manual_seed(17)
    kv = (torch.randn(2, 4, 8, 96, 128, generator=g) * 0.7).to(torch.bfloat16)      # [k/v, layers, heads, tokens, head_dim]
    kv[:, :, 3, :, 17] *= 12                                                        # a heavy channel in one head
    check(bq, kv, 128)
    cb8 = bq.Codebook()
    import oracle
    ref_c, ref_a = oracle.quantize(bits(kv.reshape(-1)), BF16, 128, oracle.make_codebook())
    c, a = bq.bq_quantize(kv.cuda().reshape(-1), 128, cb8)
    assert np.array_equal(c.cpu().numpy(), ref_c) and np.array_equal(a.cpu().numpy(), ref_a)


def test_full_size_tensor_sampled_blocks(bq):
    """The benchmark's 1 GiB tensor at full size through the vectorised kernels (blocks 64 and 1024, as bench.py times them):
    absmax of every block against a device-side max, the error bound on every element, and sampled whole blocks (first, last,
    random) bit for bit against the oracle."""
    cb = bq.Codebook4()
    cb_ref = o4.make_codebook()
    x_cpu = workloads.make("sweep1g").view(-1)
    n = x_cpu.numel()
    xd = x_cpu.cuda()
    xb = bits(x_cpu)
    rng = np.random.default_rng(321)
    for block in (64, 1024):
        nb = n // block
        p, a = bq.bq4_quantize(xd, block, cb)
        y = bq.bq4_dequantize(p, a, n, block, cb, torch.bfloat16)
        torch.cuda.synchronize()
        assert torch.equal(a.view(torch.int32), xd.view(nb, block).abs().amax(dim=1).float().view(torch.int32))
        step = 1 << 26
        for s0 in range(0, n, step):
            e0 = min(n, s0 + step)
            a_el = a[s0 // block:(e0 + block - 1) // block].repeat_interleave(block)[: e0 - s0]
            err = (xd[s0:e0].float() - y[s0:e0].float()).abs()
            bound = a_el * (0.1125 + 2.0 ** -20) + y[s0:e0].float().abs() * 2.0 ** -8          # half the widest gap + bf16 rounding of y
            assert bool((err <= bound).all().item())
        pick = np.unique(np.concatenate([[0, 1, nb - 2, nb - 1], rng.integers(0, nb, max(8, 65536 // block))]))
        for b in pick:
            seg = np.ascontiguousarray(xb[b * block:(b + 1) * block])
            p_ref, a_ref = o4.quantize(seg, BF16, block, cb_ref)
            assert np.array_equal(p[b * block // 2:(b + 1) * block // 2].cpu().numpy(), p_ref)
            assert a[b].item() == a_ref[0]
            assert np.array_equal(bits(y[b * block:(b + 1) * block]), o4.dequantize(p_ref, a_ref, block, block, cb_ref, BF16))
        del p, a, y


def check_s16(bq, x: torch.Tensor, block: int):
    """The 16-bit-scale pair against its oracle: packed codes, scale words and both outputs bit for bit."""
    cb = bq.Codebook4()
    cb_ref = o4.make_codebook()
    flat = x.reshape(-1)
    dt = DT[flat.dtype]
    p_ref, s_ref = o4.quantize_s16(bits(flat), dt, block, cb_ref)
    p, s = bq.bq4_quantize_s16(flat.cuda(), block, cb)
    torch.cuda.synchronize()
    assert s.dtype == torch.bfloat16
    assert np.array_equal(p.cpu().numpy(), p_ref)
    assert np.array_equal(bits(s), s_ref)
    for out in (flat.dtype, torch.float32):
        y = bq.bq4_dequantize_s16(p, s, flat.numel(), block, cb, out)
        y_ref = o4.dequantize_s16(p_ref, s_ref, flat.numel(), block, cb_ref, DT[out])
        view = np.uint32 if out == torch.float32 else np.uint16
        assert np.array_equal(bits(y).view(view), y_ref.view(view))
    return p_ref, s_ref


@pytest.mark.parametrize("name,rows,block", [("tiny", None, 64), ("prefill7b", 64, 256), ("decode70b", 64, 64), ("moe_prefill", 24, 2048),
                                             ("sweep1g", 16, 8), ("sweep1g", 16, 65536)])
def test_scale16_workloads(bq, name, rows, block):
    check_s16(bq, workloads.make(name, rows=rows), block)


@pytest.mark.parametrize("tdt", [torch.float32, torch.bfloat16, torch.float16])
def test_scale16_ragged_general_and_extreme_scales(bq, tdt):
    """Ragged tails and odd blocks (the general kernels), zero blocks, and blocks whose absmax sits on, just above and
    just below a bf16, in the subnormal range and near the top of the type's range."""
    g = torch.Generator().manual_seed(17)
    x = (torch.randn(6000, generator=g) * 1.5).to(tdt)
    x[100:164] = 0
    for n, block in [(5999, 64), (6000, 24), (37, 64), (1, 8), (777, 3), (4097, 4096), (1023, 32)]:
        check_s16(bq, x[:n].clone(), block)
    top = {torch.float32: 3.0e38, torch.bfloat16: 3.0e38, torch.float16: 60000.0}[tdt]
    tiny = {torch.float32: 1e-41, torch.bfloat16: 1e-39, torch.float16: 6e-8}[tdt]
    peaks = [1.0, 1.0000001, 0.99999994, 1.0078125, 1.00390625, 255.0, 256.5, top, tiny, 3 * tiny, 2.0 ** -126, 1.5 * 2.0 ** -126]
    blocks = []
    for k, pk in enumerate(peaks):
        b = torch.rand(64, generator=g) * 2 - 1
        b[k % 64] = 1.0 if k % 2 else -1.0
        blocks.append((b.double() * pk).to(tdt))
    check_s16(bq, torch.cat(blocks), 64)
    check_s16(bq, torch.cat(blocks)[:64 * len(peaks) - 8], 16)


def test_scale16_is_close_to_the_fp32_scale(bq):
    """Property at a size the oracle does not reach: every stored scale is a bf16 in [absmax, absmax (1 + 2^-7)) and the
    reconstruction error stays within the 4-bit bound against that scale."""
    cb = bq.Codebook4()
    x = workloads.make("sweep1g", rows=4096).reshape(-1).cuda()
    block = 64
    p, s = bq.bq4_quantize_s16(x, block, cb)
    _, a = bq.bq4_quantize(x, block, cb)
    sf = s.float()
    assert bool((sf >= a).all()) and bool((sf.double() < a.double() * (1 + 2.0 ** -7) + 1e-300).all())
    y = bq.bq4_dequantize_s16(p, s, x.numel(), block, cb, torch.float32)
    err = (x.float() - y).abs().view(-1, block) / sf.clamp_min(1e-30)[:, None]
    assert float(err.max()) <= 0.1125 * (1 + 1e-5)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("block", [64, 128, 256, 512, 1024, 2048, 4096])
def test_large_tensors_through_the_tiled_forward_kernel(bq, dtype, block):
    """Above 8 Mi elements the whole tiles go through the persistent forward kernel of the 8-bit path in its 4-bit flavour, the
    whole blocks left over through the 4-bit kernels, and a short last block through the general ones; packed bytes, absmax and
    the dequantised tensor must be the oracle's."""
    g = torch.Generator().manual_seed(block + 1)
    n = (1 << 23) + 5 * 24576 + 3 * block + 37                    # whole tiles, then whole blocks, then a short block
    x = (torch.randn(n, generator=g) * (1.0 + 30.0 * (torch.rand(n, generator=g) < 0.002))).to(dtype)
    x[block:2 * block] = 0
    x[7 * block] = -x[7 * block:8 * block].float().abs().max() * 2  # the absmax element is negative: xhat = -1 has no code of its own
    x[9 * block + 1] = -0.0
    check(bq, x, block, ydt=dtype)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("block", [64, 256, 512, 4096])
def test_large_tensors_with_the_bf16_scale_through_the_tiled_forward_kernel(bq, dtype, block):
    """The same split (tiles, left-over blocks, a short block) with the block scale stored as a bf16: absmax values on, just
    above and far from the bf16 grid, a zero block, and the top of the fp16 range."""
    g = torch.Generator().manual_seed(block + 5)
    n = (1 << 23) + 3 * 24576 + 2 * block + 11
    x = (torch.randn(n, generator=g) * (1.0 + 30.0 * (torch.rand(n, generator=g) < 0.002))).to(dtype)
    x[block:2 * block] = 0
    x[2 * block:3 * block] = x[2 * block:3 * block].clamp(-1, 1)
    x[2 * block] = 1.0                                              # an absmax that is itself a bf16
    x[3 * block:4 * block] = x[3 * block:4 * block].clamp(-1, 1)
    x[3 * block + 1] = 1.00390625 if dtype == torch.bfloat16 else 1.0009765625      # just above one: rounds up
    if dtype == torch.float16:
        x[5 * block] = 65504.0
    check_s16(bq, x, block)
