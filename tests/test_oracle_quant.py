"""Pins for the oracle's quantize / dequantize / roundtrip (CPU only): exact-rational brute
force, both sides of every breakpoint, closed-form special cases, library cross-checks,
the error bound and the re-quantisation invariants."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from helpers import bits_f32, codes_by_thresholds, f32_bits, frac_of, midpoints, nearest_exact, round_down32
from paper_2407_19775_b200 import workloads

F32, F16, BF16 = oracle.F32, oracle.F16, oracle.BF16
TORCH_DT = {F32: torch.float32, F16: torch.float16, BF16: torch.bfloat16}


def _bits(x: torch.Tensor) -> np.ndarray:
    return workloads.as_numpy_bits(x)


# ----------------------------------------------------------------------------- nearest code

def test_nearest_brute_force_exact(cb):
    rng = np.random.default_rng(7)
    xs = list(rng.uniform(-1, 1, 300).astype(np.float32))
    xs += list((rng.uniform(-1, 1, 200) * 10.0 ** rng.integers(-7, 0, 200)).astype(np.float32))
    xs += [np.float32(v) for v in (0.0, -0.0, 1.0, -1.0, 1e-45, -1e-45, 2.75e-7, -2.75e-7, 5.5e-7, 0.9965, -0.9965)]
    for x in xs:
        assert oracle.nearest(x, cb) == nearest_exact(x, cb), float(x)


def test_every_code_maps_to_itself(cb):
    for j in range(256):
        assert oracle.nearest(cb[j], cb) == j


def test_both_sides_of_every_breakpoint(cb):
    """A monotone step function that is right on both sides of all 255 steps is right
    everywhere.  At the round-down midpoint the code is j (ties included), one ulp above it
    is j + 1."""
    t = midpoints(cb)
    for j in range(255):
        lo = round_down32(t[j])
        hi = np.nextafter(lo, np.float32(np.inf))
        assert oracle.nearest(lo, cb) == j, j
        assert oracle.nearest(hi, cb) == j + 1, j
        if frac_of(lo) == t[j]:      # a true tie: equidistant from c_j and c_j+1 -> smaller index
            assert abs(frac_of(lo) - frac_of(cb[j])) == abs(frac_of(lo) - frac_of(cb[j + 1]))


def test_end_values(cb):
    assert oracle.nearest(1.0, cb) == 255
    assert oracle.nearest(-1.0, cb) == 0          # no -1 in the map: nearest is -0.99296875
    assert oracle.nearest(0.0, cb) == 127 and oracle.nearest(-0.0, cb) == 127
    assert oracle.nearest(2.7e-7, cb) == 127 and oracle.nearest(2.8e-7, cb) == 128
    assert oracle.nearest(-2.7e-7, cb) == 127 and oracle.nearest(-2.8e-7, cb) == 126


# ----------------------------------------------------------------------------- quantize

@pytest.mark.parametrize("dt,block", [(F32, 64), (BF16, 256), (F16, 64), (BF16, 7), (F32, 1)])
def test_quantize_against_library_steps(cb, dt, block):
    """absmax = textbook max|x| per block (torch), xhat = numpy fp32 division, code = count
    of exact midpoints below xhat: three library routines re-assembled."""
    g = torch.Generator().manual_seed(11)
    n = 5 * 1024 + 37                                 # ragged tail
    x = (torch.randn(n, generator=g) * 3.0).to(TORCH_DT[dt])
    codes, absmax = oracle.quantize(_bits(x), dt, block, cb)
    xf = x.float()
    nb = (n + block - 1) // block
    pad = torch.zeros(nb * block)
    pad[:n] = xf
    ref_absmax = pad.view(nb, block).abs().amax(dim=1).numpy()
    assert np.array_equal(absmax.view(np.uint32), ref_absmax.view(np.uint32))
    d = np.where(ref_absmax == 0, np.float32(1), ref_absmax).astype(np.float32)
    xhat = (xf.numpy() / np.repeat(d, block)[:n]).astype(np.float32)
    assert np.array_equal(codes, codes_by_thresholds(xhat, cb))


def test_quantize_tiny_exact_rational(cb):
    """Everything in exact arithmetic on a tiny input: absmax, the correctly rounded
    quotient and the nearest code."""
    from helpers import rn32
    x = np.array([0.3, -1.7, 0.0, 2.5, -2.5, 1e-3, 7e-8, -0.62], np.float32)
    codes, absmax = oracle.quantize(x, F32, 4, cb)
    for b in range(2):
        blk = x[4 * b:4 * b + 4]
        a = max(abs(frac_of(v)) for v in blk)
        assert frac_of(absmax[b]) == a
        for i, v in enumerate(blk):
            xhat = rn32(frac_of(v) / a)
            assert codes[4 * b + i] == nearest_exact(xhat, cb)


def test_normalisation_is_a_true_division(cb):
    """Pairs built so that x / a rounds onto a midpoint's round-down value while x * RN(1/a)
    rounds to its neighbour (or the reverse): the code differs between the two."""
    from helpers import reciprocal_sensitive_pairs, rn32
    pairs = reciprocal_sensitive_pairs(cb)
    assert len(pairs) > 200
    x = np.array([v for pair in pairs for v in (pair[1], pair[0])], np.float32)      # blocks of 2: [a, x]
    codes, absmax = oracle.quantize(x, F32, 2, cb)
    for k, (xv, av) in enumerate(pairs):
        assert absmax[k] == av
        assert codes[2 * k + 1] == nearest_exact(rn32(frac_of(xv) / frac_of(av)), cb), (float(xv), float(av))


def test_zero_block_negative_zero_and_flush(cb):
    x = np.zeros(64, np.float32)
    x[5] = -0.0
    codes, absmax = oracle.quantize(x, F32, 64, cb)
    assert np.all(codes == 127) and f32_bits(absmax[0]) == 0
    y = oracle.dequantize(codes, absmax, 64, cb, F32)
    assert np.all(y.view(np.uint32) == 0), "+0.0 everywhere, the sign of zero is not kept"
    # values below half the smallest code flush to code 127; -0.0 too
    x = np.array([1.0, 2.7e-7, -2.7e-7, -0.0, 2.8e-7, -2.8e-7], np.float32)
    codes, absmax = oracle.quantize(x, F32, 8, cb)
    assert list(codes) == [255, 127, 127, 127, 128, 126]


def test_absmax_sign_and_partial_block(cb):
    x = np.array([0.5, -2.0, 1.0, 2.0, 0.25], np.float32)     # blocks of 2: last one has 1 element
    codes, absmax = oracle.quantize(x, F32, 2, cb)
    assert list(absmax) == [2.0, 2.0, 0.25]
    assert codes[1] == 0, "xhat = -1 -> code 0"
    assert codes[3] == 255 and codes[4] == 255
    y = oracle.dequantize(codes, absmax, 2, cb, F32)
    assert y[1] == np.float32(-0.99296875) * np.float32(2.0) and y[3] == 2.0 and y[4] == 0.25


def test_tiny_workload_special_blocks(cb):
    x = workloads.make("tiny")
    codes, absmax = oracle.quantize(_bits(x), F32, 64, cb)
    assert absmax[0] == 0.0 and np.all(codes[:64] == 127)
    assert absmax[1] == 50.0 and codes[64] == 0
    assert absmax[2] == 50.0 and codes[128] == 255


# ----------------------------------------------------------------------------- dequantize

@pytest.mark.parametrize("dt", [F32, F16, BF16])
def test_dequantize_against_torch(cb, dt):
    rng = np.random.default_rng(3)
    n, block = 4096 + 19, 64
    codes = rng.integers(0, 256, n).astype(np.uint8)
    nb = (n + block - 1) // block
    absmax = (np.abs(rng.standard_normal(nb)) * 10.0 ** rng.integers(-6, 3, nb)).astype(np.float32)
    absmax[3] = 0.0
    y = oracle.dequantize(codes, absmax, block, cb, dt)
    v = torch.from_numpy(cb)[torch.from_numpy(codes).long()] * torch.from_numpy(np.repeat(absmax, block)[:n])
    ref = v.to(TORCH_DT[dt])
    assert np.array_equal(y.view(np.uint16 if dt != F32 else np.uint32), _bits(ref).view(np.uint16 if dt != F32 else np.uint32))


# ----------------------------------------------------------------------------- invariants

@pytest.mark.parametrize("name,block", [("tiny", 64), ("decode70b", 64), ("prefill7b", 256)])
def test_error_bound(cb, name, block):
    """|x - v| <= absmax * (half the gap between the codes bracketing xhat) + absmax * 2^-22."""
    w = workloads.WORKLOADS[name]
    x = workloads.make(name, rows=64 if name != "tiny" else None)
    dt = {torch.float32: F32, torch.float16: F16, torch.bfloat16: BF16}[w.dtype]
    y, codes, absmax = oracle.roundtrip(_bits(x), dt, block, cb, F32, side=True)
    xf = x.float().view(-1).numpy().astype(np.float64)
    a = np.repeat(absmax.astype(np.float64), block)[:xf.size]
    d = np.where(a == 0, 1.0, a)
    xhat = xf / d
    c64 = cb.astype(np.float64)
    hi = np.clip(np.searchsorted(c64, xhat, side="left"), 1, 255)
    half_gap = (c64[hi] - c64[hi - 1]) / 2.0
    half_gap = np.where(xhat < c64[0], c64[0] - xhat + 1e-12, half_gap)       # xhat in [-1, c_0): nearest is c_0
    err = np.abs(xf - y.astype(np.float64))
    assert np.all(err <= a * half_gap + a * 2.0 ** -22)
    assert np.max(err / d) <= 0.00703125 + 2.0 ** -22


def test_requantize_is_identity_when_block_holds_code_255(cb):
    rng = np.random.default_rng(5)
    block, nb = 64, 200
    codes = rng.integers(0, 256, nb * block).astype(np.uint8)
    codes[::block] = 255                                        # absmax element is +absmax
    absmax = (2.0 ** rng.uniform(-100, 100, nb)).astype(np.float32)
    v = oracle.dequantize(codes, absmax, block, cb, F32)
    codes2, absmax2 = oracle.quantize(v, F32, block, cb)
    assert np.array_equal(absmax2.view(np.uint32), absmax.view(np.uint32))
    assert np.array_equal(codes2, codes)


def test_roundtrip_equals_composition_and_is_idempotent(cb):
    x = workloads.make("decode70b", rows=16)
    xb = _bits(x)
    y, codes, absmax = oracle.roundtrip(xb, F16, 64, cb, F16, side=True)
    c2, a2 = oracle.quantize(xb, F16, 64, cb)
    y2 = oracle.dequantize(c2, a2, 64, cb, F16)
    assert np.array_equal(codes, c2) and np.array_equal(absmax.view(np.uint32), a2.view(np.uint32))
    assert np.array_equal(y, y2)
    # idempotence on blocks whose absmax element is positive (it then maps to exactly +absmax);
    # fp32 output, so that no second rounding sits between the two passes
    xf = x.float().view(-1, 64)
    pos = (xf.gather(1, xf.abs().argmax(dim=1, keepdim=True)) > 0).view(-1).numpy()
    y32 = oracle.roundtrip(xb, F16, 64, cb, F32)
    y32b = oracle.roundtrip(y32, F32, 64, cb, F32)
    same = (y32.view(np.uint32).reshape(-1, 64) == y32b.view(np.uint32).reshape(-1, 64)).all(axis=1)
    assert pos.sum() > 10 and np.all(same[pos])


def test_compression_ratio_halves_sixteen_bit():
    for block, want in [(64, 1.882), (256, 1.969), (1024, 1.992), (2048, 1.996), (4096, 1.998)]:
        n = block * 10
        stored = n + 4 * (n // block)
        assert round(2 * n / stored, 3) == want


def test_sharded_equals_single(cb):
    x = workloads.make("prefill7b", rows=8)
    xb = _bits(x)
    y, c, a = oracle.roundtrip(xb, BF16, 256, cb, BF16, side=True)
    ys, cs, as_ = oracle.roundtrip_sharded(xb, BF16, 256, cb, BF16, threads=3)
    assert np.array_equal(y, ys) and np.array_equal(c, cs) and np.array_equal(a.view(np.uint32), as_.view(np.uint32))


def test_bad_arguments(cb):
    with pytest.raises(ValueError):
        oracle.quantize(np.zeros(4, np.float32), F32, 0, cb)
    with pytest.raises(ValueError):
        oracle.quantize(np.zeros(4, np.float32), 7, 4, cb)
    c, a = oracle.quantize(np.zeros(0, np.float32), F32, 4, cb)
    assert c.size == 0 and a.size == 0
