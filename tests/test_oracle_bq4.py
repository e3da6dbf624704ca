"""Pins of the 4-bit oracle (CPU only): the 16-entry dynamic-tree codebook against exact
rationals and its bit fields, the nearest-code step on both sides of all 15 breakpoints, the
division against pairs a reciprocal gets wrong, absmax and the inverse against torch, the packing
layout, the error bound, and planted mistakes run through the same pins."""
import os
import types
from fractions import Fraction

import numpy as np
import pytest
import torch

from helpers import frac_of, reciprocal_sensitive_pairs, rn32, round_down32
from oracle import bq4_oracle as o4

F32, F16, BF16 = 0, 1, 2
SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "bq4_oracle.py")


def exact_codebook():
    mags = []
    for k in range(3):
        for j in range(2 ** k):
            mags.append(rn32(Fraction(10) ** (k - 2) * (Fraction(1, 10) + Fraction(9, 10) * Fraction(2 * j + 1, 2 ** (k + 1)))))
    return np.sort(np.array([np.float32(0), np.float32(1)] + mags + [np.float32(-m) for m in mags], np.float32))


def nearest_exact16(xhat, cb) -> int:
    xf = frac_of(xhat)
    best, best_d = 0, None
    for j in range(16):
        d = abs(xf - frac_of(cb[j]))
        if best_d is None or d < best_d:
            best, best_d = j, d
    return best


def pin_codebook(m) -> bool:
    cb = m.make_codebook()
    ok = cb.dtype == np.float32 and cb.shape == (16,)
    ok &= np.array_equal(cb.view(np.uint32), exact_codebook().view(np.uint32))
    ok &= bool(np.all(np.diff(cb) > 0)) and cb[7] == 0.0 and cb[15] == 1.0 and cb[0] == np.float32(-0.8875)
    ok &= all(cb[j] == -cb[14 - j] for j in range(15))
    # decoded from the bit fields: magnitude bits 001 -> decade 0 (one value), 01f -> decade 1, 1ff -> decade 2
    want = sorted([0.00550, 0.0325, 0.0775, 0.2125, 0.4375, 0.6625, 0.8875])
    ok &= np.allclose(cb[8:15], want, rtol=1e-6, atol=0)
    return bool(ok)


def pin_breakpoints(m) -> bool:
    cb = exact_codebook()
    ok = True
    for j in range(15):
        t = (frac_of(cb[j]) + frac_of(cb[j + 1])) / 2
        lo = round_down32(t)
        hi = np.nextafter(lo, np.float32(np.inf))
        got = m.nearest(np.array([lo, hi], np.float32), cb)
        ok &= int(got[0]) == j and int(got[1]) == j + 1
        ok &= int(got[0]) == nearest_exact16(lo, cb) and int(got[1]) == nearest_exact16(hi, cb)
    ok &= m.nearest(cb, cb).tolist() == list(range(16))
    ok &= m.nearest(np.array([-1.0, 1.0, 0.0, -0.0, 1e-9], np.float32), cb).tolist() == [0, 15, 7, 7, 7]
    return bool(ok)


def pin_quantize(m) -> bool:
    cb = exact_codebook()
    g = torch.Generator().manual_seed(5)
    x = (torch.randn(32 * 21 + 13, generator=g) * 2.0)
    x[40] = -11.0                                                # a negative absmax element
    x[64:96] = 0                                                 # a zero block
    ok = True
    for dt, tdt in ((F32, torch.float32), (BF16, torch.bfloat16), (F16, torch.float16)):
        xt = x.to(tdt)
        bits = xt.numpy() if dt == F32 else xt.view(torch.int16).numpy().view(np.uint16)
        packed, am = m.quantize(bits, dt, 32, cb)
        f = xt.float().numpy()
        n = f.size
        pad = np.concatenate([np.abs(f), np.zeros((-n) % 32, np.float32)]).reshape(-1, 32)
        ok &= np.array_equal(am, pad.max(axis=1))                 # absmax: the textbook max |x| per block
        codes = m.unpack(packed, n)
        for i in range(0, n, 5):
            a = am[i // 32]
            xhat = rn32(frac_of(f[i]) / frac_of(a)) if a != 0 else np.float32(f[i])
            ok &= int(codes[i]) == nearest_exact16(xhat, cb)
        ok &= packed.size == (n + 1) // 2 and (packed[-1] >> 4) == 0        # odd n: the last high nibble is 0
        ok &= np.all(codes[64:96] == 7) and am[2] == 0.0
    # division: pairs whose quotient sits on a breakpoint and that a multiplication by the reciprocal moves across it
    cb8 = None
    pairs = []
    rng = np.random.default_rng(0)
    for j in range(15):
        t = (frac_of(cb[j]) + frac_of(cb[j + 1])) / 2
        lo = round_down32(t)
        a = (1.0 + rng.random(6000)).astype(np.float32)
        for target in (lo, np.nextafter(lo, np.float32(np.inf))):
            xs = (target * a).astype(np.float32)
            q_div = (xs / a).astype(np.float32)
            q_rcp = (xs * (np.float32(1.0) / a)).astype(np.float32)
            both = (lo, np.nextafter(lo, np.float32(np.inf)))
            hit = (q_div != q_rcp) & np.isin(q_div, both) & np.isin(q_rcp, both) & (np.abs(xs) <= a)
            pairs += [(np.float32(xs[i]), np.float32(a[i])) for i in np.flatnonzero(hit)[:2]]
    assert len(pairs) >= 10
    xs = np.array([v for p in pairs for v in (p[1], p[0])], np.float32)
    packed, _ = m.quantize(xs, F32, 2, cb)
    codes = m.unpack(packed, xs.size)
    for k, (xv, av) in enumerate(pairs):
        ok &= int(codes[2 * k + 1]) == nearest_exact16(rn32(frac_of(xv) / frac_of(av)), cb)
    return bool(ok)


def pin_packing(m) -> bool:
    cb = exact_codebook()
    x = np.array([1.0, -1.0, 0.0, 0.25, 1.0], np.float32)        # codes 15, 0, 7, nearest(0.25), 15; one block of 8
    packed, am = m.quantize(x, F32, 8, cb)
    c3 = nearest_exact16(np.float32(0.25), cb)
    ok = packed.tolist() == [15 | (0 << 4), 7 | (c3 << 4), 15] and am.tolist() == [1.0]
    ok &= m.unpack(packed, 5).tolist() == [15, 0, 7, c3, 15]
    return bool(ok)


def pin_dequantize(m) -> bool:
    cb = exact_codebook()
    rng = np.random.default_rng(3)
    n, block = 32 * 7 + 9, 32
    codes = rng.integers(0, 16, n + 1).astype(np.uint8)
    packed = (codes[0::2] | (codes[1::2] << 4)).astype(np.uint8)
    am = (np.abs(rng.standard_normal((n + block - 1) // block)) + 0.05).astype(np.float32)
    ok = True
    for dt, tdt in ((F32, torch.float32), (BF16, torch.bfloat16), (F16, torch.float16)):
        y = m.dequantize(packed, am, n, block, cb, dt)
        want = (torch.from_numpy(cb)[torch.from_numpy(codes[:n].astype(np.int64))] * torch.from_numpy(np.repeat(am, block)[:n])).to(tdt)
        wb = want.numpy() if dt == F32 else want.view(torch.int16).numpy().view(np.uint16)
        ok &= np.array_equal(y.view(np.uint32 if dt == F32 else np.uint16), wb.view(np.uint32 if dt == F32 else np.uint16))
    return bool(ok)


def pin_error_bound(m) -> bool:
    """|x - y| <= absmax * (half the gap between the codes bracketing xhat) (+ fp32 rounding); the largest half gap is
    0.1125 (between the two top magnitudes and between -1 and the lowest code)."""
    cb = exact_codebook()
    g = torch.Generator().manual_seed(8)
    x = (torch.randn(64 * 50, generator=g) * 3).numpy().astype(np.float32)
    packed, am = m.quantize(x, F32, 64, cb)
    y = m.dequantize(packed, am, x.size, 64, cb, F32)
    a = np.repeat(am, 64)
    err = np.abs(x.astype(np.float64) - y.astype(np.float64)) / a
    gaps = np.diff(cb.astype(np.float64)) / 2
    ok = err.max() <= max(gaps.max(), 1 - 0.8875) * (1 + 1e-6) and err.max() > 0.05
    # re-quantising the dequantised values with the same absmax present in each block returns the codes
    y2 = y.copy()
    p2, am2 = m.quantize(y2, F32, 64, cb)
    has_top = np.array([np.any(m.unpack(packed, x.size)[b * 64:(b + 1) * 64] == 15) for b in range(50)])
    codes, codes2 = m.unpack(packed, x.size).reshape(50, 64), m.unpack(p2, x.size).reshape(50, 64)
    ok &= np.array_equal(codes[has_top], codes2[has_top]) and np.array_equal(am[has_top], am2[has_top]) and has_top.sum() > 10
    return bool(ok)


def pin_scale16(m) -> bool:
    """The 16-bit scale: the smallest bf16 >= absmax (torch's bf16 grid and exact rationals say which), the codes of
    x / scale against the exact nearest value, the inverse against torch, and the bound |x| <= scale < absmax (1 + 2^-7)."""
    cb = exact_codebook()
    ok = True
    # the rounding itself, on values torch can narrow: scale is a bf16, >= a, and the bf16 just below it is < a
    rng = np.random.default_rng(11)
    vals = np.concatenate([np.abs(rng.standard_normal(400)).astype(np.float32) * np.float32(10.0) ** rng.integers(-20, 20, 400).astype(np.float32),
                           np.array([0.0, 1.0, 1.0000001, 0.99999994, 3.0, 2.0 ** -126, 2.0 ** -140, 3.3895314e38, 3.4e38], np.float32)])
    for a in vals:
        bits = m.scale16_of(a)
        s = torch.tensor([bits], dtype=torch.int32).to(torch.int16).view(torch.bfloat16).float().item()
        if a > 3.3895314e38:
            ok &= bits == 0x7F7F
            continue
        ok &= frac_of(np.float32(s)) >= frac_of(a)
        if bits > 0:
            below = torch.tensor([bits - 1], dtype=torch.int32).to(torch.int16).view(torch.bfloat16).float().item()
            ok &= frac_of(np.float32(below)) < frac_of(a)
        else:
            ok &= a == 0
        if torch.tensor([float(a)]).to(torch.bfloat16).float().item() == float(a):
            ok &= np.float32(s) == a                               # a bf16 stays itself
    g = torch.Generator().manual_seed(21)
    x = torch.randn(32 * 9 + 5, generator=g) * 3.0
    x[32:64] = 0
    x[70] = -7.3
    # a block whose absmax 1.001 is stored as 1.0078125: 0.9475 / 1.001 lies above the breakpoint 0.94375 between the two
    # top codes, 0.9475 / 1.0078125 below it
    x[96:128] *= 0.05
    x[96], x[97] = 1.001, 0.9475
    for dt, tdt in ((F32, torch.float32), (BF16, torch.bfloat16), (F16, torch.float16)):
        xt = x.to(tdt)
        bits = xt.numpy() if dt == F32 else xt.view(torch.int16).numpy().view(np.uint16)
        packed, sc = m.quantize_s16(bits, dt, 32, cb)
        f = xt.float().numpy()
        n = f.size
        ok &= sc.dtype == np.uint16 and sc.size == (n + 31) // 32 and sc[1] == 0
        sf = torch.from_numpy(sc.astype(np.int32)).to(torch.int16).view(torch.bfloat16).float().numpy()
        pad = np.concatenate([np.abs(f), np.zeros((-n) % 32, np.float32)]).reshape(-1, 32).max(axis=1)
        ok &= bool(np.all(sf >= pad)) and bool(np.all(sf.astype(np.float64) < pad.astype(np.float64) * (1 + 2.0 ** -7) + 1e-300))
        codes = m.unpack(packed, n)
        for i in range(n):
            d = sf[i // 32]
            xhat = rn32(frac_of(f[i]) / frac_of(d)) if d != 0 else np.float32(f[i])
            ok &= int(codes[i]) == nearest_exact16(xhat, cb)
        ok &= bool(np.all(codes[32:64] == 7))
        if dt != BF16:
            ok &= int(codes[97]) == 14 and int(sc[3]) == 0x3F81
        y = m.dequantize_s16(packed, sc, n, 32, cb, dt)
        want = (torch.from_numpy(cb)[torch.from_numpy(codes.astype(np.int64))] * torch.from_numpy(np.repeat(sf, 32)[:n])).to(tdt)
        wb = want.numpy() if dt == F32 else want.view(torch.int16).numpy().view(np.uint16)
        ok &= np.array_equal(y.view(np.uint32 if dt == F32 else np.uint16), wb.view(np.uint32 if dt == F32 else np.uint16))
    return bool(ok)


PINS = {"scale16": pin_scale16, "codebook": pin_codebook, "breakpoints": pin_breakpoints, "quantize": pin_quantize, "packing": pin_packing,
        "dequantize": pin_dequantize, "error_bound": pin_error_bound}


@pytest.mark.parametrize("name", sorted(PINS))
def test_pin(name):
    assert PINS[name](o4)


MUTATIONS = {
    "two_decades_only": ("for k in range(3):", "for k in range(2):", {"codebook"}),
    "bin_edges": ("9 * (2 * j + 1)", "9 * (2 * j)", {"codebook"}),
    "ties_to_larger_index": ("np.argmin(d, axis=1)", "(15 - np.argmin(d[:, ::-1], axis=1))", {"breakpoints"}),
    "absmax_forgets_abs": ("a = np.float32(np.max(np.abs(seg)))", "a = np.float32(np.max(seg))", {"quantize"}),
    "multiply_by_reciprocal": ("xhat = (seg / d).astype(np.float32)", "xhat = (seg * (np.float32(1.0) / d)).astype(np.float32)", {"quantize"}),
    "nibbles_swapped": ("packed = (codes[0::2] | (codes[1::2] << np.uint8(4)))", "packed = (codes[1::2] | (codes[0::2] << np.uint8(4)))", {"packing"}),
    "wrong_block_scale": ("scale = np.repeat(np.ascontiguousarray(absmax, np.float32), block)[:n]", "scale = np.repeat(np.ascontiguousarray(absmax, np.float32), block)[1:n + 1]", {"dequantize"}),
    "scale16_rounds_to_nearest": ("    if low:\n        top += 1", "    if low >= 0x8000:\n        top += 1", {"scale16"}),
    "scale16_divides_by_absmax": ("        s = widen(np.array([s16], np.uint16), BF16)[0]\n", "        s = np.float32(np.max(np.abs(seg)))\n", {"scale16"}),
    "unpack_high_first": ("codes[0::2] = packed & np.uint8(15)\n    codes[1::2] = packed >> np.uint8(4)", "codes[1::2] = packed & np.uint8(15)\n    codes[0::2] = packed >> np.uint8(4)", {"packing", "dequantize"}),
}


def mutated(find, repl):
    text = open(SRC).read()
    assert text.count(find) == 1, "mutation anchor not found exactly once"
    text = text.replace(find, repl).replace("from .mmd_oracle import", "from oracle.mmd_oracle import")
    mod = types.ModuleType("bq4_oracle_mutant")
    exec(compile(text, "bq4_oracle_mutant", "exec"), mod.__dict__)
    return mod


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name):
    find, repl, must_fail = MUTATIONS[name]
    m = mutated(find, repl)
    failed = set()
    for pin, fn in PINS.items():
        try:
            with np.errstate(all="ignore"):
                if not fn(m):
                    failed.add(pin)
        except Exception:
            failed.add(pin)
    assert must_fail <= failed, f"{name}: pins {must_fail - failed} did not notice"
