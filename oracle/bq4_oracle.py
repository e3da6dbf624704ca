"""CPU oracle of the 4-bit variant of dynamic blockwise quantization (test infrastructure only).

The paper (section "Compression techniques", item 1) compresses the exchanged hidden states by
dynamic blockwise quantization and fixes no bit width beyond the halving it reports for 8 bits.
This is the same method with a 16-entry codebook, two codes per byte (a quarter of a 16-bit
payload), one of the natural variants of the path.  Readings, all stated:

  codebook   the dynamic-tree construction with 4 bits: a sign bit, and in the other 3 bits the
             position of the first set bit picks decade k = 0..2 (scale 10^(k-2)) and leaves k bits
             of linear fraction: m(k, j) = 10^(k-2) (0.1 + 0.9 (2j + 1) / 2^(k+1)), j < 2^k;
             7 magnitudes with both signs, plus 0 and 1; ascending; the code is the index
             (0.0 is code 7, +1.0 is code 15).  Each magnitude is one ratio of exact integers
             divided in double and rounded once to fp32.
  per block  absmax in fp32; xhat = x / absmax as one IEEE fp32 division (divisor 1 for a zero
             block); code = nearest value, distances in double, ties to the smaller index.
  packing    element 2i in the low nibble of byte i, element 2i + 1 in the high nibble; the unused
             high nibble of a last odd element is 0.
  inverse    y = narrow(RN32(value[code] * absmax)).

  16-bit scale (the *_s16 pair) the block's scale is its absmax rounded toward +infinity to a bf16
             (never above the largest finite bf16), stored as the bf16's 16 bits; x is divided by
             that scale and the inverse multiplies by it; everything else as above.

Nothing here is imported by the CUDA library or its binding; it shares no code with it.
fp16 / bf16 arrays are ``uint16`` bit patterns, fp32 arrays are ``float32``.
Pins: tests/test_oracle_bq4.py (exact rationals, both sides of all 15 breakpoints, torch
cross-checks, packing layout, error bound, planted mistakes).  Parity with any outside
library's 4-bit map: parity unpinned.
"""
from __future__ import annotations

import numpy as np

from .mmd_oracle import narrow, widen

F32, F16, BF16 = 0, 1, 2


def make_codebook() -> np.ndarray:
    vals = [0.0, 1.0]
    for k in range(3):
        bins2 = 2 ** (k + 1)
        pow10 = 10 ** (3 - k)
        for j in range(2 ** k):
            m = np.float32(np.float64(bins2 + 9 * (2 * j + 1)) / np.float64(bins2 * pow10))
            vals += [m, -m]
    return np.sort(np.array(vals, dtype=np.float32))


def _as_f32(x: np.ndarray, dt: int) -> np.ndarray:
    x = np.ascontiguousarray(x).reshape(-1)
    return x.astype(np.float32) if dt == F32 else widen(x, dt)


def nearest(xhat: np.ndarray, cb: np.ndarray) -> np.ndarray:
    """Index of the nearest codebook value; np.argmin keeps the first (smallest) index on ties."""
    d = np.abs(xhat.astype(np.float64)[:, None] - cb.astype(np.float64)[None, :])
    return np.argmin(d, axis=1).astype(np.uint8)


def quantize(x: np.ndarray, dt: int, block: int, cb: np.ndarray):
    """-> (packed uint8 [ceil(n / 2)], absmax float32 [ceil(n / block)])."""
    v = _as_f32(x, dt)
    n = v.size
    nb = (n + block - 1) // block
    absmax = np.zeros(nb, np.float32)
    codes = np.zeros(n + (n & 1), np.uint8)
    for b in range(nb):
        seg = v[b * block:min(n, (b + 1) * block)]
        a = np.float32(np.max(np.abs(seg)))
        absmax[b] = a
        d = a if a != 0 else np.float32(1.0)
        xhat = (seg / d).astype(np.float32)                      # one fp32 division per element
        codes[b * block:b * block + seg.size] = nearest(xhat, cb)
    packed = (codes[0::2] | (codes[1::2] << np.uint8(4))).astype(np.uint8)
    return packed, absmax


def unpack(packed: np.ndarray, n: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, np.uint8)
    codes = np.empty(packed.size * 2, np.uint8)
    codes[0::2] = packed & np.uint8(15)
    codes[1::2] = packed >> np.uint8(4)
    return codes[:n]


def dequantize(packed: np.ndarray, absmax: np.ndarray, n: int, block: int, cb: np.ndarray, ydt: int) -> np.ndarray:
    codes = unpack(packed, n)
    scale = np.repeat(np.ascontiguousarray(absmax, np.float32), block)[:n]
    v = (cb[codes] * scale).astype(np.float32)                   # one fp32 multiply per element
    return narrow(v, ydt)


BF16_MAX_BITS = 0x7F7F                                           # the largest finite bf16


def scale16_of(absmax: float) -> int:
    """The 16 bits of the smallest bf16 that is >= absmax (absmax >= 0, finite), capped at the largest finite bf16."""
    bits = int(np.float32(absmax).view(np.uint32))
    top, low = bits >> 16, bits & 0xFFFF
    if low:
        top += 1                                                 # the next bf16 up: magnitudes order like their bit patterns
    return min(top, BF16_MAX_BITS)


def quantize_s16(x: np.ndarray, dt: int, block: int, cb: np.ndarray):
    """-> (packed uint8 [ceil(n / 2)], scale uint16 [ceil(n / block)])."""
    v = _as_f32(x, dt)
    n = v.size
    nb = (n + block - 1) // block
    scale = np.zeros(nb, np.uint16)
    codes = np.zeros(n + (n & 1), np.uint8)
    for b in range(nb):
        seg = v[b * block:min(n, (b + 1) * block)]
        s16 = scale16_of(np.max(np.abs(seg)))
        scale[b] = s16
        s = widen(np.array([s16], np.uint16), BF16)[0]
        d = s if s != 0 else np.float32(1.0)
        xhat = np.divide(seg, d, dtype=np.float32)               # one fp32 division per element, by the stored scale
        codes[b * block:b * block + seg.size] = nearest(xhat, cb)
    low, high = codes[0::2], codes[1::2]                          # element 2i in the low nibble of byte i
    return (low + np.uint8(16) * high).astype(np.uint8), scale


def dequantize_s16(packed: np.ndarray, scale: np.ndarray, n: int, block: int, cb: np.ndarray, ydt: int) -> np.ndarray:
    return dequantize(packed, widen(np.ascontiguousarray(scale, np.uint16), BF16), n, block, cb, ydt)
