"""Pins for the oracle's dynamic-tree codebook (CPU only).

What fixes the codebook (the reading taken of the paper's "dynamic blockwise
quantization", section "Compression techniques" item 1, which does not define the map): an 8-bit map over [-1, 1] made of a
sign bit, a variable-length exponent field and a linear fraction.  The checks below rebuild
it three independent ways (exact rationals, the bit-field decoding, structural invariants)."""
import hashlib
import os
from fractions import Fraction

import numpy as np

import oracle
from helpers import bits_f32, exact_codebook, f32_bits, frac_of, midpoints, rn32, round_down32, tree_magnitudes

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_hex(name):
    vals, sha = [], None
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("sha256"):
                sha = line.split()[1]
            else:
                vals.append(bits_f32(int(line, 16)))
    return np.array(vals, np.float32), sha


def test_invariants(cb):
    assert cb.dtype == np.float32 and cb.shape == (256,)
    assert np.all(np.diff(cb.astype(np.float64)) > 0), "strictly ascending, hence unique"
    assert cb[127] == 0.0 and f32_bits(cb[127]) == 0, "+0.0 sits at index 127"
    assert cb[255] == 1.0 and cb.min() >= -1.0 and cb.max() <= 1.0
    assert np.count_nonzero(cb == 0.0) == 1
    # mirror: every magnitude appears with both signs; only +1 has no partner
    assert np.array_equal(cb[:255], -cb[254::-1][:255])
    # the signed magnitudes cancel, leaving 0 + 1
    assert float(cb.astype(np.float64).sum()) == 1.0


def test_equals_exact_rational_construction(cb):
    assert np.array_equal(cb.view(np.uint32), exact_codebook().view(np.uint32))


def test_bit_field_decoding(cb):
    """Decode every byte as sign | exponent field | fraction and compare the value set."""
    vals = []
    for byte in range(256):
        sign = byte >> 7
        rest = byte & 0x7F
        if rest == 0:
            vals.append(Fraction(1) if sign else Fraction(0))     # the two end values
            continue
        k = rest.bit_length() - 1           # bits left after the first set bit = fraction width
        frac = rest - (1 << k)              # linear fraction, k bits
        mag = Fraction(10) ** (k - 6) * (Fraction(1, 10) + Fraction(9, 10) * Fraction(2 * frac + 1, 2 ** (k + 1)))
        vals.append(-mag if sign else mag)
    decoded = np.sort(np.array([rn32(v) for v in vals], np.float32))
    assert np.array_equal(decoded.view(np.uint32), cb.view(np.uint32))


def test_decade_structure(cb):
    pos = cb[128:255].astype(np.float64)            # 127 magnitudes below 1
    start = 0
    for k in range(7):
        cnt = 2 ** k
        dec = pos[start:start + cnt]
        start += cnt
        scale = 10.0 ** (k - 6)
        assert np.all(dec > 0.1 * scale) and np.all(dec < 1.0 * scale), k
        width = 0.9 * scale / cnt                   # bin width; codes are the bin midpoints
        expect = 0.1 * scale + width * (np.arange(cnt) + 0.5)
        assert np.allclose(dec, expect, rtol=1e-6, atol=0), k
    assert start == 127
    gaps = np.diff(cb.astype(np.float64))
    assert abs(gaps.min() - 5.5e-7) < 1e-12 and abs(gaps.max() - 0.0140625) < 1e-7
    assert gaps.argmin() in (126, 127) and gaps.argmax() < 64


def test_magnitude_count_and_keys():
    mags = tree_magnitudes()
    assert len(mags) == 127 and len(set(mags.values())) == 127


def test_golden_codebook(cb):
    gold, sha = _read_hex("codebook_dynamic_tree.txt")
    assert np.array_equal(gold.view(np.uint32), cb.view(np.uint32))
    assert hashlib.sha256(cb.astype("<f4").tobytes()).hexdigest() == sha
    spot = {0: 0xBF7E3333, 1: 0xBF7A999A, 2: 0xBF770000, 63: 0xBDDB3333, 64: 0xBDC9EB85, 126: 0xB513A3B6,
            127: 0x00000000, 128: 0x3513A3B6, 129: 0x365A1A93, 130: 0x370205FF, 191: 0x3DDB3333,
            192: 0x3DF80000, 254: 0x3F7E3333, 255: 0x3F800000}
    for i, u in spot.items():
        assert f32_bits(cb[i]) == u, i


def test_golden_thresholds(cb):
    gold, sha = _read_hex("thresholds_round_down.txt")
    t = midpoints(cb)
    down = np.array([round_down32(x) for x in t], np.float32)
    assert np.array_equal(gold.view(np.uint32), down.view(np.uint32))
    assert hashlib.sha256(down.astype("<f4").tobytes()).hexdigest() == sha
    # midpoints are exact in double: sum of two fp32 codes needs fewer than 53 bits
    t64 = (cb[:-1].astype(np.float64) + cb[1:].astype(np.float64)) / 2.0
    assert all(frac_of(t64[j]) == t[j] for j in range(255))
    representable = sum(1 for j in range(255) if frac_of(down[j]) == t[j])
    assert representable == 110
