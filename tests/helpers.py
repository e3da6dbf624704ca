"""Exact-arithmetic helpers shared by the CPU tests.  They re-derive what the method fixes
(codebook values, midpoints, nearest code) with Python integers and Fractions, so that the
oracle is checked against something other than its own floating-point code."""
from __future__ import annotations

import struct
from fractions import Fraction

import numpy as np


def f32_bits(v) -> int:
    return struct.unpack("<I", struct.pack("<f", float(v)))[0]


def bits_f32(u: int) -> np.float32:
    return np.float32(struct.unpack("<f", struct.pack("<I", u & 0xFFFFFFFF))[0])


def frac_of(v) -> Fraction:
    """Exact value of a float as a rational."""
    return Fraction(float(v))


def rn32(fr: Fraction) -> np.float32:
    """Correctly rounded (nearest, ties to even) float32 of a rational, by exact comparison."""
    if fr == 0:
        return np.float32(0.0)
    guess = np.float32(float(fr))          # within 1 ulp; refine among the neighbours exactly
    cands = {guess, np.nextafter(guess, np.float32(-np.inf)), np.nextafter(guess, np.float32(np.inf))}
    best = None
    for c in cands:
        d = abs(frac_of(c) - fr)
        key = (d, f32_bits(c) & 1)          # ties: even mantissa wins
        if best is None or key < best[0]:
            best = (key, c)
    return best[1]


def tree_magnitudes():
    """The 127 positive magnitudes of the dynamic-tree map as exact rationals, keyed (k, j)."""
    out = {}
    for k in range(7):
        for j in range(2 ** k):
            out[(k, j)] = Fraction(10) ** (k - 6) * (Fraction(1, 10) + Fraction(9, 10) * Fraction(2 * j + 1, 2 ** (k + 1)))
    return out


def exact_codebook() -> np.ndarray:
    mags = [rn32(m) for m in tree_magnitudes().values()]
    vals = [np.float32(0.0), np.float32(1.0)] + mags + [np.float32(-m) for m in mags]
    return np.sort(np.array(vals, dtype=np.float32))


def midpoints(cb: np.ndarray):
    """Exact midpoints t_j between neighbouring codes, j = 0..254."""
    return [(frac_of(cb[j]) + frac_of(cb[j + 1])) / 2 for j in range(255)]


def nearest_exact(xhat, cb: np.ndarray) -> int:
    """Nearest code in exact rational arithmetic; equal distances go to the smaller index."""
    xf = frac_of(xhat)
    best, best_d = 0, None
    for j in range(256):
        d = abs(xf - frac_of(cb[j]))
        if best_d is None or d < best_d:
            best, best_d = j, d
    return best


def round_down32(fr: Fraction) -> np.float32:
    """Largest float32 that is <= fr."""
    g = np.float32(float(fr))
    while frac_of(g) > fr:
        g = np.nextafter(g, np.float32(-np.inf))
    while frac_of(np.nextafter(g, np.float32(np.inf))) <= fr:
        g = np.nextafter(g, np.float32(np.inf))
    return g


def codes_by_thresholds(xhat: np.ndarray, cb: np.ndarray) -> np.ndarray:
    """Vectorised nearest code through the exact midpoints: #{ j : t_j < xhat }.  The
    midpoints are exact in float64 for this codebook (checked by the caller's test)."""
    t = (cb[:-1].astype(np.float64) + cb[1:].astype(np.float64)) / 2.0
    return np.searchsorted(t, xhat.astype(np.float64), side="left").astype(np.uint8)


def reciprocal_sensitive_pairs(cb: np.ndarray, per_threshold: int = 3, seed: int = 0):
    """(x, a) pairs, |x| <= a, whose correctly rounded quotient x / a sits exactly on a
    round-down midpoint (so the code is j) while the product x * RN(1/a) lands one float
    higher (code j + 1), or the other way round.  A normalisation that multiplies by a
    rounded reciprocal gets these wrong; a true division gets them right."""
    rng = np.random.default_rng(seed)
    out = []
    for t in midpoints(cb):
        lo = round_down32(t)
        if abs(float(lo)) < 1e-6:
            continue
        a = (1.0 + rng.random(4000)).astype(np.float32) * np.float32(2.0) ** rng.integers(-3, 4, 4000).astype(np.float32)
        for target in (lo, np.nextafter(lo, np.float32(np.inf))):
            x = (target * a).astype(np.float32)
            q_div = (x / a).astype(np.float32)
            q_rcp = (x * (np.float32(1.0) / a)).astype(np.float32)
            lo_hi = (lo, np.nextafter(lo, np.float32(np.inf)))
            hit = (q_div != q_rcp) & np.isin(q_div, lo_hi) & np.isin(q_rcp, lo_hi) & (np.abs(x) <= a)
            for i in np.flatnonzero(hit)[:per_threshold]:
                out.append((np.float32(x[i]), np.float32(a[i])))
    return out
