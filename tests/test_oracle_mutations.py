"""Do the pins bite?  Each case below plants one plausible mistake in a COPY of the oracle's
source (on the CPU, in a temporary directory), builds it, and checks that the pins which are
meant to catch that kind of mistake fail on it, while the unmodified oracle passes them all.
The pins here are the same exact-arithmetic / library checks as in test_oracle_*.py, in a
form that takes the library to check as an argument."""
import ctypes
import os
import subprocess
from fractions import Fraction

import numpy as np
import pytest
import torch

from helpers import exact_codebook, frac_of, midpoints, nearest_exact, reciprocal_sensitive_pairs, rn32, round_down32

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "bq_oracle.cpp")
F32, F16, BF16 = 0, 1, 2

MUTATIONS = {
    # name: (text to find exactly once, replacement, pins that must fail)
    "ties_to_larger_index": ("if (dist < best_dist)", "if (dist <= best_dist)", {"breakpoints"}),
    "bin_edges_instead_of_midpoints": ("double(bins2 + 9 * (2 * j + 1))", "double(bins2 + 9 * (2 * j))", {"codebook"}),
    "decade_count_off_by_one": ("for (int k = 0; k <= 6; ++k) {", "for (int k = 1; k <= 6; ++k) {", {"codebook"}),
    "absmax_forgets_abs": ("const float v = std::fabs(load_elem(x, xdt, i));", "const float v = load_elem(x, xdt, i);", {"absmax"}),
    "multiply_by_reciprocal": ("const float xhat = load_elem(x, xdt, i) / d;", "const float xhat = load_elem(x, xdt, i) * (1.0f / d);", {"division"}),
    "zero_block_divides_by_absmax": ("const float d = (a != 0.0f) ? a : 1.0f;", "const float d = a;", {"zero_block"}),
    "bf16_truncates": ("if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) upper += 1;", "(void)lower;", {"narrow"}),
    "bf16_ties_away": ("(lower == 0x8000u && (upper & 1u))", "(lower == 0x8000u)", {"narrow"}),
    "dequantize_uses_wrong_block": ("codebook[codes[i]] * absmax[i / B]", "codebook[codes[i]] * absmax[(i + 1) / B]", {"dequantize"}),
    "scan_skips_last_code": ("for (int j = 1; j < 256; ++j) {", "for (int j = 1; j < 255; ++j) {", {"breakpoints"}),
}


def _build(tmp_path, name, find=None, repl=None):
    text = open(SRC).read()
    if find is not None:
        assert text.count(find) == 1, f"mutation anchor for {name} not found exactly once"
        text = text.replace(find, repl)
    d = tmp_path / name
    d.mkdir()
    (d / "bq_oracle.cpp").write_text(text)
    (d / "bq_oracle.h").write_text(open(os.path.join(ROOT, "oracle", "bq_oracle.h")).read())
    so = str(d / "lib.so")
    subprocess.run(["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-o", so, str(d / "bq_oracle.cpp")], check=True)
    L = ctypes.CDLL(so)
    L.bq_oracle_nearest.argtypes = [ctypes.c_float, ctypes.c_void_p]
    L.bq_oracle_narrow.argtypes = [ctypes.c_float, ctypes.c_int]
    L.bq_oracle_narrow.restype = ctypes.c_uint16
    return L


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def failing_pins(L) -> set:
    """Runs the pins against library L and returns the names of those that fail."""
    failed = set()
    cb = np.empty(256, np.float32)
    L.bq_oracle_make_codebook(_p(cb))
    ref_cb = exact_codebook()
    if not np.array_equal(cb.view(np.uint32), ref_cb.view(np.uint32)):
        failed.add("codebook")
    cb = ref_cb          # the remaining pins use the true codebook so that they are independent of the first

    # both sides of every breakpoint, ties to the smaller index, the end values
    ok = True
    for j, t in enumerate(midpoints(cb)):
        lo = round_down32(t)
        hi = np.nextafter(lo, np.float32(np.inf))
        ok &= L.bq_oracle_nearest(ctypes.c_float(float(lo)), _p(cb)) == j
        ok &= L.bq_oracle_nearest(ctypes.c_float(float(hi)), _p(cb)) == j + 1
    ok &= L.bq_oracle_nearest(ctypes.c_float(1.0), _p(cb)) == 255
    if not ok:
        failed.add("breakpoints")

    def quant(x, dt, block):
        n = x.size
        codes = np.empty(n, np.uint8)
        am = np.empty((n + block - 1) // block, np.float32)
        assert L.bq_oracle_quantize(_p(x), dt, ctypes.c_size_t(n), block, _p(cb), _p(codes), _p(am)) == 0
        return codes, am

    g = torch.Generator().manual_seed(3)
    x = (torch.randn(64 * 40, generator=g) * 2.5).numpy().astype(np.float32)
    x[5] = -9.0                                           # the absmax element of block 0 is negative
    codes, am = quant(x, F32, 64)
    ref_am = np.abs(x).reshape(-1, 64).max(axis=1)
    if not np.array_equal(am, ref_am):
        failed.add("absmax")
    # correctly rounded quotient + exact nearest code, element by element
    ok = True
    for i in range(0, x.size, 7):
        xhat = rn32(frac_of(x[i]) / frac_of(ref_am[i // 64]))
        ok &= int(codes[i]) == nearest_exact(xhat, cb)
    pairs = reciprocal_sensitive_pairs(cb, per_threshold=1)
    xs = np.array([v for pair in pairs for v in (pair[1], pair[0])], np.float32)
    pc, _ = quant(xs, F32, 2)
    for k, (xv, av) in enumerate(pairs):
        ok &= int(pc[2 * k + 1]) == nearest_exact(rn32(frac_of(xv) / frac_of(av)), cb)
    if not ok and "absmax" not in failed:
        failed.add("division")

    z = np.zeros(64, np.float32)
    zc, za = quant(z, F32, 64)
    if not (np.all(zc == 127) and za[0] == 0.0):
        failed.add("zero_block")

    # narrowing against torch on halfway and random patterns
    rng = np.random.default_rng(0)
    pats = np.concatenate([((np.arange(0x3F00, 0x4000, dtype=np.uint32) << 16) | 0x8000),
                           rng.integers(0x30000000, 0x4F000000, 4000, dtype=np.uint64).astype(np.uint32)])
    f = pats.view(np.float32)
    ref = torch.from_numpy(f.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([L.bq_oracle_narrow(ctypes.c_float(float(v)), BF16) for v in f], np.uint16)
    if not np.array_equal(got, ref):
        failed.add("narrow")

    # dequantize against torch
    n, block = 64 * 9 + 5, 64
    q = rng.integers(0, 256, n).astype(np.uint8)
    a = np.abs(rng.standard_normal((n + block - 1) // block)).astype(np.float32) + 0.1
    y = np.empty(n, np.float32)
    assert L.bq_oracle_dequantize(_p(q), _p(a), ctypes.c_size_t(n), block, _p(cb), _p(y), F32) == 0
    want = cb[q] * np.repeat(a, block)[:n]
    if not np.array_equal(y.view(np.uint32), want.astype(np.float32).view(np.uint32)):
        failed.add("dequantize")
    return failed


def test_unmodified_oracle_passes_every_pin(tmp_path):
    assert failing_pins(_build(tmp_path, "clean")) == set()


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(tmp_path, name):
    find, repl, must_fail = MUTATIONS[name]
    failed = failing_pins(_build(tmp_path, name, find, repl))
    assert must_fail <= failed, f"{name}: pins {must_fail - failed} did not notice"
