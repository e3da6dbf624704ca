"""CPU checks of the CUDA library's host-side logic: the search tables it builds and the
arithmetic its tuned kernels apply to them, restated in tests/host_check.cpp."""
import ctypes
import os
import subprocess

import numpy as np
import pytest

import oracle
from helpers import bits_f32, f32_bits, midpoints, round_down32

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "host_check.cpp")
LIB = os.path.join(HERE, "libhost_check.so")
TABLES_H = os.path.join(os.path.dirname(HERE), "paper_2407_19775_b200", "csrc", "bq_tables.h")


@pytest.fixture(scope="module")
def hc():
    newest = max(os.path.getmtime(SRC), os.path.getmtime(TABLES_H))
    if not os.path.exists(LIB) or os.path.getmtime(LIB) < newest:
        tmp = LIB + f".tmp{os.getpid()}"
        subprocess.run(["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-mfma", "-fPIC", "-shared", "-o", tmp, SRC], check=True)
        os.replace(tmp, LIB)
    L = ctypes.CDLL(LIB)
    L.hc_check_quick_division.restype = ctypes.c_long
    L.hc_check_rowquant_division.restype = ctypes.c_long
    L.hc_code_folded.argtypes = [ctypes.c_float]
    L.hc_code_general.argtypes = [ctypes.c_float]
    L.hc_value_folded.argtypes = [ctypes.c_float, ctypes.c_float]
    L.hc_value_folded.restype = ctypes.c_float
    return L


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _tables(hc):
    vals = np.zeros(256, np.float32); thr = np.zeros(256, np.float32); tk = np.zeros(128, np.uint32)
    cm = np.zeros(132, np.float32); gs = np.zeros(1409, np.uint32); nl = ctypes.c_float()
    folded = hc.hc_tables(_p(vals), _p(thr), _p(tk), _p(cm), _p(gs), ctypes.byref(nl))
    return folded, vals, thr, tk, cm, gs, nl.value


def test_library_codebook_equals_oracle(hc, cb):
    folded, vals, thr, tk, cm, gs, nl = _tables(hc)
    assert folded == 1
    assert np.array_equal(vals.view(np.uint32), cb.view(np.uint32))
    down = np.array([round_down32(t) for t in midpoints(cb)], np.float32)
    assert np.array_equal(thr[:255].view(np.uint32), down.view(np.uint32)) and np.isinf(thr[255])
    assert np.array_equal(cm[:129].view(np.uint32), cb[127:].view(np.uint32))
    assert gs.size == 1409


def _codes(hc, bits: np.ndarray):
    out_f = np.empty(bits.size, np.uint8)
    out_g = np.empty(bits.size, np.uint8)
    for i, b in enumerate(bits):
        x = bits_f32(int(b))
        out_f[i] = hc.hc_code_folded(x)
        out_g[i] = hc.hc_code_general(x)
    return out_f, out_g


def test_searches_agree_with_oracle_around_every_breakpoint(hc, cb):
    pats = []
    for t in midpoints(cb):
        b = f32_bits(round_down32(t))
        for d in range(-3, 4):
            pats.append((b + d) & 0xFFFFFFFF if b + d >= 0 else 0)
    pats += [0, 0x80000000, 1, 0x80000001, 0x3F800000, 0xBF800000, 0x3F7FFFFF, 0xBF7FFFFF]
    pats += [f32_bits(c) for c in cb]
    pats = np.array(pats, np.uint64).astype(np.uint32)
    f, g = _codes(hc, pats)
    want = np.array([oracle.nearest(bits_f32(int(b)), cb) for b in pats], np.uint8)
    assert np.array_equal(g, want)
    assert np.array_equal(f, want)


def test_searches_agree_on_random_and_cell_edges(hc, cb):
    rng = np.random.default_rng(0)
    mags = rng.integers(0, 0x3F800001, 400_000, dtype=np.uint64).astype(np.uint32)
    signs = rng.integers(0, 2, mags.size, dtype=np.uint64).astype(np.uint32) << 31
    lo = np.uint32(0)
    out_f = np.empty(1 << 20, np.uint8); out_g = np.empty(1 << 20, np.uint8)
    bad = 0
    # dense sweeps: the smallest decades, near 2^-22 (where keys are clamped), and the top of the range
    for start in (0x33000000, 0x34700000, 0x3F700000, 0xB3000000, 0xB4700000, 0xBF700000):
        hc.hc_codes_of_bits(ctypes.c_uint32(start), ctypes.c_uint32(1 << 20), _p(out_f), _p(out_g))
        bad += int((out_f != out_g).sum())
    assert bad == 0
    pats = mags | signs
    f, g = _codes(hc, pats[:20000])
    assert np.array_equal(f, g)
    want = np.array([oracle.nearest(bits_f32(int(b)), cb) for b in pats[:3000]], np.uint8)
    assert np.array_equal(g[:3000], want)


def test_folded_value_matches_oracle_dequantize(hc, cb):
    rng = np.random.default_rng(2)
    xs = np.concatenate([rng.uniform(-1, 1, 2000), [0.0, -0.0, -1.0, 1.0, -1e-9, 1e-9, -0.9965, -0.997]]).astype(np.float32)
    for a in (np.float32(3.5), np.float32(1e-30), np.float32(0.0)):
        for x in xs:
            q = oracle.nearest(x, cb)
            if a == 0 and q != 127:
                continue          # the fused path meets absmax 0 only with xhat = +-0, i.e. code 127
            want = oracle.dequantize(np.array([q], np.uint8), np.array([a], np.float32), 1, cb, oracle.F32)[0]
            got = np.float32(hc.hc_value_folded(float(x), float(a)))
            assert f32_bits(got) == f32_bits(want), (float(x), float(a))


@pytest.mark.parametrize("sig_bits,d_exp", [(8, 0), (8, -64), (8, 64), (11, 0), (11, -64), (11, 64)])
def test_reciprocal_quotient_is_the_ieee_quotient_for_16bit_inputs(hc, sig_bits, d_exp):
    """bf16 has 8 significant bits, fp16 (subnormals included, once widened) at most 11.  Every
    pair of significands, both signs, every exponent gap down to xhat ~ 2^-34, and every reciprocal within 2 ulp of
    the correctly rounded one."""
    cm, ck = ctypes.c_long(), ctypes.c_long()
    bad = hc.hc_check_quick_division(sig_bits, 34, d_exp, ctypes.byref(cm), ctypes.byref(ck))
    assert ck.value > 4_000_000 and bad == 0 and cm.value == 0


@pytest.mark.parametrize("sig_bits,d_exp", [(8, 0), (11, 0), (11, -64), (11, 64)])
def test_reciprocal_route_of_the_row_kernel_is_the_ieee_quotient(hc, sig_bits, d_exp):
    """RN32(127 x / d) from an approximate reciprocal, for every pair of 16-bit significands, both signs, exponent gaps
    down to 127 x / d ~ 2^-19 (everything below rounds to the integer 0 on either route) and every reciprocal within 2 ulp
    of the correctly rounded one."""
    im, ck = ctypes.c_long(), ctypes.c_long()
    bad = hc.hc_check_rowquant_division(sig_bits, 26, d_exp, ctypes.byref(im), ctypes.byref(ck))
    assert ck.value > 3_000_000 and bad == 0 and im.value == 0


def test_user_codebook_rules(hc, cb):
    assert hc.hc_user_tables_folded(_p(cb.copy())) == 1
    lin = np.linspace(-1, 1, 256).astype(np.float32)
    assert hc.hc_user_tables_folded(_p(lin)) == -1, "no exact zero"
    lin = np.concatenate([np.linspace(-1, 0, 128), np.linspace(0, 1, 129)[1:]]).astype(np.float32)
    assert hc.hc_user_tables_folded(_p(lin)) == 0, "valid but not mirrored around index 127"
    bad = cb.copy(); bad[10] = bad[11]
    assert hc.hc_user_tables_folded(_p(bad)) == -1
    bad = cb.copy(); bad[200] = np.nan
    assert hc.hc_user_tables_folded(_p(bad)) == -1
