"""Pins of the mixed-matrix-decomposition oracle (CPU only).

The paper (section "Compression techniques", item 2) fixes only the idea: 8-bit weights plus a
small 16-bit part.  The arithmetic of the reading is pinned here by things other than the
oracle's own code: exact rational arithmetic for the rounding chain, plain integer loops for
the product, closed forms where the quantization is exact, the decomposition's error bound,
torch's CPU conversions, and planted mistakes that the pins must notice.
"""
import os
import types
from fractions import Fraction

import numpy as np
import pytest
import torch

from helpers import frac_of, rn32
from oracle import mmd_oracle as mo
from paper_2407_19775_b200 import workloads

F32, F16, BF16 = 0, 1, 2
SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "mmd_oracle.py")


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy().view(np.uint16).reshape(t.shape)


def exact_q(v: float, d: float) -> int:
    """rint(RN32(127 v / d)) with the division and both roundings done on rationals."""
    t = frac_of(rn32(Fraction(127) * frac_of(v) / frac_of(d)))
    fl = t.numerator // t.denominator
    r = t - fl
    if r > Fraction(1, 2) or (r == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return int(fl)


def small_case(dt, seed=0, R=6, K=48, ko=(5, 17)):
    g = torch.Generator().manual_seed(seed)
    tdt = torch.bfloat16 if dt == BF16 else torch.float16
    v = (torch.randn(R, K, generator=g) * 1.7).to(tdt)
    v[:, list(ko)] *= 30.0
    return v, np.array(ko, np.int32)


# ------------------------------------------------------------------------------------------
# the pins, in a form that takes the module to check (so that planted mistakes can be run
# through the same code)

def pin_convert(m) -> bool:
    pats = np.arange(65536, dtype=np.uint16)
    ok = True
    for dt, tdt in ((BF16, torch.bfloat16), (F16, torch.float16)):
        ref = torch.from_numpy(pats.view(np.int16).copy()).view(tdt).float().numpy()
        got = m.widen(pats, dt)
        fin = np.isfinite(ref)
        ok &= np.array_equal(got[fin].view(np.uint32), ref[fin].view(np.uint32))
        rng = np.random.default_rng(1)
        u = rng.integers(0x33000000, 0x47000000, 200000, dtype=np.uint64).astype(np.uint32)
        u = np.concatenate([u, (np.arange(0x3F00, 0x4100, dtype=np.uint32) << 16) | 0x8000,      # bf16 halfway cases
                            (np.arange(0x3F800, 0x3FA00, dtype=np.uint32) << 12) | 0x1000])        # fp16 halfway cases
        u = np.concatenate([u, u | 0x80000000])
        f = u.view(np.float32)
        want = torch.from_numpy(f.copy()).to(tdt).view(torch.int16).numpy().view(np.uint16)
        ok &= np.array_equal(m.narrow(f, dt), want)
    return bool(ok)


def pin_rowquant_exact(m) -> bool:
    ok = True
    for dt in (BF16, F16):
        v, idx = small_case(dt, seed=3 + dt)
        v[1, :] = 0.0                                             # a zero row
        v[2, 7] = -v[2].abs().max() * 2                           # the absmax element is negative
        v[3, 0] = 0.75; v[3, 1] = 1.5 * 0.75 / 127                # 127 v/d = 1.5 exactly: tie, to even (2)
        v[3, 2] = 2.5 * 0.75 / 127                                # 2.5 -> 2
        q, s, side = m.rowquant(bits_of(v), dt, idx)
        f = v.float().numpy()
        regular = np.ones(f.shape[1], bool)
        regular[idx] = False
        for r in range(f.shape[0]):
            a = np.abs(f[r, regular]).max()
            d = a if a != 0 else np.float32(1.0)
            ok &= s[r] == rn32(frac_of(a) / 127)
            for k in range(f.shape[1]):
                ok &= int(q[r, k]) == (0 if not regular[k] else exact_q(f[r, k], d))
        ok &= np.array_equal(side[:, :len(idx)], bits_of(v)[:, idx]) and not side[:, len(idx):].any()
        ok &= side.shape[1] == 64
    return bool(ok)


def reciprocal_sensitive_pairs(limit=24):
    """bf16 pairs (v, d), 0 < v <= d, for which multiplying 127 v by the rounded reciprocal of d
    lands on another integer than the division does (found with plain float32 arithmetic; the
    expected value of each is then taken from exact_q)."""
    vals = (np.arange(0x3C00, 0x4300, dtype=np.uint32) << 16).view(np.float32)
    out = []
    for d in vals[::7]:
        scaled = vals * np.float32(127)
        differ = (np.rint(scaled / d) != np.rint(scaled * (np.float32(1) / d))) & (vals <= d)
        out += [(float(v), float(d)) for v in vals[differ][:2]]
    return out[:limit]


def pin_rowquant_division(m) -> bool:
    pairs = reciprocal_sensitive_pairs()
    assert len(pairs) >= 16
    v = torch.zeros(len(pairs), 16)
    for r, (x, d) in enumerate(pairs):
        v[r, 0], v[r, 1], v[r, 2] = d, x, -x
    v = v.to(torch.bfloat16)
    q, _, _ = m.rowquant(bits_of(v), BF16, np.zeros(0, np.int32))
    ok = True
    for r, (x, d) in enumerate(pairs):
        ok &= int(q[r, 0]) == 127 and int(q[r, 1]) == exact_q(x, d) and int(q[r, 2]) == exact_q(-x, d)
    # exact ties: with d = 127/64 the quotient 127 v / d is 64 v, so v = (n + 1/2)/64 sits on a tie
    ties = [0.5, 1.5, 2.5, -4.5, -5.5, 100.5, -126.5]
    for dt, tdt in ((BF16, torch.bfloat16), (F16, torch.float16)):
        t = torch.tensor([[127.0 / 64] + [h / 64 for h in ties] + [0.0] * 8]).to(tdt)
        assert np.array_equal(t.double().numpy()[0, 1:8] * 64, np.array(ties))
        q, _, _ = m.rowquant(bits_of(t), dt, np.zeros(0, np.int32))
        ok &= q[0, :8].tolist() == [127, 0, 2, 2, -4, -6, 100, -126]
    return bool(ok)


def pin_rowquant_properties(m) -> bool:
    ok = True
    v, idx = small_case(BF16, seed=9, R=40, K=256, ko=(3, 100, 255))
    q, s, _ = m.rowquant(bits_of(v), BF16, idx)
    f = v.float().numpy()
    regular = np.ones(256, bool)
    regular[idx] = False
    ok &= np.abs(q.astype(int)).max() <= 127 and not q[:, idx].any()
    arg = np.abs(f[:, regular]).argmax(axis=1)
    ok &= np.all(np.abs(q[:, regular][np.arange(40), arg].astype(int)) == 127)     # the absmax element maps to +-127
    qn, sn, _ = m.rowquant(bits_of(-v), BF16, idx)
    ok &= np.array_equal(qn, -q) and np.array_equal(sn, s)                      # odd symmetry
    # |w - q s| <= s/2 (1 + 2^-14) off the critical features (s/2 from the rounding to an integer; the fp32
    # roundings of 127 w / d and of a / 127 each move q s by at most 127 s 2^-24), exact on them
    _, _, side = m.rowquant(bits_of(v), BF16, idx)
    rec = m.reconstruct(q, s, side, BF16, idx)
    err = np.abs(rec - f.astype(np.float64))
    ok &= np.all(err[:, regular] <= s.astype(np.float64)[:, None] * 0.5 * (1 + 2.0 ** -14))
    ok &= not err[:, idx].any()
    # features outside the rows' range must not move the scale
    v2 = v.clone()
    v2[:, idx] *= 1000.0
    q2, s2, _ = m.rowquant(bits_of(v2), BF16, idx)
    ok &= np.array_equal(q2, q) and np.array_equal(s2, s)
    return bool(ok)


def pin_int_product(m) -> bool:
    rng = np.random.default_rng(5)
    a = rng.integers(-127, 128, (5, 23)).astype(np.int8)
    b = rng.integers(-127, 128, (7, 23)).astype(np.int8)
    want = [[sum(int(a[i, k]) * int(b[j, k]) for k in range(23)) for j in range(7)] for i in range(5)]
    ok = np.array_equal(m.int_product(a, b), np.array(want))
    a = np.full((2, 40000), 127, np.int8)
    b = np.stack([np.full(40000, 127, np.int8), np.full(40000, -127, np.int8)])
    ok &= np.array_equal(m.int_product(a, b), np.array([[40000 * 16129, -40000 * 16129]] * 2))    # above 2^24 and 2^29
    a = rng.integers(-127, 128, (33, 700)).astype(np.int8)
    b = rng.integers(-127, 128, (21, 700)).astype(np.int8)
    ok &= np.array_equal(m.int_product(a, b), a.astype(np.int64) @ b.astype(np.int64).T)
    return bool(ok)


def pin_linear_closed_form(m) -> bool:
    """Integer-valued rows whose regular part has absmax 127 (times a power of two) quantize
    without error, so the layer must return the exact product X W^T."""
    rng = np.random.default_rng(7)
    M, N, K = 9, 11, 96
    idx = np.array([4, 50], np.int32)
    ok = True
    for dt, tdt in ((BF16, torch.bfloat16), (F16, torch.float16)):
        xi = rng.integers(-127, 128, (M, K)); xi[:, 0] = 127
        wi = rng.integers(-127, 128, (N, K)); wi[:, 1] = -127
        xi[:, idx] = rng.integers(-4, 5, (M, 2)) * 64                  # outlier features: large, still exact in 16 bits
        wi[:, idx] = rng.integers(-8, 9, (N, 2))
        X = torch.from_numpy(xi * 2.0 ** -3).to(tdt)
        W = torch.from_numpy(wi * 2.0 ** -9).to(tdt)
        assert np.array_equal(X.double().numpy(), xi * 2.0 ** -3) and np.array_equal(W.double().numpy(), wi * 2.0 ** -9)
        qw, sw, wo = m.rowquant(bits_of(W), dt, idx)
        y = m.linear(bits_of(X), dt, qw, sw, wo, idx, F32)
        exact = X.double().numpy() @ W.double().numpy().T
        ok &= np.array_equal(y, exact.astype(np.float32)) and np.array_equal(exact.astype(np.float32).astype(np.float64), exact)
        # the transposed product is a different matrix: a swapped operand cannot pass
        ok &= y.shape == (M, N)
        # without critical features the side part vanishes and the padded width is zero
        none = np.zeros(0, np.int32)
        qw0, sw0, wo0 = m.rowquant(bits_of(W), dt, none)
        ok &= wo0.shape == (N, 0)
        y16 = m.linear(bits_of(X), dt, qw, sw, wo, idx, dt)
        ok &= np.array_equal(y16, m.narrow(exact.astype(np.float32), dt))
    return bool(ok)


def pin_linear_error_bound(m) -> bool:
    """|Y - X W^T| is bounded by the two quantization errors: with e_x <= sx/2, e_w <= sw/2 per
    regular element, |sum_k (x w - xq wq)| <= sum_k (|x| sw/2 + |w| sx/2 + sx sw/4)."""
    X, W, idx = workloads.make_linear("mmd_tiny")
    dt = BF16
    qw, sw, wo = m.rowquant(bits_of(W), dt, idx)
    y = m.linear(bits_of(X), dt, qw, sw, wo, idx, F32).astype(np.float64)
    xf, wf = X.double().numpy(), W.double().numpy()
    exact = xf @ wf.T
    _, sx, _ = m.rowquant(bits_of(X), dt, idx)
    regular = np.ones(xf.shape[1], bool)
    regular[idx] = False
    ax = np.abs(xf[:, regular]).sum(axis=1)
    aw = np.abs(wf[:, regular]).sum(axis=1)
    kr = regular.sum()
    sxd, swd = sx.astype(np.float64), sw.astype(np.float64)
    bound = (ax[:, None] * swd[None, :] + aw[None, :] * sxd[:, None]) / 2 + kr * sxd[:, None] * swd[None, :] / 4
    bound = bound * (1 + 2.0 ** -18) + np.abs(exact) * 2.0 ** -22
    err = np.abs(y - exact)
    ok = np.all(err <= bound)
    ok &= err.max() > 0                                           # it is a lossy method
    # the critical features are carried exactly: zeroing the regular part leaves X_O W_O^T
    Xo = X.clone(); Xo[:, regular] = 0
    y2 = m.linear(bits_of(Xo), dt, qw, sw, wo, idx, F32)
    want = (Xo.double().numpy() @ wf.T).astype(np.float32)
    ok &= np.array_equal(y2, want)
    return bool(ok)


def pin_select(m) -> bool:
    a = np.array([0.1, 6.0, 5.999, 7.5, 0.0, 6.0], np.float32)
    return np.array_equal(m.select_features(a, 6.0), np.array([1, 3, 5], np.int32)) and m.select_features(a, 100.0).size == 0


PINS = {"convert": pin_convert, "rowquant_exact": pin_rowquant_exact, "division": pin_rowquant_division, "rowquant_properties": pin_rowquant_properties,
        "int_product": pin_int_product, "closed_form": pin_linear_closed_form, "error_bound": pin_linear_error_bound,
        "select": pin_select}


@pytest.mark.parametrize("name", sorted(PINS))
def test_pin(name):
    assert PINS[name](mo)


# ------------------------------------------------------------------------------------------
# planted mistakes: each is applied to a copy of the oracle's source, on the CPU

MUTATIONS = {
    "absmax_includes_critical_features": ("a = np.max(np.abs(v[:, regular]), axis=1)", "a = np.max(np.abs(v), axis=1)", {"rowquant_exact", "rowquant_properties"}),
    "scale_by_128": ("scaled = (v * np.float32(127.0))", "scaled = (v * np.float32(128.0))", {"rowquant_exact"}),
    "round_half_away": ("q = np.rint(t).astype(np.int8)", "q = (np.sign(t) * np.floor(np.abs(t) + 0.5)).astype(np.int8)", {"division"}),
    "multiply_by_reciprocal": ("t = (scaled / d[:, None]).astype(np.float32)", "t = (scaled * (np.float32(1.0) / d)[:, None]).astype(np.float32)", {"division"}),
    "critical_features_not_zeroed": ("q[:, ~regular] = 0", "pass", {"rowquant_exact", "closed_form"}),
    "scale_is_absmax": ("s = (a / np.float32(127.0)).astype(np.float32)", "s = a", {"rowquant_exact", "closed_form"}),
    "weights_not_transposed": ("np.matmul(qx.astype(np.float64), qw.astype(np.float64).T)", "np.matmul(qx.astype(np.float64), qw.astype(np.float64)[:qx.shape[1], :qx.shape[1]])", {"int_product"}),
    "side_part_dropped": ("v = (t * scale + side).astype(np.float32)", "v = (t * scale).astype(np.float32)", {"closed_form", "error_bound"}),
    "side_part_subtracted": ("v = (t * scale + side).astype(np.float32)", "v = (t * scale - side).astype(np.float32)", {"closed_form"}),
    "scale_uses_one_side": ("scale = (sx[:, None] * sw[None, :])", "scale = (sx[:, None] * sx[:, None] + 0 * sw[None, :])", {"closed_form"}),
    "bf16_truncates": ("u = u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))", "u = u", {"convert"}),
    "side_gathers_wrong_columns": ("side[:, :len(idx)] = np.ascontiguousarray(vbits)[:, idx]", "side[:, :len(idx)] = np.ascontiguousarray(vbits)[:, :len(idx)]", {"rowquant_exact", "closed_form"}),
    "select_is_strict": ("np.nonzero(a >= np.float32(tau))", "np.nonzero(a > np.float32(tau))", {"select"}),
}


def mutated(find, repl):
    text = open(SRC).read()
    assert text.count(find) == 1, "mutation anchor not found exactly once"
    mod = types.ModuleType("mmd_oracle_mutant")
    exec(compile(text.replace(find, repl), "mmd_oracle_mutant", "exec"), mod.__dict__)
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
