"""Pins of the block-size selection oracle (CPU only): hand-computed error sums from the paper-defined codebook's
printed values, closed forms (values that are codes reconstruct exactly; a scaled tensor scales its sums), the
monotone effect of an outlier, every branch of the selection rule on hand-made tables, and planted mistakes."""
import math
import os
import types
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from helpers import frac_of
from oracle import tune_oracle as to

F32, F16, BF16 = 0, 1, 2
SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "tune_oracle.py")


def pin_sums(m) -> bool:
    cb = oracle.make_codebook()
    ok = True
    # one block [1, 0.5, -0.25, 0]: xhat = x; the reconstruction is the nearest code value, found here by exact rationals
    x = np.array([1.0, 0.5, -0.25, 0.0], np.float32)
    want = Fraction(0)
    for v in x:
        want += min((frac_of(v) - frac_of(c)) ** 2 for c in cb)
    err2, norm2 = m.block_errors(x, F32, [4, 64], cb)
    ok &= abs(Fraction(err2[0]) - want) <= want * Fraction(1, 10 ** 12) and err2[0] == err2[1] and err2[0] > 0
    ok &= norm2 == 1.0 + 0.25 + 0.0625
    # values that are code values times a power-of-two absmax reconstruct exactly when the block holds +1.0
    vals = (cb[[255, 200, 130, 127, 60, 3]] * np.float32(8.0)).astype(np.float32)
    err2, norm2 = m.block_errors(vals, F32, [6], cb)
    ok &= err2 == [0.0] and norm2 == math.fsum(float(v) ** 2 for v in vals.astype(np.float64))
    # scaling the tensor by 2^k scales both sums by 4^k exactly; bf16 and fp16 inputs are widened, not reinterpreted
    g = torch.Generator().manual_seed(3)
    t = torch.randn(64 * 12, generator=g)
    for dt, tdt in ((F32, torch.float32), (BF16, torch.bfloat16), (F16, torch.float16)):
        a = t.to(tdt)
        b = (t.to(tdt).float() * 8).to(tdt)
        bits = (lambda u: u.numpy() if dt == F32 else u.view(torch.int16).numpy().view(np.uint16))
        e1, n1 = m.block_errors(bits(a), dt, [64, 256], cb)
        e2, n2 = m.block_errors(bits(b), dt, [64, 256], cb)
        ok &= e2 == [64.0 * e for e in e1] and n2 == 64.0 * n1
        ok &= n1 == math.fsum((a.double() ** 2).tolist())
        y = oracle.roundtrip(bits(a), dt, 64, cb, dt)
        yt = torch.from_numpy(y.copy()) if dt == F32 else torch.from_numpy(y.view(np.int16).copy()).view(tdt)
        ok &= e1[0] == math.fsum(((a.double() - yt.double()) ** 2).tolist()) and 0 < e1[0] < 1e-3 * n1
    # an outlier stretches the scale of its block: the larger block loses more
    z = t.clone()
    z[5] = 300.0
    e, _ = m.block_errors(z.numpy(), F32, [64, 256, 768], cb)
    ok &= e[0] < e[1] < e[2]
    return bool(ok)


def pin_rule(m) -> bool:
    ok = True
    blocks = [64, 256, 1024]
    err2, norm2 = [1.0, 2.0, 5.0], 100.0                        # relative rms 0.1, 0.1414, 0.2236
    ok &= m.pick_block(blocks, err2, norm2, 0.15) == 256
    ok &= m.pick_block(blocks, err2, norm2, 0.3) == 1024
    ok &= m.pick_block([64, 256], [0.5, 1.0], 64.0, 0.125) == 256             # 1.0 <= 0.125^2 * 64 exactly: the bound is inclusive
    ok &= m.pick_block(blocks, err2, norm2, 0.05) == 64         # none admissible: the smallest error
    ok &= m.pick_block([1024, 64, 256], [5.0, 1.0, 2.0], norm2, 0.15) == 256   # the order of the candidates does not matter
    ok &= m.pick_block([64, 256], [3.0, 3.0], norm2, 0.01) == 256              # none admissible, equal sums: the larger block
    ok &= m.pick_block([64, 256], [0.0, 0.0], 0.0, 0.0) == 256                 # an all-zero tensor
    ok &= m.pick_block([64, 256, 1024], [2.0, 1.0, 5.0], norm2, 0.15) == 256   # admissible means within the bound, not "smallest"
    return bool(ok)


PINS = {"sums": pin_sums, "rule": pin_rule}


@pytest.mark.parametrize("name", sorted(PINS))
def test_pin(name):
    assert PINS[name](to)


MUTATIONS = {
    "error_against_zero": ("        d = v - y\n", "        d = y\n", {"sums"}),
    "absolute_not_squared": ("        err2.append(math.fsum(d * d))", "        err2.append(math.fsum(np.abs(d)))", {"sums"}),
    "norm_of_reconstruction": ("    return err2, math.fsum(v * v)", "    return err2, math.fsum(y * y)", {"sums"}),
    "bits_not_widened": ("x.astype(np.float64) if dt == F32 else widen(x, dt).astype(np.float64)", "x.astype(np.float64)", {"sums"}),
    "bound_not_squared": ("    bound = max_rel_rms * max_rel_rms * norm2", "    bound = max_rel_rms * norm2", {"rule"}),
    "smallest_admissible": ("        return max(admissible)", "        return min(admissible)", {"rule"}),
    "strict_bound": ("if e <= bound]", "if e < bound]", {"rule"}),
    "fallback_largest_error": ("    smallest = min(err2)", "    smallest = max(err2)", {"rule"}),
}


def mutated(find, repl):
    text = open(SRC).read()
    assert text.count(find) == 1, "mutation anchor not found exactly once"
    text = text.replace(find, repl).replace("from . import F32, roundtrip", "from oracle import F32, roundtrip").replace("from .mmd_oracle import", "from oracle.mmd_oracle import")
    mod = types.ModuleType("tune_oracle_mutant")
    exec(compile(text, "tune_oracle_mutant", "exec"), mod.__dict__)
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
