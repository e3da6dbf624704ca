"""CPU oracle of the block-size selection (test infrastructure only).

The paper's "Dynamic Quantization" item fixes no block size.  This module states, as plain
definitions, what the library's selection calls compute:

  block_errors  for each candidate block: y = the 8-bit roundtrip of x (the oracle's own, in
                ``bq_oracle.cpp``), err2 = sum_i (x_i - y_i)^2 and norm2 = sum_i x_i^2 over the
                widened elements, each as an exactly rounded sum of fp64 terms (math.fsum; the
                differences are exact in fp64, the squares are rounded once).
  pick_block    admissible: err2 <= max_rel_rms^2 * norm2 (fp64); the largest admissible block;
                if none, the candidate with the smallest err2, the larger block on equal sums.

Nothing here is imported by the CUDA library or its binding; it shares no code with it.
Pins: tests/test_oracle_tune.py (hand-computed sums from printed codebook values, closed forms,
every branch of the rule, planted mistakes).
"""
from __future__ import annotations

import math

import numpy as np

from . import F32, roundtrip
from .mmd_oracle import widen


def _as_f64(x: np.ndarray, dt: int) -> np.ndarray:
    x = np.ascontiguousarray(x).reshape(-1)
    return x.astype(np.float64) if dt == F32 else widen(x, dt).astype(np.float64)


def block_errors(x: np.ndarray, dt: int, blocks, cb: np.ndarray):
    """-> ([err2 per candidate], norm2)."""
    v = _as_f64(x, dt)
    err2 = []
    for b in blocks:
        y = _as_f64(roundtrip(x, dt, int(b), cb, dt), dt)
        d = v - y
        err2.append(math.fsum(d * d))
    return err2, math.fsum(v * v)


def pick_block(blocks, err2, norm2: float, max_rel_rms: float) -> int:
    bound = max_rel_rms * max_rel_rms * norm2
    admissible = [int(b) for b, e in zip(blocks, err2) if e <= bound]
    if admissible:
        return max(admissible)
    smallest = min(err2)
    return max(int(b) for b, e in zip(blocks, err2) if e == smallest)
