"""CPU oracle of the mixed matrix decomposition (test infrastructure only).

Paper, section "Compression techniques", item 2 ("Mixed matrix decomposition"): the weight
matrices go from 16-bit to 8-bit values while a small fraction of critical weights stays at
16-bit precision.  The paper states no more than that; the reading taken here (every point
is a stated reading, listed in the design notes) is the vector-wise int8 decomposition with
a 16-bit side matrix over a fixed set O of critical input features:

  rowquant (weights once, activations per call), for every row r of a [R, K] 16-bit matrix
      a_r  = max over k not in O of |v[r,k]|                      (exact)
      d_r  = a_r, or 1 when a_r == 0
      q[r,k] = 0 for k in O, else rint( RN32( RN32(127 * v[r,k]) / d_r ) )   (ties to even)
      s_r  = RN32( a_r / 127 )
      side[r,j] = v[r, O_j] for j < |O|, zero for the padding columns up to a multiple of 64
  linear  Y = X W^T for X [M, K], W [N, K]
      acc[m,n]  = sum_k qx[m,k] * qw[n,k]                         (exact integer)
      side[m,n] = sum_j xo[m,j] * wo[n,j]                         (real sum)
      y[m,n]    = narrow( fl(acc) * RN32(sx[m] * sw[n]) + side ),  fl = int -> fp32 (RNE)

Nothing here is imported by the CUDA library or its binding; only the tests, the smoke
check and the CPU legs of the benchmark call it.  It shares no code with the CUDA path.
Element types follow the other oracle: fp16 / bf16 arrays are ``uint16`` bit patterns.

Pins (tests/test_oracle_mmd.py): exact-rational brute force of the rounding chain, the
textbook integer product by plain loops, closed forms where the quantization is exact,
the error bound of the decomposition, torch CPU conversions, and planted mistakes.
Parity with any outside library's int8 decomposition: parity unpinned.
"""
from __future__ import annotations

import numpy as np

F32, F16, BF16 = 0, 1, 2
SIDE_PAD = 64          # the side matrices are padded with zero columns to a multiple of this


def widen(bits: np.ndarray, dt: int) -> np.ndarray:
    """16-bit patterns -> float32, exact."""
    bits = np.ascontiguousarray(bits)
    if dt == BF16:
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    if dt == F16:
        return bits.view(np.float16).astype(np.float32)
    raise ValueError("rowquant takes fp16 or bf16")


def narrow(v: np.ndarray, dt: int) -> np.ndarray:
    """float32 -> dt with round-to-nearest-even (finite inputs)."""
    v = np.ascontiguousarray(v, np.float32)
    if dt == F32:
        return v
    if dt == F16:
        return v.astype(np.float16).view(np.uint16)
    u = v.view(np.uint32).astype(np.uint64)
    u = u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))
    return (u >> np.uint64(16)).astype(np.uint16)


def side_columns(ko: int) -> int:
    return ((ko + SIDE_PAD - 1) // SIDE_PAD) * SIDE_PAD


def select_features(feature_absmax: np.ndarray, tau: float) -> np.ndarray:
    """Critical input features: those whose calibration magnitude reaches tau; ascending."""
    a = np.asarray(feature_absmax, np.float32)
    return np.nonzero(a >= np.float32(tau))[0].astype(np.int32)


def rowquant(vbits: np.ndarray, dt: int, idx: np.ndarray):
    """-> (q int8 [R,K], s float32 [R], side uint16 [R, side_columns(len(idx))])."""
    v = widen(vbits, dt)
    R, K = v.shape
    idx = np.asarray(idx, np.int64)
    regular = np.ones(K, bool)
    regular[idx] = False
    a = np.zeros(R, np.float32)
    if regular.any():
        a = np.max(np.abs(v[:, regular]), axis=1).astype(np.float32)
    d = np.where(a != 0, a, np.float32(1.0)).astype(np.float32)
    scaled = (v * np.float32(127.0)).astype(np.float32)                 # exact for 16-bit inputs
    t = (scaled / d[:, None]).astype(np.float32)                        # one IEEE division
    q = np.rint(t).astype(np.int8)                                      # ties to even
    q[:, ~regular] = 0
    s = (a / np.float32(127.0)).astype(np.float32)
    side = np.zeros((R, side_columns(len(idx))), np.uint16)
    side[:, :len(idx)] = np.ascontiguousarray(vbits)[:, idx]
    return q, s, side


def int_product(qx: np.ndarray, qw: np.ndarray) -> np.ndarray:
    """acc = qx qw^T as exact integers.  The float64 product is exact: every partial sum is an
    integer below 2^53 (K * 127^2 < 2^53), so the order of the additions cannot matter."""
    return np.matmul(qx.astype(np.float64), qw.astype(np.float64).T).astype(np.int64)


def linear(xbits: np.ndarray, dt: int, qw: np.ndarray, sw: np.ndarray, wo: np.ndarray, idx: np.ndarray, ydt: int,
           parts: bool = False):
    """The decomposed linear layer.  ydt is F32 or dt.  With parts=True also returns
    (acc, side sum in float64, sum of |side products|) for tolerance derivations."""
    qx, sx, xo = rowquant(xbits, dt, idx)
    acc = int_product(qx, qw)
    t = acc.astype(np.float32).astype(np.float64)                       # int -> fp32, RNE
    scale = (sx[:, None] * sw[None, :]).astype(np.float32).astype(np.float64)
    xo_f = widen(xo, dt).astype(np.float64)
    wo_f = widen(wo, dt).astype(np.float64)
    side = xo_f @ wo_f.T
    v = (t * scale + side).astype(np.float32)                           # t * scale is exact in float64
    y = narrow(v, ydt)
    if parts:
        return y, acc, side, np.abs(xo_f) @ np.abs(wo_f).T
    return y


def reconstruct(q: np.ndarray, s: np.ndarray, side: np.ndarray, dt: int, idx: np.ndarray) -> np.ndarray:
    """The matrix the decomposition stands for, in float64: q * s outside O, the kept 16-bit
    values inside O."""
    w = q.astype(np.float64) * s.astype(np.float64)[:, None]
    w[:, np.asarray(idx, np.int64)] = widen(side, dt).astype(np.float64)[:, :len(idx)]
    return w
