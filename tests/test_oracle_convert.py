"""The oracle's hand-written fp16 / bf16 conversions against torch's CPU casts (CPU only)."""
import numpy as np
import torch

import oracle
from paper_2407_19775_b200 import workloads

F16, BF16 = oracle.F16, oracle.BF16


def _all_patterns(dtype):
    bits = np.arange(65536, dtype=np.uint16)
    return bits, workloads.from_numpy_bits(bits, dtype)


def test_widen_all_patterns():
    for dt, tdt in ((F16, torch.float16), (BF16, torch.bfloat16)):
        bits, t = _all_patterns(tdt)
        ref = t.float().numpy()
        got = np.array([oracle.widen(int(b), dt) for b in bits], np.float32)
        nan = np.isnan(ref)
        assert np.array_equal(np.isnan(got), nan)
        assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))


def test_narrow_is_inverse_of_widen():
    for dt, tdt in ((F16, torch.float16), (BF16, torch.bfloat16)):
        bits, t = _all_patterns(tdt)
        f = t.float().numpy()
        for b, v in zip(bits[::7], f[::7]):
            if np.isnan(v):
                continue
            assert oracle.narrow(float(v), dt) == int(b)


def test_narrow_rounding_against_torch():
    rng = np.random.default_rng(1)
    u = rng.integers(0, 2 ** 32, 200_000, dtype=np.uint64).astype(np.uint32)
    # every halfway pattern of a few exponents, the overflow edge and the fp16 subnormal range
    half_bf16 = ((np.arange(0x3F00, 0x4100, dtype=np.uint32) << 16) | 0x8000)
    edge = np.array([0x477FE000, 0x477FEFFF, 0x477FF000, 0x33000000, 0x33000001, 0x33800000, 0x387FC000,
                     0x387FE000, 0x00000001, 0x80000001, 0x7F7FFFFF, 0x7F800000, 0xFF800000], np.uint32)
    sub = rng.integers(0x33000000, 0x38800000, 50_000, dtype=np.uint64).astype(np.uint32)
    halfway16 = (rng.integers(0x38800000 >> 13, 0x47800000 >> 13, 20_000, dtype=np.uint64).astype(np.uint32) << 13) | 0x1000
    allu = np.concatenate([u, half_bf16, edge, sub, halfway16])
    f = allu.view(np.float32)
    f = f[~np.isnan(f)]
    t = torch.from_numpy(f.copy())
    for dt, tdt in ((F16, torch.float16), (BF16, torch.bfloat16)):
        ref = workloads.as_numpy_bits(t.to(tdt))
        got = np.array([oracle.narrow(float(v), dt) for v in f], np.uint16)
        assert np.array_equal(got, ref)
