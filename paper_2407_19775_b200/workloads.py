"""Seeded synthetic hidden-state tensors (input generators only).

This module holds none of the method's arithmetic: it only draws the activations that
cross a shard boundary, with the shapes ([batch, seq, hidden] of 7B / 70B / MoE-class
models), the element types and the value structure (heavy tails, a few persistent outlier
channels, sparse spikes) of LLM hidden states.  The same bytes are handed to the CUDA
library and to the CPU checker, so everything is drawn on the CPU with a seeded
``torch.Generator`` in fp32 and cast once (round-to-nearest-even) to the workload's type.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    shape: tuple
    dtype: torch.dtype
    blocks: tuple          # block sizes this workload is run with
    seed: int
    recipe: str

    @property
    def n(self) -> int:
        return int(np.prod(self.shape))


WORKLOADS = {
    "tiny": Workload("tiny", (64, 256), torch.float32, (64,), 0,
                     "N(0,1); block 0 all zero; block 1 elem 0 = -50; block 2 elem 0 = +50"),
    "prefill7b": Workload("prefill7b", (1, 2048, 4096), torch.bfloat16, (256,), 1,
                          "N(0,0.5); 6 outlier channels x40"),
    "decode70b": Workload("decode70b", (64, 1, 8192), torch.float16, (64,), 2,
                          "Student-t(nu=3) x0.3"),
    "moe_prefill": Workload("moe_prefill", (8, 4096, 4096), torch.bfloat16, (2048,), 3,
                            "N(0,1); 0.1% of elements replaced by +-U(20,80)"),
    "sweep1g": Workload("sweep1g", (16, 4096, 8192), torch.bfloat16, (64, 256, 1024, 4096), 4,
                        "Laplace(0,0.5); 8 outlier channels x60"),
}

_CHUNK_ROWS_ELEMS = 1 << 24      # fp32 staging is drawn in pieces of at most this many elements


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return g


def _rows_per_chunk(hidden: int) -> int:
    return max(1, _CHUNK_ROWS_ELEMS // hidden)


def _tiny(w: Workload, rows: int | None) -> torch.Tensor:
    g = _gen(w.seed)
    x = torch.randn(w.shape, generator=g, dtype=torch.float32)
    flat = x.view(-1)
    flat[0:64] = 0.0
    flat[64] = -50.0
    flat[128] = 50.0
    return x


def _prefill7b(w: Workload, rows: int | None) -> torch.Tensor:
    g = _gen(w.seed)
    hidden = w.shape[-1]
    tokens = w.n // hidden if rows is None else rows
    x = torch.randn((w.n // hidden, hidden), generator=g, dtype=torch.float32)[:tokens] * 0.5
    channels = torch.randperm(hidden, generator=g)[:6]
    x[:, channels] *= 40.0
    return x.to(w.dtype)


def _decode70b(w: Workload, rows: int | None) -> torch.Tensor:
    g = _gen(w.seed)
    hidden = w.shape[-1]
    total = w.n // hidden
    z = torch.randn((total, hidden), generator=g, dtype=torch.float32)
    chi2 = torch.zeros_like(z)
    for _ in range(3):
        chi2 += torch.randn((total, hidden), generator=g, dtype=torch.float32) ** 2
    x = z / torch.sqrt(chi2 / 3.0) * 0.3
    if rows is not None:
        x = x[:rows]
    return x.to(w.dtype)


def _moe_prefill(w: Workload, rows: int | None) -> torch.Tensor:
    g = _gen(w.seed)
    hidden = w.shape[-1]
    total = w.n // hidden if rows is None else rows
    out = torch.empty((total, hidden), dtype=w.dtype)
    step = _rows_per_chunk(hidden)
    for r0 in range(0, total, step):
        r1 = min(total, r0 + step)
        x = torch.randn((r1 - r0, hidden), generator=g, dtype=torch.float32)
        mask = torch.rand((r1 - r0, hidden), generator=g) < 0.001
        sign = torch.where(torch.rand((r1 - r0, hidden), generator=g) < 0.5, -1.0, 1.0)
        spike = sign * (20.0 + 60.0 * torch.rand((r1 - r0, hidden), generator=g))
        out[r0:r1] = torch.where(mask, spike, x).to(w.dtype)
    return out


def _sweep1g(w: Workload, rows: int | None) -> torch.Tensor:
    g = _gen(w.seed)
    hidden = w.shape[-1]
    total = w.n // hidden if rows is None else rows
    channels = torch.randperm(hidden, generator=g)[:8]      # drawn first so a row prefix is stable
    out = torch.empty((total, hidden), dtype=w.dtype)
    step = _rows_per_chunk(hidden)
    for r0 in range(0, total, step):
        r1 = min(total, r0 + step)
        u = torch.rand((r1 - r0, hidden), generator=g, dtype=torch.float32) - 0.5
        # inverse CDF of Laplace(0, b = 0.5): x = -b * sgn(u) * ln(1 - 2|u|)
        x = -0.5 * torch.sign(u) * torch.log1p(-2.0 * u.abs())
        x = torch.nan_to_num(x, posinf=8.0, neginf=-8.0)  # u = -0.5 exactly would give inf
        x[:, channels] *= 60.0
        out[r0:r1] = x.to(w.dtype)
    return out


_MAKERS = {"tiny": _tiny, "prefill7b": _prefill7b, "decode70b": _decode70b,
           "moe_prefill": _moe_prefill, "sweep1g": _sweep1g}


def make(name: str, rows: int | None = None) -> torch.Tensor:
    """Draw workload ``name`` on the CPU.  ``rows`` keeps only the first ``rows`` rows of the
    flattened [tokens, hidden] tensor (the chunked generators make a prefix identical to the
    same rows of the full tensor); ``None`` draws all of it.  The result is contiguous and is
    returned flattened to [tokens, hidden] (``tiny`` keeps its 64 x 256 shape)."""
    w = WORKLOADS[name]
    x = _MAKERS[name](w, rows)
    return x.contiguous()


def as_numpy_bits(x: torch.Tensor) -> np.ndarray:
    """View a CPU tensor as the flat numpy array the CPU checker takes: float32 as is,
    fp16 / bf16 as their uint16 bit patterns."""
    x = x.detach().cpu().contiguous().view(-1)
    if x.dtype == torch.float32:
        return x.numpy()
    return x.view(torch.int16).numpy().view(np.uint16)


def from_numpy_bits(a: np.ndarray, dtype: torch.dtype) -> torch.Tensor:
    """Inverse of :func:`as_numpy_bits`."""
    if dtype == torch.float32:
        return torch.from_numpy(np.ascontiguousarray(a, np.float32))
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(dtype)
