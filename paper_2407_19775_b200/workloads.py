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


# ------------------------------------------------------------------------------------------
# Linear layers for the mixed matrix decomposition: activations X [tokens, in_features] with
# a few persistent outlier features, weights W [out_features, in_features], and the indices
# of the planted outlier features (what a calibration pass would report as critical).

@dataclass(frozen=True)
class LinearWorkload:
    name: str
    tokens: int
    in_features: int
    out_features: int
    dtype: torch.dtype
    n_outlier_features: int
    seed: int
    recipe: str


LINEAR_WORKLOADS = {
    "mmd_tiny": LinearWorkload("mmd_tiny", 37, 320, 72, torch.bfloat16, 3, 10,
                               "X = 0.5 N(0,1), 3 features x40; W = 0.05 N(0,1); ragged tokens and out_features"),
    "mmd_decode70b": LinearWorkload("mmd_decode70b", 64, 8192, 8192, torch.float16, 8, 11,
                                    "X = 0.3 Student-t(3), 8 features x30; W = 0.02 N(0,1)"),
    "mmd_prefill_moe": LinearWorkload("mmd_prefill_moe", 4096, 6144, 16384, torch.bfloat16, 6, 12,
                                      "X = 0.5 N(0,1), 6 features x40; W = 0.02 N(0,1) with 0.05% entries x8"),
}


def make_linear(name: str, tokens: int | None = None, out_features: int | None = None):
    """Draws (X, W, outlier_features) of linear workload ``name`` on the CPU.  ``tokens`` /
    ``out_features`` keep only the first rows of X / W (a prefix equals the same rows of the
    full draw).  outlier_features is an ascending int32 numpy array."""
    w = LINEAR_WORKLOADS[name]
    g = _gen(w.seed)
    K = w.in_features
    feats = torch.sort(torch.randperm(K, generator=g)[:w.n_outlier_features]).values
    M = w.tokens if tokens is None else min(tokens, w.tokens)
    N = w.out_features if out_features is None else min(out_features, w.out_features)
    gx = _gen(w.seed + 1000)
    gw = _gen(w.seed + 2000)
    X = torch.empty((M, K), dtype=w.dtype)
    step = _rows_per_chunk(K)
    for r0 in range(0, M, step):
        r1 = min(M, r0 + step)
        if name == "mmd_decode70b":
            z = torch.randn((r1 - r0, K), generator=gx)
            chi2 = sum(torch.randn((r1 - r0, K), generator=gx) ** 2 for _ in range(3))
            x = z / torch.sqrt(chi2 / 3.0) * 0.3
            x[:, feats] *= 30.0
        else:
            x = torch.randn((r1 - r0, K), generator=gx) * 0.5
            x[:, feats] *= 40.0
        X[r0:r1] = x.to(w.dtype)
    W = torch.empty((N, K), dtype=w.dtype)
    for r0 in range(0, N, step):
        r1 = min(N, r0 + step)
        v = torch.randn((r1 - r0, K), generator=gw) * (0.05 if name == "mmd_tiny" else 0.02)
        if name == "mmd_prefill_moe":
            v = torch.where(torch.rand((r1 - r0, K), generator=gw) < 0.0005, v * 8.0, v)
        W[r0:r1] = v.to(w.dtype)
    return X.contiguous(), W.contiguous(), feats.numpy().astype(np.int32)


def bits_2d(x: torch.Tensor) -> np.ndarray:
    """A 2-D fp16 / bf16 CPU tensor as a uint16 bit-pattern array of the same shape."""
    return as_numpy_bits(x).reshape(x.shape)


# ------------------------------------------------------------------------------------------
# Computation graphs for the slicing of topological orders: layered networks that are not a plain
# chain of equal blocks (a U-shaped denoiser with skip connections and a conditioning node that
# feeds every stage; a trunk with several prediction heads of different depth), the kind of model
# the paper's dynamic sharding is for.  Node attributes are integers: work in microseconds,
# sizeparam and sizeout in bytes; B is the link's bytes per microsecond, M the fast memory in bytes.
# The priority vectors of a population are uniform keys in [0, 1).  Only inputs are drawn here:
# decoding keys into orders and costing blocks is the method's work.

@dataclass(frozen=True)
class GraphWorkload:
    name: str
    kind: str
    n: int
    k: int
    population: int
    B: int
    M: int
    seed: int
    recipe: str


GRAPH_WORKLOADS = {
    "mtpp_tiny": GraphWorkload("mtpp_tiny", "random", 14, 3, 6, 3, 4000, 20, "random DAG, edge probability 0.25"),
    "mtpp_heads": GraphWorkload("mtpp_heads", "heads", 96, 4, 24, 125, 6 << 20, 21,
                                "a trunk of 40 operations and 4 heads of 8..20 operations reading different trunk depths; 1 Gbit/s link"),
    "mtpp_unet": GraphWorkload("mtpp_unet", "unet", 256, 8, 2048, 125, 48 << 20, 22,
                               "U-shaped denoiser: 7 stages down, one across, 7 up, each an entry, three parallel branches, a merge and a closing operation; skip connections; one conditioning node feeding every stage; 1 Gbit/s link"),
}


def make_graph(name: str):
    """Returns (n, edges int32 [m, 2], work, sizeparam, sizeout as int64 arrays) of graph workload ``name``."""
    w = GRAPH_WORKLOADS[name]
    rng = np.random.default_rng(w.seed)
    n = w.n
    edges = []
    if w.kind == "random":
        edges = [(u, v) for u in range(n) for v in range(u + 1, n) if rng.random() < 0.25]
    elif w.kind == "heads":
        trunk = 40
        edges += [(i, i + 1) for i in range(trunk - 1)]
        at = trunk
        for h, depth in enumerate((8, 12, 16, 20)):
            tap = 9 + 10 * h                                  # each head reads another depth of the trunk
            edges.append((tap, at))
            edges += [(at + i, at + i + 1) for i in range(depth - 1)]
            if h % 2:
                edges.append((tap - 4, at + depth // 2))      # and a second, earlier feature half-way
            at += depth
        assert at == n
    else:
        # node 0 is the conditioning node; then stages of 17 operations: an entry, three parallel branches of 7, 5 and 2
        # operations (so that a stage has many topological orders), a merge and a closing operation
        per, branches = 17, (7, 5, 2)
        stages = (n - 1) // per
        assert 1 + stages * per == n and stages % 2 == 1
        closing = []
        merges = []
        for s in range(stages):
            entry = 1 + s * per
            edges.append((0, entry))                          # conditioning enters every stage
            if s:
                edges.append((closing[-1], entry))
            at = entry + 1
            merge = entry + 1 + sum(branches)
            for depth in branches:
                edges.append((entry, at))
                edges += [(at + i, at + i + 1) for i in range(depth - 1)]
                edges.append((at + depth - 1, merge))
                at += depth
            edges.append((merge, merge + 1))
            merges.append(merge)
            closing.append(merge + 1)
        for s in range(stages // 2):
            edges.append((closing[s], merges[stages - 1 - s]))                   # skip: end of down-stage s -> merge of its up-stage
    work = rng.integers(20, 2000, n)
    sizeparam = rng.integers(0, 8 << 20, n) * (rng.random(n) < 0.6)
    sizeout = rng.integers(64 << 10, 4 << 20, n)
    e = np.asarray(sorted(set(edges)), np.int32).reshape(-1, 2)
    return n, e, work.astype(np.int64), sizeparam.astype(np.int64), sizeout.astype(np.int64)


def make_keys(name: str, population: int | None = None) -> torch.Tensor:
    """Uniform priority vectors [population, n] float32 (a row of equal keys is put first)."""
    w = GRAPH_WORKLOADS[name]
    P = w.population if population is None else population
    keys = torch.rand((P, w.n), generator=_gen(w.seed + 500), dtype=torch.float32)
    keys[0] = 0.5
    return keys
