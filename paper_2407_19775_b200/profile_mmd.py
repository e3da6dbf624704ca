"""Runs a few launches of the decomposed linear layer on a slice of a linear workload, for
profilers and for timing.

    python -m paper_2407_19775_b200.profile_mmd --workload mmd_prefill_moe --tokens 2048 --out-features 4096 --launches 3

Prints the CUDA-event time of every call (row kernel + product kernel) and, with --graph, the
GPU time of the same call replayed from a CUDA graph (no host launch overhead).
"""
from __future__ import annotations

import argparse

import torch

from . import DecomposedLinear, workloads
from .mmd import PATH_AUTO, PATH_GENERAL, PATH_TENSOR, PATH_TENSOR_SOLO, PATH_TENSOR_STREAMK, PATH_TENSOR_TILE


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="mmd_prefill_moe", choices=sorted(workloads.LINEAR_WORKLOADS))
    ap.add_argument("--tokens", type=int, default=None)
    ap.add_argument("--out-features", type=int, default=None)
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--path", default="auto", choices=["auto", "general", "tensor", "tile", "solo", "streamk"])
    ap.add_argument("--no-features", action="store_true", help="decompose without critical features")
    ap.add_argument("--graph", action="store_true", help="also time a CUDA-graph replay of the call")
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    X, W, idx = workloads.make_linear(args.workload, args.tokens, args.out_features)
    if args.no_features:
        idx = idx[:0]
    X, W = X.to(dev), W.to(dev)
    lin = DecomposedLinear(W, idx)
    M, N, K = X.shape[0], W.shape[0], W.shape[1]
    y = torch.empty((M, N), dtype=X.dtype, device=dev)
    ws = lin.workspace(M, streamk=(args.path == "streamk"))
    path = {"auto": PATH_AUTO, "general": PATH_GENERAL, "tensor": PATH_TENSOR, "tile": PATH_TENSOR_TILE, "solo": PATH_TENSOR_SOLO, "streamk": PATH_TENSOR_STREAMK}[args.path]
    torch.cuda.synchronize()
    for i in range(args.launches):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        lin.linear(X, y_out=y, path=path, workspace=ws)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        print(f"mmd_linear {args.workload} M={M} K={K} N={N} features={idx.size} path={args.path} call {i}: {ms:.4f} ms, "
              f"{2.0 * M * N * K / ms / 1e9:.0f} TOP/s, status {lin.kernel_status()}")
    if args.graph:
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            lin.linear(X, y_out=y, path=path, workspace=ws)
            s.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                lin.linear(X, y_out=y, path=path, workspace=ws)
            reps = 20
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g.replay()
            e0.record(s)
            for _ in range(reps):
                g.replay()
            e1.record(s)
            s.synchronize()
        ms = e0.elapsed_time(e1) / reps
        print(f"graph replay: {ms:.4f} ms per call, {2.0 * M * N * K / ms / 1e9:.0f} TOP/s")


if __name__ == "__main__":
    main()
