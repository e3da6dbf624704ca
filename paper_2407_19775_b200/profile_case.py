"""Runs a few launches of one library call on a prefix of a workload, for profilers.

    python -m paper_2407_19775_b200.profile_case --op roundtrip --block 4096 --rows 8192 --launches 3

`--rows 8192` of `sweep1g` is 64 Mi bf16 elements (128 MiB in, larger than L2) and keeps the
device footprint well under 1 GB, which is what a counter-collecting profiler wants.  Prints
the CUDA-event time of each launch.

    python -m paper_2407_19775_b200.profile_case --op mtpp --workload mtpp_unet --launches 3

decodes and slices the workload's population of topological orders (two kernels per launch).
"""
from __future__ import annotations

import argparse

import torch

from . import Codebook, Codebook4, bq4_dequantize, bq4_quantize, bq_dequantize, bq_quantize, bq_roundtrip, mtpp, tune, workloads


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="sweep1g")
    ap.add_argument("--op", default="roundtrip", choices=["quantize", "dequantize", "roundtrip", "roundtrip_side", "quantize4", "dequantize4", "block_errors", "sweep", "mtpp"])
    ap.add_argument("--block", type=int, default=4096)
    ap.add_argument("--rows", type=int, default=8192)
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--dtype", default=None, choices=[None, "bf16", "fp16", "fp32"], help="cast the workload to this type first")
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    if args.op == "mtpp":
        name = args.workload if args.workload in workloads.GRAPH_WORKLOADS else "mtpp_unet"
        w = workloads.GRAPH_WORKLOADS[name]
        graph = mtpp.SliceGraph(*workloads.make_graph(name), device=dev)
        keys = workloads.make_keys(name, w.population).to(dev)
        orders = out = None
        for i in range(args.launches):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            ev[0].record()
            orders = graph.decode_orders(keys, orders)
            ev[1].record()
            out = graph.slice_orders(orders, w.k, w.B, w.M, out)
            ev[2].record()
            torch.cuda.synchronize()
            print(f"{name} population {w.population} launch {i}: decode {ev[0].elapsed_time(ev[1]):.4f} ms, slice {ev[1].elapsed_time(ev[2]):.4f} ms, "
                  f"flagged {int(out[3].sum())}")
        return
    x = workloads.make(args.workload, rows=args.rows).view(-1).to(dev)
    if args.dtype is not None:
        x = x.to({"bf16": torch.bfloat16, "fp16": torch.float16, "fp32": torch.float32}[args.dtype])
    n = x.numel()
    cb = Codebook(device=dev)
    codes = torch.empty(n, dtype=torch.uint8, device=dev)
    absmax = torch.empty((n + min(args.block, 64) - 1) // min(args.block, 64), dtype=torch.float32, device=dev)
    y = torch.empty_like(x)
    cb4 = Codebook4()
    packed = codes[: (n + 1) // 2]
    if args.op == "dequantize":
        bq_quantize(x, args.block, cb, codes, absmax)
    if args.op == "dequantize4":
        bq4_quantize(x, args.block, cb4, packed, absmax)
    if args.op == "block_errors":                                # one candidate: the roundtrip, then the two kernels of the sums
        tune_ws = torch.empty(tune.workspace_bytes(x.dtype, n), dtype=torch.uint8, device=dev)
        tune_sums = torch.empty(2, dtype=torch.float64, device=dev)
    if args.op == "sweep":
        # the benchmark's step, launch by launch: for each block size quantize, dequantize, fused roundtrip (12 launches per pass)
        for i in range(args.launches):
            for block in (64, 256, 1024, 4096):
                am = absmax[: n // block]
                for op in ("quantize", "dequantize", "roundtrip"):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    if op == "quantize":
                        bq_quantize(x, block, cb, codes, am)
                    elif op == "dequantize":
                        bq_dequantize(codes, am, block, cb, x.dtype, y)
                    else:
                        bq_roundtrip(x, block, cb, y_out=y)
                    e1.record()
                    torch.cuda.synchronize()
                    print(f"{op} {str(x.dtype)[6:]} block={block} n={n} pass {i}: {e0.elapsed_time(e1):.4f} ms")
        return
    torch.cuda.synchronize()
    for i in range(args.launches):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        if args.op == "quantize":
            bq_quantize(x, args.block, cb, codes, absmax)
        elif args.op == "dequantize":
            bq_dequantize(codes, absmax, args.block, cb, x.dtype, y)
        elif args.op == "quantize4":
            bq4_quantize(x, args.block, cb4, packed, absmax)
        elif args.op == "dequantize4":
            bq4_dequantize(packed, absmax, n, args.block, cb4, x.dtype, y)
        elif args.op == "block_errors":
            tune.block_errors(x, [args.block], cb, tune_ws, tune_sums)
        elif args.op == "roundtrip":
            bq_roundtrip(x, args.block, cb, y_out=y)
        else:
            bq_roundtrip(x, args.block, cb, y_out=y, codes_out=codes, absmax_out=absmax)
        e1.record()
        torch.cuda.synchronize()
        print(f"{args.op} {str(x.dtype)[6:]} block={args.block} n={n} launch {i}: {e0.elapsed_time(e1):.4f} ms")


if __name__ == "__main__":
    main()
