#!/usr/bin/env python
"""Benchmark of the blockwise-quantization hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload: the 1 GiB bf16 block-size sweep ([16, 4096, 8192], Laplace(0, 0.5) with 8 outlier
channels x60, seed 4).  One step is one pass of the whole hot path over that tensor: for
each block size in {64, 256, 1024, 4096}: bq_quantize, bq_dequantize and the fused
bq_roundtrip (12 kernel launches).  The metric is GB/s of input activation processed
(n * 2 bytes per call, 12 calls per step).  The tensor is larger than L2, so every launch
streams from HBM.  One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2407_19775_b200 import workloads

WORKLOAD = "sweep1g"
BLOCKS = (64, 256, 1024, 4096)
OPS = ("quantize", "dequantize", "roundtrip")
METRIC = "quantize+dequantize GB/s of activations and fraction of HBM roofline, 1xB200"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def algorithmic_bytes(op: str, n: int, block: int, s_in: int = 2, s_out: int = 2) -> float:
    """Bytes one launch must move: input read once, outputs written once."""
    nb = (n + block - 1) // block
    if op == "quantize":
        return n * s_in + n + 4 * nb
    if op == "dequantize":
        return n + 4 * nb + n * s_out
    return n * s_in + n * s_out


def progress(section: str, payload) -> None:
    """Finished sections go to stderr as they complete (one JSON object per line), so that a run that
    is killed keeps what it had measured; stdout carries only the final line."""
    sys.stderr.write(json.dumps({"section": section, "result": payload}) + "\n")
    sys.stderr.flush()


def sha256_of(t: torch.Tensor) -> str:
    """SHA-256 of a host tensor's bytes (the seeded input as the kernels and the oracle both see it)."""
    import hashlib
    flat = t.contiguous().view(-1).view(torch.uint8).numpy()
    h = hashlib.sha256()
    step = 1 << 26
    for s0 in range(0, flat.size, step):
        h.update(flat[s0:s0 + step].data)
    return h.hexdigest()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------ distributed plumbing

def dist_setup(n_gpus: int, backend: str):
    """Returns (rank, world).  One process per GPU; torchrun sets the environment."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        if not dist.is_initialized():
            dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def barrier(world: int, device=None):
    if world > 1:
        import torch.distributed as dist
        if device is not None and device.type == "cuda":
            dist.barrier(device_ids=[device.index])
        else:
            dist.barrier()


def max_over_ranks(value: float, world: int, device=None) -> float:
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: float, world: int, max_seconds: float) -> float:
    """Weak scaling: every rank processes the same number of units; the job's rate is all
    ranks' units over the slowest rank's time."""
    return units_per_rank * world / max_seconds


# ------------------------------------------------------------------------------------------ clocks

class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = f"/tmp/bq_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "50"], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, smax, power, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        try:
            for line in open(self.path):
                f = [c.strip() for c in line.split(",")]
                if len(f) < 9:
                    continue
                sm.append(float(f[1])); smax.append(float(f[2])); power.append(float(f[3]))
                for name, v in zip(names, f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.remove(self.path)
        except Exception:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "power_w_max": float(max(power)),
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ the CUDA arm

def run_ours(args):
    import paper_2407_19775_b200 as bq
    from paper_2407_19775_b200 import binding
    binding.lib()                                   # fail now if the CUDA library is missing
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the hot path has no CPU fallback")
    rank, world = dist_setup(args.gpus, "nccl")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)

    global WORKLOAD, BLOCKS
    WORKLOAD = args.config
    w = workloads.WORKLOADS[WORKLOAD]
    BLOCKS = tuple(w.blocks)
    x_host = workloads.make(WORKLOAD).view(-1)
    n = x_host.numel()
    es = x_host.element_size()
    x_pin = x_host.pin_memory()
    del x_host
    input_sha = sha256_of(x_pin) if rank == 0 else None
    cb = bq.Codebook(device=dev)
    x = x_pin.to(dev, non_blocking=True)
    codes = torch.empty(n, dtype=torch.uint8, device=dev)
    absmax = {b: torch.empty((n + b - 1) // b, dtype=torch.float32, device=dev) for b in BLOCKS}
    y = torch.empty(n, dtype=w.dtype, device=dev)
    # A tensor that fits in L2 (126 MB) would be timed L2-resident: a 256 MiB buffer is written before every
    # launch, outside the per-launch events, and `value` is then taken from the launches' own event times.
    fits_l2 = 2 * n * es < (120 << 20)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if fits_l2 else None
    torch.cuda.synchronize()

    def launch(op, b):
        if op == "quantize":
            bq.bq_quantize(x, b, cb, codes, absmax[b])
        elif op == "dequantize":
            bq.bq_dequantize(codes, absmax[b], b, cb, w.dtype, y)
        else:
            bq.bq_roundtrip(x, b, cb, y_out=y)

    def step(events=None):
        for b in BLOCKS:
            for op in OPS:
                if flush is not None:
                    flush.fill_(1)
                if events is not None:
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    launch(op, b)
                    e1.record()
                    events.append((op, b, e0, e1))
                else:
                    launch(op, b)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    events = []
    barrier(world, dev)
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        step(events)
    t1.record()
    torch.cuda.synchronize()
    barrier(world, dev)
    local_s = t0.elapsed_time(t1) / 1e3
    clocks = sampler.stop() if rank == 0 else None
    max_s = max_over_ranks(local_s, world, dev)

    bytes_per_step = n * es * len(BLOCKS) * len(OPS)
    # per-kernel durations from the events recorded inside the timed region
    peak, peak_kind = measured_peak()
    per = {}
    for op, b, e0, e1 in events:
        per.setdefault((op, b), []).append(e0.elapsed_time(e1))
    if flush is not None:                            # the flush writes are not the path's work: count the launches' own time
        local_s = sum(sum(v) for v in per.values()) / 1e3
        max_s = max_over_ranks(local_s, world, dev)
    value = whole_job_value(bytes_per_step * args.steps, world, max_s) / 1e9
    kernels = {}
    for (op, b), ms in per.items():
        avg = float(np.mean(ms))
        ab = algorithmic_bytes(op, n, b, es, es)
        kernels[f"{op}_b{b}"] = {
            "ms": round(avg, 4), "ms_min": round(float(np.min(ms)), 4), "algorithmic_bytes": int(ab), "traffic": TRAFFIC_BYTES.get(f"{op}_b{b}"),
            "input_gbs": round(n * (1 if op == "dequantize" else es) / avg / 1e6, 1),
            "total_gbs": round(ab / avg / 1e6, 1),
            "frac_of_measured": round(ab / avg / 1e6 / peak, 4),
            "frac_of_nominal_8tbs": round(ab / avg / 1e6 / NOMINAL_HBM_GBS, 4),
        }
    totals = {k: v["ms"] for k, v in kernels.items()}
    dominant = max(totals, key=totals.get)
    dop, db = dominant.split("_b")
    dab = algorithmic_bytes(dop, n, int(db), es, es)
    achieved = dab / kernels[dominant]["ms"] / 1e6
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": round(achieved, 1), "peak": peak, "peak_kind": peak_kind,
                "unit": "GB/s", "frac": round(achieved / peak, 4), "traffic": TRAFFIC_BYTES.get(dominant) if WORKLOAD == "sweep1g" else None}
    if rank == 0:
        progress("kernels", {"value_gbs": round(value, 1), "ms_per_step": round(max_s * 1e3 / args.steps, 4), "roofline": roofline,
                             "kernels": kernels, "input_sha256": input_sha})

    # end to end: host buffers in, host buffers out, copies inside the timed region
    e2e = guarded("e2e", lambda: run_e2e(bq, cb, x_pin, dev, w.dtype, n, args, world))
    if rank == 0:
        progress("e2e", e2e)
    full = WORKLOAD == "sweep1g"                     # the variants and the other configurations ride on the headline run only

    # compression and reconstruction error (block 4096 outputs are still resident: recompute per block cheaply)
    quality = {}
    for b in BLOCKS:
        bq.bq_roundtrip(x, b, cb, y_out=y)
        num = torch.zeros((), dtype=torch.float64, device=dev)
        den = torch.zeros((), dtype=torch.float64, device=dev)
        for s in range(0, n, 1 << 27):
            xs, ys = x[s:s + (1 << 27)].float(), y[s:s + (1 << 27)].float()
            num += ((xs - ys) ** 2).sum(dtype=torch.float64)
            den += (xs ** 2).sum(dtype=torch.float64)
        quality[f"b{b}"] = {"compression_ratio": round(es * b / (b + 4), 3), "rel_rms_error": round(float((num / den).sqrt().item()), 5)}
    if rank == 0:
        progress("quality", quality)

    bq4 = guarded("bq4", lambda: run_bq4(bq, dev, x, y, codes, absmax, n, w, peak)) if full else {}
    if rank == 0 and full:
        progress("bq4", bq4)
    cpu = guarded("cpu_baseline", lambda: cpu_baseline(x_pin, w, rank)) if (rank == 0 and world == 1 and not args.no_cpu_baseline) else None
    if cpu is not None:
        progress("cpu_baseline", cpu)
    if not full:
        return finish(rank, world, args, value, max_s, n, w, e2e, events, clocks, roofline, kernels, quality, cpu, input_sha,
                      None, None, None, None)

    tune = guarded("autotune", lambda: run_autotune(bq, dev, x, cb, n, w, peak))
    if rank == 0:
        progress("autotune", tune)

    del x, y, codes, absmax
    torch.cuda.empty_cache()
    small = guarded("small_configs", lambda: run_small(bq, dev)) if rank == 0 else None
    if rank == 0:
        progress("small_configs", small)
    mmd = guarded("mmd", lambda: run_mmd(bq, dev, args)) if (rank == 0 and not args.no_mmd) else None
    if mmd is not None:
        progress("mmd", mmd)
    transport = guarded("transport", lambda: run_transport(bq, dev, args)) if (rank == 0 and not args.no_transport) else None
    if transport is not None:
        progress("transport", transport)
    mtpp = guarded("mtpp", lambda: run_mtpp(bq, dev, args)) if (rank == 0 and not args.no_mtpp) else None
    if mtpp is not None:
        progress("mtpp", mtpp)
    return finish(rank, world, args, value, max_s, n, w, e2e, events, clocks, roofline, kernels, quality, cpu, input_sha,
                  bq4, tune, small, mmd, transport, mtpp)


def workload_label(w) -> str:
    """The line's `config.workload`, the same text for both arms."""
    blocks = "/".join(str(b) for b in w.blocks)
    return (f"{w.name}: {list(w.shape)} {str(w.dtype)[6:]}, {w.recipe}, seed {w.seed}; blocks {blocks}; "
            "quantize+dequantize+roundtrip per block")


def finish(rank, world, args, value, max_s, n, w, e2e, events, clocks, roofline, kernels, quality, cpu, input_sha, bq4, tune, small, mmd,
           transport=None, mtpp=None):
    if rank == 0:
        es = torch.empty(0, dtype=w.dtype).element_size()
        fits_l2 = 2 * n * es < (120 << 20)
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": round(max_s * 1e3 / args.steps, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_label(w), "elements": n,
                       "l2": ("tensor fits in L2: a 256 MiB buffer is written before every launch and the value counts the launches' own "
                              "event times" if fits_l2 else f"input ({n * es >> 20} MiB) larger than L2, no flush needed"),
                       "parallelism": f"replicated x{world}, no collective", "input_sha256": input_sha},
            "e2e": e2e, "gpu_launches": len(events), "clocks": clocks, "roofline": roofline, "kernels": kernels,
            "quality": quality, "cpu_baseline": cpu, "bq4": bq4, "autotune": tune, "small_configs": small, "mmd": mmd,
            "transport": transport, "mtpp": mtpp,
            "paper_context": "the paper reports no throughput for this path; it states only that hidden-state quantization halves the bandwidth",
        }
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def guarded(name: str, fn):
    """The sections beside the headline measurement must not take the line down with them: an exception in one of them is
    recorded under its key (and on stderr) and the run goes on."""
    try:
        return fn()
    except Exception as exc:                                   # noqa: BLE001 - whatever it is, the headline numbers are kept
        sys.stderr.write(f"bench.py: section {name} failed: {exc!r}\n")
        return {"error": repr(exc)}


def run_bq4(bq, dev, x, y, codes, absmax, n, w, peak):
    """The 4-bit variant of the same path (16-entry codebook, two codes per byte) on the same tensor."""
    cb4 = bq.Codebook4()
    bq4 = {}
    for b, s16 in ((64, False), (1024, False), (64, True)):       # s16: the block scale stored as a bf16 (2 bytes instead of 4)
        packed = codes[: n // 2]
        scale16 = absmax[b].view(torch.bfloat16)[: n // b]
        times = {}
        if s16:
            ops = (("quantize4", lambda: bq.bq4_quantize_s16(x, b, cb4, packed, scale16)),
                   ("dequantize4", lambda: bq.bq4_dequantize_s16(packed, scale16, n, b, cb4, w.dtype, y)))
        else:
            ops = (("quantize4", lambda: bq.bq4_quantize(x, b, cb4, packed, absmax[b])),
                   ("dequantize4", lambda: bq.bq4_dequantize(packed, absmax[b], n, b, cb4, w.dtype, y)))
        for op, fn in ops:
            for _ in range(3):
                fn()
            ev = []
            for _ in range(10):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); fn(); e1.record()
                ev.append((e0, e1))
            torch.cuda.synchronize()
            times[op] = float(np.mean([a.elapsed_time(b_) for a, b_ in ev]))
        scale_bytes = 2 if s16 else 4
        ab = n * 2 + n // 2 + scale_bytes * (n // b)
        num = torch.zeros((), dtype=torch.float64, device=dev)
        den = torch.zeros((), dtype=torch.float64, device=dev)
        for s in range(0, n, 1 << 27):
            xs, ys = x[s:s + (1 << 27)].float(), y[s:s + (1 << 27)].float()
            num += ((xs - ys) ** 2).sum(dtype=torch.float64)
            den += (xs ** 2).sum(dtype=torch.float64)
        bq4[f"b{b}" + ("_scale16" if s16 else "")] = {
            "quantize_ms": round(times["quantize4"], 4), "dequantize_ms": round(times["dequantize4"], 4), "algorithmic_bytes": int(ab),
            "quantize_frac_of_measured": round(ab / times["quantize4"] / 1e6 / peak, 4),
            "dequantize_frac_of_measured": round(ab / times["dequantize4"] / 1e6 / peak, 4),
            "compression_ratio": round(2.0 * n / (n / 2 + scale_bytes * (n // b)), 3),
            "rel_rms_error": round(float((num / den).sqrt().item()), 5), "gpu_launches": 26}
    return bq4


def run_autotune(bq, dev, x, cb, n, w, peak):
    """Block-size selection on the same tensor: the roundtrip and the error sums of four candidates in one call."""
    tune_blocks = [64, 256, 1024, 4096]
    tune_ws = torch.empty(bq.tune.workspace_bytes(w.dtype, n), dtype=torch.uint8, device=dev)
    tune_sums = torch.empty(len(tune_blocks) + 1, dtype=torch.float64, device=dev)
    for _ in range(2):
        bq.tune.block_errors(x, tune_blocks, cb, tune_ws, tune_sums)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        bq.tune.block_errors(x, tune_blocks, cb, tune_ws, tune_sums)
    e1.record()
    torch.cuda.synchronize()
    tune_ms = e0.elapsed_time(e1) / 5
    tune_bytes = len(tune_blocks) * 4 * n * 2                     # per candidate: roundtrip reads x and writes y, the sums read both
    sums_host = tune_sums.cpu().numpy()
    tune = {"blocks": tune_blocks, "ms_per_call": round(tune_ms, 4), "algorithmic_bytes": int(tune_bytes),
            "frac_of_measured": round(tune_bytes / tune_ms / 1e6 / peak, 4),
            "rel_rms_error": [round(float(v), 5) for v in np.sqrt(sums_host[:-1] / sums_host[-1])],
            "picked_for_rel_rms_0.01": bq.tune.pick_block(tune_blocks, sums_host, 0.01), "gpu_launches": 7 * 3 * len(tune_blocks)}
    return tune


# ------------------------------------------------------------------------------------------ the small configurations

def run_small(bq, dev):
    """GPU time per call of the three operations on the four configurations beside the headline one, each with its own
    block size.  `warm_us` replays the call on the same buffers (for the three configurations that fit in L2 the tensors
    stay there: the launch-bound figure); for those, the roundtrip also gets `cold_us`: a 256 MiB buffer is written before
    every call (the tensor then comes from DRAM, and the call also pays for the flush buffer's dirty lines it displaces) and
    the time of the writes alone is subtracted.  CUDA-graph replays, so no host launch gap is in any figure."""
    cb = bq.Codebook(device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    side = torch.cuda.Stream()

    def replay_time(fns, reps=20):
        with torch.cuda.stream(side):
            for f in fns:
                f()
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for f in fns:
                    f()
            graph.replay()
            side.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(side)
            for _ in range(reps):
                graph.replay()
            e1.record(side)
            side.synchronize()
        return e0.elapsed_time(e1) / reps

    out = {}
    inner = 8
    peak, _ = measured_peak()
    t_flush = replay_time([lambda: flush.fill_(1)] * inner) / inner
    for name in ("tiny", "decode70b", "prefill7b", "moe_prefill"):
        w = workloads.WORKLOADS[name]
        x = workloads.make(name).reshape(-1).to(dev)
        n = x.numel()
        y = torch.empty_like(x)
        b = w.blocks[0]
        codes = torch.empty(n, dtype=torch.uint8, device=dev)
        absmax = torch.empty(n // b, dtype=torch.float32, device=dev)
        calls = {"quantize": lambda: bq.bq_quantize(x, b, cb, codes, absmax),
                 "dequantize": lambda: bq.bq_dequantize(codes, absmax, b, cb, x.dtype, y),
                 "roundtrip": lambda: bq.bq_roundtrip(x, b, cb, y_out=y)}
        es = x.element_size()
        nbytes = {"quantize": n * es + n + 4 * (n // b), "dequantize": n + 4 * (n // b) + n * es, "roundtrip": 2 * n * es}
        entry = {"shape": list(w.shape), "dtype": str(x.dtype)[6:], "block": b, "fits_l2": bool(2 * n * es < (100 << 20))}
        launches = 0
        for op, call in calls.items():
            warm = replay_time([call] * inner) / inner
            launches += inner * 22
            entry[op] = {"warm_us": round(warm * 1e3, 2), "algorithmic_bytes": int(nbytes[op]), "gbs": round(nbytes[op] / warm / 1e6, 1),
                         "frac_of_measured": round(nbytes[op] / warm / 1e6 / peak, 4)}
            if entry["fits_l2"] and op == "roundtrip":
                both = []
                for _ in range(inner):
                    both += [lambda: flush.fill_(1), call]
                cold = replay_time(both) / inner - t_flush
                launches += inner * 22
                entry[op]["cold_us"] = round(cold * 1e3, 2)
        entry["gpu_launches"] = launches
        out[name] = entry
        del x, y, codes, absmax
    return out


# ------------------------------------------------------------------------------------------ slicing topological orders

def run_mtpp(bq, dev, args, name="mtpp_unet"):
    """The paper's other fully stated algorithm (its Algorithm 1), batched over a population of orders: priority
    vectors are decoded into topological orders and every order is cut into at most k blocks of least bottleneck
    cost.  One CTA per order; integer arithmetic; no HBM traffic to speak of (the graph and a row of n node
    numbers per order), so the figure is orders per second and the time per order, beside the oracle's time
    on a sample of orders.  Its results are compared with the oracle by tests/test_gpu_mtpp.py."""
    import oracle.mtpp_oracle as mo
    w = workloads.GRAPH_WORKLOADS[name]
    n, edges, work, sizeparam, sizeout = workloads.make_graph(name)
    dg = bq.mtpp.SliceGraph(n, edges, work, sizeparam, sizeout, device=dev)
    keys_host = workloads.make_keys(name)
    keys = keys_host.to(dev)
    P = keys.shape[0]
    orders = torch.empty((P, n), dtype=torch.int32, device=dev)
    out = dg.slice_orders(dg.decode_orders(keys, orders), w.k, w.B, w.M)
    torch.cuda.synchronize()
    reps = max(3, min(args.steps, 20))

    def timed(fn):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    ms_decode = timed(lambda: dg.decode_orders(keys, orders))
    ms_slice = timed(lambda: dg.slice_orders(orders, w.k, w.B, w.M, out))
    cost = out[0].cpu().numpy()
    # the oracle on two orders of the same population (decode + slice), one thread
    g = mo.Graph(n, [tuple(e) for e in edges.tolist()], work.tolist(), sizeparam.tolist(), sizeout.tolist())
    t = time.perf_counter()
    sample = 2
    for p in range(sample):
        mo.slice_order(g, mo.decode_order(g, keys_host[p].tolist()), w.k, w.B, w.M)
    cpu_s = (time.perf_counter() - t) / sample
    dg.close()
    # What bounds the slicing kernel is integer arithmetic.  Algorithmic operations of one order: every candidate cut of the
    # dynamic programme is one max and one compare (rows 2..k, right ends r, cuts l = row - 1 .. r - 1); every column entry
    # (l, r) takes 4 running updates, 7 operations to put the cost together and 2 compares + 2 conditional adds per producer
    # edge of the node at r.  Peak: one 16-lane integer pipe per scheduler, 4 schedulers per SM, at the top SM clock.
    rr = np.arange(1, n + 1, dtype=np.int64)
    kmax = min(w.k, n)
    dp_ops = 2 * sum(int(np.maximum(rr - kk + 1, 0).sum()) for kk in range(2, kmax + 1))
    col_ops = 11 * int(rr.sum()) + 4 * edges.shape[0] * (n + 1) // 2          # an edge's consumer sits at position (n + 1) / 2 on average
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    alu_peak = sm_count * 4 * 16 * 1.965e9
    alu_achieved = P * (dp_ops + col_ops) / (ms_slice * 1e-3)
    return {"workload": f"{name}: {w.recipe}; n = {n} nodes, {edges.shape[0]} edges, at most k = {w.k} blocks, population {P}",
            "roofline": {"bound": "alu", "kernel": "slice_orders", "achieved": round(alu_achieved / 1e12, 3), "peak": round(alu_peak / 1e12, 2),
                         "peak_kind": "derived: SMs x 4 schedulers x 16 integer lanes x 1965 MHz", "unit": "Tint-op/s", "frac": round(alu_achieved / alu_peak, 4),
                         "algorithmic_ops_per_order": dp_ops + col_ops, "traffic": None},
            "decode_ms": round(ms_decode, 4), "slice_ms": round(ms_slice, 4), "orders_per_s": round(P / (ms_decode + ms_slice) * 1e3, 1),
            "us_per_order": round((ms_decode + ms_slice) * 1e3 / P, 3), "best_bottleneck": int(cost.min()), "worst_bottleneck": int(cost.max()),
            "cpu_baseline": {"value": round(1.0 / cpu_s, 3), "unit": "orders/s", "cores": 1, "kind": "oracle", "sample": f"{sample} orders of the population, decode + slice"},
            "gpu_launches": 2 * (reps + 2) + 2}


# ------------------------------------------------------------------------------------------ the boundary transport (loop-back)

NVLINK_PEER_GBS = 770.0          # a measured NVLink 5 peer copy rate per direction between two B200s (context for the projection only)


def run_transport(bq, dev, args, block=256):
    """The hand-off across a shard boundary on ONE device (sender and receiver both here: loop-back):
    the sending side's quantize kernel fills a mailbox piece by piece, the receiving side's dequantize kernel
    drains it on a second stream.  Timed against handing over the raw 16-bit tensor the same way (a device
    copy per piece) and against the fused roundtrip kernel.  No link is crossed here, so the figures are the
    cost of the pipeline itself; what NVLink would add is printed as a projection from the bytes, and labelled so."""
    from paper_2407_19775_b200 import transport
    x = workloads.make(WORKLOAD).view(-1).to(dev)
    n = x.numel()
    es = x.element_size()
    y = torch.empty_like(x)
    cb = bq.Codebook(device=dev)
    chunk, slots = 1 << 25, 3
    rx = transport.Receiver(cb, chunk, min_block=block, slots=slots)
    s_send, s_recv = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    reps = max(3, min(args.steps, 20))

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s_send.wait_stream(torch.cuda.current_stream(dev))
        s_recv.wait_stream(torch.cuda.current_stream(dev))
        t0.record(s_send)
        s_recv.wait_event(t0)
        for _ in range(reps):
            fn()
        s_recv.wait_stream(s_send)
        t1.record(s_recv)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / reps

    out = {"workload": f"{WORKLOAD}, block {block}", "link": "loop-back on one device (sender and receiver are the same GPU); NVLink unmeasured on hardware",
           "pieces": len(transport.plan(n, block, chunk, slots)), "chunk_elems": chunk, "slots": slots,
           "payload_bytes": transport.payload_bytes(n, block), "raw_bytes": n * es,
           "bytes_ratio": round(n * es / transport.payload_bytes(n, block), 3)}
    for name, mode in (("store", transport.STORE), ("copy", transport.COPY)):
        tx = transport.Sender(cb, rx.export(), mode)
        ms = timed(lambda: transport.transfer(tx, rx, x, block, y, s_send, s_recv))
        out[name] = {"ms": round(ms, 4), "activation_gbs": round(n * es / ms / 1e6, 1)}
        tx.close()
    ref = bq.bq_roundtrip(x, block, cb)
    torch.cuda.synchronize()
    out["bit_identical_to_roundtrip"] = bool(torch.equal(ref.view(torch.int16), y.view(torch.int16)))
    pieces = [(lo, min(n, lo + chunk)) for lo in range(0, n, chunk)]

    def raw():
        for lo, hi in pieces:                                   # the uncompressed hand-off: one device copy per piece, then nothing to expand
            with torch.cuda.stream(s_send):
                y[lo:hi].copy_(x[lo:hi], non_blocking=True)

    out["raw_copy"] = {"ms": round(timed(raw), 4)}
    with torch.cuda.stream(s_send):
        out["fused_roundtrip"] = {"ms": round(timed(lambda: bq.bq_roundtrip(x, block, cb, y_out=y)), 4)}
    out["nvlink_projection"] = {"assumed_gbs": NVLINK_PEER_GBS, "payload_ms": round(out["payload_bytes"] / NVLINK_PEER_GBS / 1e6, 4),
                                "raw_ms": round(n * es / NVLINK_PEER_GBS / 1e6, 4),
                                "note": "bytes over an assumed link rate, not a measurement: the stores of the quantize kernel would be link-bound"}
    out["gpu_launches"] = 2 * (reps + 3) * (2 * out["pieces"]) + (reps + 3)
    rx.close()
    return out


# ------------------------------------------------------------------------------------------ the decomposed linear layer

MMD_WORKLOAD = "mmd_prefill_moe"
NOMINAL_INT8_OVER_BF16 = 2.0          # dense int8 (4.5 POP/s) over dense bf16 (2.25 PFLOP/s)
FALLBACK_BF16_TFLOPS = 1590.0
# dram__bytes_read.sum + dram__bytes_write.sum of one full-size launch of the product kernel (a one-pass ncu capture of
# the full layer: 130.28 MB read for 128.5 MB of codes, side columns and scales; 104.04 MB written, the rest of the 134.2 MB
# of Y still being dirty lines in L2 when the kernel ends).  Set to None when the kernel changes until it is re-measured.
MMD_TRAFFIC_BYTES = 234320000


def measured_tensor_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        return FALLBACK_BF16_TFLOPS, "fallback"


def run_mmd(bq, dev, args):
    """The paper's second compression technique on one layer of the MoE-class prefill shape:
    weights decomposed once, then timed calls of the layer (row kernel over the activations +
    tensor-core product).  Reported beside the main metric with its own roofline: operations
    2 M N K per call over the product kernel's time (the call's GPU time minus the row kernel's,
    both taken from CUDA-graph replays so that no host launch gap is counted)."""
    import oracle.mmd_oracle as mo
    wl = workloads.LINEAR_WORKLOADS[MMD_WORKLOAD]
    X, W, idx = workloads.make_linear(MMD_WORKLOAD)
    M, K, N = X.shape[0], X.shape[1], W.shape[0]
    x_pin, Xd, Wd = X.pin_memory(), X.to(dev), W.to(dev)
    lin = bq.DecomposedLinear(Wd, idx)
    y = torch.empty((M, N), dtype=wl.dtype, device=dev)
    ws = lin.workspace(M)
    idx_d = torch.from_numpy(idx).to(dev)
    reps = max(3, min(args.steps, 50))

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ev = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            ev.append((e0, e1))
        torch.cuda.synchronize()
        return float(np.mean([a.elapsed_time(b) for a, b in ev]))

    def timed_gpu(fn, inner):
        """GPU time per call with no host launch gaps: `inner` calls captured in a CUDA graph, replayed `reps` times
        (a call of a few tens of microseconds is otherwise timed by the host's launch rate, not by the GPU)."""
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            fn()
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for _ in range(inner):
                    fn()
            graph.replay()
            side.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(side)
            for _ in range(reps):
                graph.replay()
            e1.record(side)
            side.synchronize()
        return e0.elapsed_time(e1) / (reps * inner)

    qx, sx, sd = lin.workspace_parts(M, ws)
    lin.linear(Xd, y_out=y, workspace=ws)                    # first call outside any capture (one-time set-up of the kernels)
    bq.mmd.rowquant_into(Xd, idx_d, qx, sx, sd)
    torch.cuda.synchronize()
    ms_call = timed_gpu(lambda: lin.linear(Xd, y_out=y, workspace=ws), 2)
    status = lin.kernel_status()
    ms_row = timed_gpu(lambda: bq.mmd.rowquant_into(Xd, idx_d, qx, sx, sd), 8)
    ms_prod = ms_call - ms_row
    ops = 2.0 * M * N * K
    bf16, kind = measured_tensor_peak()
    peak = bf16 * NOMINAL_INT8_OVER_BF16
    hbm, _ = measured_peak()
    row_bytes = M * K * 3 + M * 4 + M * sd.shape[1] * 2

    # end to end: activations from pinned host memory, the result back to pinned host memory
    y_pin = torch.empty((M, N), dtype=wl.dtype).pin_memory()
    x_dev = torch.empty_like(Xd)

    def e2e_call():
        x_dev.copy_(x_pin, non_blocking=True)
        lin.linear(x_dev, y_out=y, workspace=ws)
        y_pin.copy_(y, non_blocking=True)

    ms_e2e = timed(e2e_call)

    # reconstruction error of the decomposed weights (first 1024 rows), from the handle's own parts on the device
    q_dev, s_dev, side_dev, idx_dev = lin.view()
    rec = q_dev[:1024].float() * s_dev[:1024, None]
    rec[:, idx_dev.long()] = side_dev[:1024, :idx.size].float()
    wf = Wd[:1024].float()
    w_err = float((((rec - wf) ** 2).sum(dtype=torch.float64) / (wf ** 2).sum(dtype=torch.float64)).sqrt().item())

    # CPU baseline: the oracle on a bounded sample of the same layer (it decomposes the weights first, as the GPU did; that
    # step is not timed on either side)
    qw, sw, wo = mo.rowquant(workloads.bits_2d(W), mo.BF16, idx)
    t = time.perf_counter()
    mo.linear(workloads.bits_2d(X[:256]), mo.BF16, qw, sw, wo, idx, mo.BF16)
    cpu_s = time.perf_counter() - t
    lin.close()

    # a decode step through a 70B-class layer: 64 tokens, every weight read once (HBM-bound).  The codes of one layer (67 MB)
    # would stay in the 126 MB L2 from call to call, so the timed graph cycles through four copies of the layer (268 MB):
    # every call streams its weights from DRAM, as consecutive layers of a model do.
    def decode_entry(out_features, copies):
        dX, dW, didx = workloads.make_linear("mmd_decode70b")
        dXd = dX.to(dev)
        dWd = dW.to(dev)
        if out_features is not None:                             # a wider layer: the workload's rows repeated (timing only)
            dWd = dWd.repeat((out_features + dWd.shape[0] - 1) // dWd.shape[0], 1)[:out_features].contiguous()
        dM, dK, dN = dX.shape[0], dX.shape[1], dWd.shape[0]
        dlins = [bq.DecomposedLinear(dWd, didx) for _ in range(copies)]
        del dWd
        dy = torch.empty((dM, dN), dtype=dX.dtype, device=dev)
        dws = dlins[0].workspace(dM)
        for dl in dlins:
            dl.linear(dXd, y_out=dy, workspace=dws)
        torch.cuda.synchronize()
        turn = [0]

        def decode_call():
            dlins[turn[0] % copies].linear(dXd, y_out=dy, workspace=dws)
            turn[0] += 1

        ms_dec = timed_gpu(decode_call, 2 * copies)
        dstatus = max(dl.kernel_status() for dl in dlins)
        dec_bytes = dN * dK + dM * dK * 3 + dM * dN * 2
        entry = {"workload": f"mmd_decode70b{'' if out_features is None else ' (weight rows repeated)'}: X [{dM},{dK}] x W [{dN},{dK}]^T fp16, {didx.size} critical features; "
                             f"{copies} copies of the layer in turn ({copies * dN * dK >> 20} MiB of codes, larger than L2)",
                 "us_per_call": round(ms_dec * 1e3, 2),
                 "algorithmic_bytes": int(dec_bytes), "gbs": round(dec_bytes / ms_dec / 1e6, 1),
                 "frac_of_measured_hbm": round(dec_bytes / ms_dec / 1e6 / hbm, 4), "kernel_status": dstatus}
        for dl in dlins:
            dl.close()
        return entry

    decode = decode_entry(None, DECODE_LAYER_COPIES)            # the 8192 -> 8192 projection
    decode_wide = decode_entry(28672, 2)                        # the 8192 -> 28672 projection: more tiles than SMs
    return {
        "workload": f"{MMD_WORKLOAD}: X [{M},{K}] x W [{N},{K}]^T bf16, {idx.size} critical features; {wl.recipe}",
        "ms_per_call": round(ms_call, 4), "tops": round(ops / ms_call / 1e9, 1), "kernel_status": status,
        "rowquant": {"ms": round(ms_row, 4), "algorithmic_bytes": int(row_bytes), "gbs": round(row_bytes / ms_row / 1e6, 1),
                     "frac_of_measured_hbm": round(row_bytes / ms_row / 1e6 / hbm, 4)},
        # the whole call as timed (row kernel + product kernel) over the tensor peak; the product kernel alone is an estimate
        # (call minus row kernel: an upper estimate, because part of the row kernel hides under the product kernel's set-up)
        "roofline": {"bound": "tensor", "kernel": "whole mmd_linear call: rowquant + gemm_tc2 (persistent CTA pairs, int8 tcgen05 cta_group::2)",
                     "achieved": round(ops / ms_call / 1e9, 1), "peak": round(peak, 1),
                     "peak_kind": f"{kind} bf16 x {NOMINAL_INT8_OVER_BF16} (nominal int8 / bf16 ratio)", "unit": "TOP/s",
                     "frac": round(ops / ms_call / 1e9 / peak, 4), "ms": round(ms_call, 4), "traffic": MMD_TRAFFIC_BYTES,
                     "product_kernel_estimate": {"ms": round(ms_prod, 4), "achieved": round(ops / ms_prod / 1e9, 1),
                                                 "frac": round(ops / ms_prod / 1e9 / peak, 4), "how": "call minus row kernel (upper estimate)"}},
        "e2e": {"ms_per_call": round(ms_e2e, 4), "tops": round(ops / ms_e2e / 1e9, 1), "h2d_bytes_per_call": int(M * K * 2),
                "d2h_bytes_per_call": int(M * N * 2)},
        "quality": {"weight_bytes_ratio": round(2.0 * N * K / (N * K + 4 * N + 2 * N * sd.shape[1]), 3),
                    "weight_rel_rms_error": round(w_err, 5)},
        "cpu_baseline": {"value": round(2.0 * 256 * N * K / cpu_s / 1e12, 4), "unit": "TOP/s", "cores": os.cpu_count(), "kind": "oracle",
                         "sample": "first 256 tokens through the whole layer (weights already decomposed); numpy/BLAS threads"},
        "decode": decode, "decode_wide": decode_wide,
        "gpu_launches": (2 * 2 + 8 + 2 * 8 + 2 * 4) * reps + 2 * (reps + 3),
    }


DECODE_LAYER_COPIES = 4

# DRAM bytes per full-size launch (dram__bytes_read.sum + dram__bytes_write.sum): a one-pass ncu capture of the twelve full-size
# launches of a step on the current binary (profiles/bench_sweep1g_dram_traffic_full_size.md).  Reads equal the algorithmic input
# bytes to 0.03 %; writes fall short of the algorithmic output bytes by the dirty lines still in L2 when the kernel ends.  Set an
# entry to None when its kernel changes until it is re-measured.
TRAFFIC_BYTES = {
    "quantize_b64": 1587131136, "quantize_b256": 1562008064, "quantize_b1024": 1572190720, "quantize_b4096": 1575371008,
    "dequantize_b64": 1582662144, "dequantize_b256": 1557130496, "dequantize_b1024": 1551257856, "dequantize_b4096": 1549172224,
    "roundtrip_b64": 2094758144, "roundtrip_b256": 2093994240, "roundtrip_b1024": 2093844480, "roundtrip_b4096": 2094068992,
}


def run_e2e(bq, cb, x_pin, dev, dtype, n, args, world):
    """One end-to-end step per block size through the library's host-buffer calls (bq_quantize_host,
    bq_dequantize_host, bq_roundtrip_host), everything starting and ending in pinned host memory: sender
    (x up, quantize, codes+absmax down), receiver (codes+absmax up, dequantize, y down) and the fused loop
    (x up, roundtrip, y down).  The three legs of each call overlap piece by piece on the pipe's three streams;
    the timed region ends when the last byte is back in host memory."""
    from paper_2407_19775_b200.pipeline import HostBoundary
    steps = max(1, min(args.steps, args.e2e_steps))
    es = x_pin.element_size()
    chunk = min(1 << 25, max(max(BLOCKS), (n // max(BLOCKS)) * max(BLOCKS)))
    hb = HostBoundary(cb, dtype, chunk=chunk, slots=3, min_block=min(BLOCKS))
    c_pin = torch.empty(n, dtype=torch.uint8).pin_memory()
    y_pin = torch.empty(n, dtype=dtype).pin_memory()
    a_pin = {b: torch.empty((n + b - 1) // b, dtype=torch.float32).pin_memory() for b in BLOCKS}
    h2d = d2h = 0

    def one_step(count=False):
        nonlocal h2d, d2h
        for b in BLOCKS:
            hb.quantize(x_pin, b, c_pin, a_pin[b])
            hb.dequantize(c_pin, a_pin[b], b, y_pin)
            hb.roundtrip(x_pin, b, y_pin)
            if count:
                nb = (n + b - 1) // b
                h2d += 2 * n * es + n + 4 * nb
                d2h += n + 4 * nb + 2 * n * es

    one_step()
    hb.wait()
    torch.cuda.synchronize()
    barrier(world, dev)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(steps):
        one_step(count=(i == 0))
    hb.wait_on_current_stream()
    t1.record()
    torch.cuda.synchronize()
    barrier(world, dev)
    sec = max_over_ranks(t0.elapsed_time(t1) / 1e3, world, dev)
    hb.close()
    bytes_per_step = n * es * len(BLOCKS) * len(OPS)
    return {"value": round(whole_job_value(bytes_per_step * steps, world, sec) / 1e9, 2), "unit": "GB/s", "steps": steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "api": f"bq_quantize_host / bq_dequantize_host / bq_roundtrip_host (C ABI, host pointers; {chunk >> 20} Mi-element pieces, 3 slots, 3 streams)"}


# ------------------------------------------------------------------------------------------ the CPU oracle arm

def oracle_step(oracle, xb, odt, cb, threads):
    for b in BLOCKS:
        c, a = oracle.quantize_sharded(xb, odt, b, cb, threads)
        oracle.dequantize_sharded(c, a, b, cb, odt, threads)
        oracle.roundtrip_sharded(xb, odt, b, cb, odt, threads)


def cpu_baseline(x_pin, w, rank, elems=1 << 24):
    """The CPU oracle, as it stands, on a bounded sample (the first 16 Mi elements, or the whole tensor when it
    is smaller) of the same tensor, one thread, every block size of the workload x 3 operations."""
    import oracle
    odt = {torch.float32: oracle.F32, torch.float16: oracle.F16, torch.bfloat16: oracle.BF16}[w.dtype]
    xb = workloads.as_numpy_bits(x_pin[:elems]) if w.dtype != torch.float32 else x_pin[:elems].numpy()
    cb = oracle.make_codebook()
    oracle_step(oracle, xb[:8192 * 8], odt, cb, 1)        # touch the library once
    t = time.perf_counter()
    oracle_step(oracle, xb, odt, cb, 1)
    sec = time.perf_counter() - t
    return {"value": round(xb.size * x_pin.element_size() * len(BLOCKS) * len(OPS) / sec / 1e9, 5), "unit": "GB/s", "cores": 1, "kind": "oracle",
            "host_cores_total": os.cpu_count(), "seconds": round(sec, 2),
            "sample": f"first {xb.size} elements of {w.name}, {len(BLOCKS)} block size(s) x 3 ops, single thread"}


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on all host cores, on a bounded sample (a prefix of whole rows) of the
    same workload per step, sized so that the run ends within about two minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    global WORKLOAD, BLOCKS
    WORKLOAD = args.config
    w = workloads.WORKLOADS[WORKLOAD]
    BLOCKS = tuple(w.blocks)
    odt = {torch.float32: oracle.F32, torch.float16: oracle.F16, torch.bfloat16: oracle.BF16}[w.dtype]
    threads = os.cpu_count() or 1
    hidden = w.shape[-1]
    total_rows = w.n // hidden
    # one element through one (block size x 3 operations) costs about 0.8 us of one core
    per_elem_s = 0.83e-6 * len(BLOCKS) / max(1, threads) * 1.5
    rows = int(120.0 / ((args.steps + args.warmup) * per_elem_s) // hidden)
    rows = max(1, min(rows, 4096, total_rows))
    x = workloads.make(WORKLOAD, rows=rows).reshape(-1)
    xb = workloads.as_numpy_bits(x) if w.dtype != torch.float32 else x.numpy()
    cb = oracle.make_codebook()
    for _ in range(args.warmup):
        oracle_step(oracle, xb, odt, cb, threads)
    t = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(oracle, xb, odt, cb, threads)
    sec = time.perf_counter() - t
    value = xb.size * x.element_size() * len(BLOCKS) * len(OPS) * args.steps / sec / 1e9
    sample = (f"first {rows} rows ({xb.size} elements) of {w.name} per step, {len(BLOCKS)} block size(s) x 3 ops, {threads} threads over whole blocks")
    line = {
        "impl": "reference", "metric": METRIC, "value": round(value, 5), "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(sec * 1e3 / args.steps, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_label(w), "sample": sample},
        "cpu_baseline": {"value": round(value, 5), "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 5), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-mmd", action="store_true", help="skip the decomposed-linear-layer section")
    ap.add_argument("--no-transport", action="store_true", help="skip the loop-back boundary-transport section")
    ap.add_argument("--no-mtpp", action="store_true", help="skip the order-slicing section")
    ap.add_argument("--config", default="sweep1g", choices=sorted(workloads.WORKLOADS),
                    help="the workload the step runs on (default: the largest, which the metric is quoted on); the 4-bit, block-selection, "
                         "small-configuration, linear-layer and transport sections ride on the default only")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
