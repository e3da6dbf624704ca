"""The benchmark's multi-process plumbing on CPU (gloo, world size 2) and its byte counts."""
import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank_main(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import bench
    r, w = bench.dist_setup(world, "gloo")
    bench.barrier(w)
    slowest = bench.max_over_ranks(0.5 * (rank + 1), w)           # rank 1 is the slow one: 1.0 s
    value = bench.whole_job_value(100.0, w, slowest)               # every rank did 100 units
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"rank": r, "world": w, "slowest": slowest, "value": value}, f)
    import torch.distributed as dist
    dist.destroy_process_group()


def test_two_ranks_gloo(tmp_path):
    port = _free_port()
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for rank in (0, 1):
        d = json.load(open(tmp_path / f"r{rank}.json"))
        assert d == {"rank": rank, "world": 2, "slowest": 1.0, "value": 200.0}


def test_algorithmic_bytes():
    import bench
    n = 1 << 20
    assert bench.algorithmic_bytes("quantize", n, 64) == n * 2 + n + 4 * (n // 64)
    assert bench.algorithmic_bytes("dequantize", n, 4096) == n + 4 * (n // 4096) + 2 * n
    assert bench.algorithmic_bytes("roundtrip", n, 256) == 4 * n
    assert abs(bench.algorithmic_bytes("quantize", n, 64) / n - 3.0625) < 1e-12


def test_reference_arm_other_ranks_exit_quietly():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
