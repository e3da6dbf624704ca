"""Builds ``libbq.so`` (the CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2407_19775_b200.build [--force] [--verbose] [--debug]

Each translation unit is compiled on its own (in parallel) and the objects are linked into
``paper_2407_19775_b200/libbq.so``.  nvcc cross-compiles, so no GPU is needed to build.

``--debug`` also links ``libbq_debug.so``: the units that use the host-side assertions of
``csrc/bq_debug.h`` compiled with ``-DBQ_DEBUG``, the kernels as in the release build.  Load it
with ``BQ_LIB=.../libbq_debug.so``.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libbq.so")
OBJ_DEBUG = os.path.join(HERE, "_build_debug")
LIB_DEBUG = os.path.join(HERE, "libbq_debug.so")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")

NVCC_FLAGS = [
    "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "--fmad=false", "-Xcompiler", "-fPIC", "-Xptxas", "-v", "-I", INCLUDE,
]


def _sources():
    return sorted(f for f in os.listdir(CSRC) if f.endswith(".cu"))


def _newest_header() -> float:
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    deps += [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE) if f.endswith(".h")]
    return max(os.path.getmtime(p) for p in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    hdr = _newest_header()
    jobs = []
    for src in _sources():
        s = os.path.join(CSRC, src)
        o = os.path.join(OBJ, src[:-3] + ".o")
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr):
            jobs.append((s, o))

    def compile_one(job):
        s, o = job
        r = subprocess.run(["nvcc", *NVCC_FLAGS, "-c", s, "-o", o], capture_output=True, text=True)
        with open(o[:-2] + ".log", "w") as f:
            f.write(r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {s}:\n{r.stdout}\n{r.stderr}")
        if verbose:
            sys.stderr.write(r.stderr)
        return o

    if jobs:
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4)) as ex:
            list(ex.map(compile_one, jobs))
    objs = [os.path.join(OBJ, src[:-3] + ".o") for src in _sources()]
    stale = not os.path.exists(LIB) or any(os.path.getmtime(o) > os.path.getmtime(LIB) for o in objs)
    if jobs or force or stale:
        tmp = LIB + f".tmp{os.getpid()}"
        r = subprocess.run(["nvcc", "-shared", "-o", tmp, *objs, "-gencode", "arch=compute_100a,code=sm_100a"],
                           capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
        os.replace(tmp, LIB)
    return LIB


def build_debug(force: bool = False) -> str:
    """libbq_debug.so: the release objects, except that the units with assertions are compiled with -DBQ_DEBUG."""
    build(force=force)
    os.makedirs(OBJ_DEBUG, exist_ok=True)
    hdr = _newest_header()
    objs = []
    for src in _sources():
        s = os.path.join(CSRC, src)
        with open(s) as f:
            asserting = "bq_debug.h" in f.read()
        if not asserting:
            objs.append(os.path.join(OBJ, src[:-3] + ".o"))
            continue
        o = os.path.join(OBJ_DEBUG, src[:-3] + ".o")
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr):
            r = subprocess.run(["nvcc", *NVCC_FLAGS, "-DBQ_DEBUG", "-c", s, "-o", o], capture_output=True, text=True)
            if r.returncode != 0:
                raise RuntimeError(f"nvcc failed on {s}:\n{r.stdout}\n{r.stderr}")
        objs.append(o)
    if force or not os.path.exists(LIB_DEBUG) or any(os.path.getmtime(o) > os.path.getmtime(LIB_DEBUG) for o in objs):
        tmp = LIB_DEBUG + f".tmp{os.getpid()}"
        r = subprocess.run(["nvcc", "-shared", "-o", tmp, *objs, "-gencode", "arch=compute_100a,code=sm_100a"], capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
        os.replace(tmp, LIB_DEBUG)
    return LIB_DEBUG


if __name__ == "__main__":
    if "--debug" in sys.argv:
        print(build_debug(force="--force" in sys.argv))
    else:
        print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
