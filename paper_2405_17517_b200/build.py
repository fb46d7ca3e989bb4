"""Builds libwash.so (sm_100a only) in-tree with nvcc.

    python -m paper_2405_17517_b200.build [--force] [--verbose]

wash_inst.cu (the dense operators) is compiled once per population size listed in
csrc/wash_nlist.h (plus once for run-time N); the objects are compiled in parallel and
linked with the C ABI into paper_2405_17517_b200/libwash.so.
"""
from __future__ import annotations

import concurrent.futures as cf
import os
import re
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
BUILD = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libwash.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libwash.so cannot be built")


def population_sizes() -> list[int]:
    with open(os.path.join(CSRC, "wash_nlist.h")) as f:
        text = f.read()
    line = [ln for ln in text.splitlines() if ln.startswith("#define WASH_N_LIST")][0]
    return [int(x) for x in re.findall(r"X\((\d+)\)", line.split("WASH_N_LIST(X)")[1])]


def _sources_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "wash.h"), __file__]
    return max(os.path.getmtime(p) for p in paths)


def is_stale() -> bool:
    return (not os.path.exists(LIB)) or os.path.getmtime(LIB) < _sources_mtime()


def _compile(job):
    src, obj, defs, verbose = job
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + defs + ["-c", src, "-o", obj]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed: %s\n%s\n%s" % (" ".join(cmd), res.stdout, res.stderr))
    return obj, res.stderr


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    os.makedirs(BUILD, exist_ok=True)
    jobs = [(os.path.join(CSRC, "wash_api.cu"), os.path.join(BUILD, "wash_api.o"), [], verbose),
            (os.path.join(CSRC, "wash_dispatch.cu"), os.path.join(BUILD, "wash_dispatch.o"), [], verbose)]
    for name in ("wash_noalloc", "wash_shuffle", "wash_shuffle_loop", "wash_exchange"):
        jobs.append((os.path.join(CSRC, name + ".cu"), os.path.join(BUILD, name + ".o"), [], verbose))
    for n in [0] + population_sizes():
        jobs.append((os.path.join(CSRC, "wash_inst.cu"), os.path.join(BUILD, "wash_inst_n%d.o" % n), ["-DWASH_N=%d" % n], verbose))
    workers = max(1, min(len(jobs), os.cpu_count() or 1))
    objs = []
    with cf.ThreadPoolExecutor(workers) as pool:
        for obj, log in pool.map(_compile, jobs):
            objs.append(obj)
            if verbose and log:
                sys.stderr.write(log)
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = [_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed: %s\n%s" % (res.stdout, res.stderr))
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
