"""Builds ``libasd.so`` (CUDA, sm_100a) in-tree next to this file."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libasd.so")
ROWS = list(range(1, 10)) + [16]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC,-fopenmp"]


def _sources():
    out = [os.path.join(CSRC, f) for f in sorted(os.listdir(CSRC))]
    out.append(os.path.join(os.path.dirname(HERE), "include", "asd.h"))
    return out


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(s) > t for s in _sources())


def _run(cmd):
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("command failed: %s\n%s\n%s" % (" ".join(cmd), r.stdout, r.stderr))
    return r.stdout + r.stderr


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every kernel for sm_100a and link the shared library. Returns its path."""
    if not force and not is_stale():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    nvcc = os.environ.get("NVCC", "nvcc")
    extra = ["-Xptxas", "-v"] if verbose else []
    jobs = []
    for m in ROWS:
        obj = os.path.join(OBJ, "inst_m%d.o" % m)
        jobs.append([nvcc, *NVCC_FLAGS, *extra, "-DASD_M=%d" % m, "-c", os.path.join(CSRC, "inst.cu"), "-o", obj])
    for name in sorted(os.listdir(CSRC)):
        if name.endswith(".cu") and name != "inst.cu":
            obj = os.path.join(OBJ, name[:-3] + ".o")
            jobs.append([nvcc, *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, name), "-o", obj])
    with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4)) as ex:
        logs = list(ex.map(_run, jobs))
    if verbose:
        sys.stderr.write("\n".join(logs))
    objs = [j[-1] for j in jobs]
    _run([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-Xcompiler", "-fopenmp", "-o", LIB, *objs])
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
