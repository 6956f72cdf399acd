"""Builds libmuse.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Usage: python -m paper_2509_10406_b200.build [--force] [--verbose] [--debug]

--debug builds libmuse_debug.so instead: the same sources with -DMUSE_DEBUG (every data-derived index
checked against its bound, violations recorded for muse_debug_report, nothing traps).
"""
from __future__ import annotations

import concurrent.futures
import hashlib
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(CSRC, "build")
LIB = os.path.join(HERE, "libmuse.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = (["-DMUSE_PHASE_CLOCKS"] if os.environ.get("MUSE_PHASE_CLOCKS") else []) + ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--expt-relaxed-constexpr"]


def _sources():
    return sorted(f for f in os.listdir(CSRC) if f.endswith(".cu"))


def _digest() -> str:
    h = hashlib.sha256(" ".join(FLAGS).encode())
    files = sorted(os.listdir(CSRC)) + [os.path.join("..", "..", "include", "muse.h")]
    for f in files:
        p = os.path.join(CSRC, f)
        if os.path.isfile(p) and f.endswith((".cu", ".cuh", ".h")):
            h.update(f.encode())
            h.update(open(p, "rb").read())
    return h.hexdigest()


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile every .cu under csrc/ and link libmuse.so (libmuse_debug.so with debug); no-op when sources are unchanged."""
    OBJ = os.path.join(CSRC, "build_debug" if debug else "build")
    LIB = os.path.join(HERE, "libmuse_debug.so" if debug else "libmuse.so")
    FLAGS = globals()["FLAGS"] + (["-DMUSE_DEBUG"] if debug else [])
    os.makedirs(OBJ, exist_ok=True)
    stamp = os.path.join(OBJ, "stamp")
    dig = _digest() + ("-debug" if debug else "")
    if not force and os.path.exists(LIB) and os.path.exists(stamp) and open(stamp).read() == dig:
        return LIB

    def cc(src):
        obj = os.path.join(OBJ, src[:-3] + ".o")
        cmd = [NVCC, *FLAGS, "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
        if verbose:
            sys.stderr.write(r.stderr)
        return obj

    with concurrent.futures.ThreadPoolExecutor(max_workers=os.cpu_count() or 4) as ex:
        objs = list(ex.map(cc, _sources()))
    r = subprocess.run([NVCC, "-shared", "-o", LIB, *objs, "-gencode", "arch=compute_100a,code=sm_100a"],
                       capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    open(stamp, "w").write(dig)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
