"""Compile libssa.so (sm_100a) in-tree with nvcc.

    python -m paper_2404_09336_b200.build [-o OUT] [-DNAME=VALUE ...]
"""
from __future__ import annotations

import glob
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libssa.so")
PROBE_SRC = os.path.join(HERE, "probe", "gather_probe.cu")
PROBE_LIB = os.path.join(HERE, "libssa_probe.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared", "-Xptxas", "-v", "--threads", "0",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(out, deps):
    if not os.path.exists(out):
        return True
    t = os.path.getmtime(out)
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, defines=(), out: str = LIB, verbose: bool = False) -> str:
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(ROOT, "include", "ssa.h")]
    if not force and not defines and not _stale(out, deps):
        return out
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        raise RuntimeError("nvcc not found: libssa.so cannot be built")
    tmp = out + f".tmp{os.getpid()}"
    cmd = [nvcc, *NVCC_FLAGS, *defines, "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", tmp, *sources()]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    os.replace(tmp, out)
    if verbose:
        print(res.stderr)
    return out


def build_probe(force: bool = False) -> str:
    """The gather micro-benchmark (bench.py --probe gather): a library of its own, not part of libssa."""
    if not force and not _stale(PROBE_LIB, [PROBE_SRC]):
        return PROBE_LIB
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        raise RuntimeError("nvcc not found: libssa_probe.so cannot be built")
    tmp = PROBE_LIB + f".tmp{os.getpid()}"
    res = subprocess.run([nvcc, *NVCC_FLAGS, "-o", tmp, PROBE_SRC], capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    os.replace(tmp, PROBE_LIB)
    return PROBE_LIB


if __name__ == "__main__":
    args = sys.argv[1:]
    out = args[args.index("-o") + 1] if "-o" in args else LIB
    build_library(force=True, defines=[a for a in args if a.startswith("-D")], out=out, verbose=True)
    if "-o" not in args:
        build_probe(force=True)
