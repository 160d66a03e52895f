"""Builds libdte.so (the C-ABI CUDA library) and libdte_probes.so (measurement probes used by the
benchmark only) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB = os.path.join(_HERE, "libdte.so")
PROBES_LIB = os.path.join(_HERE, "libdte_probes.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    # bit-exactness: no FMA contraction, no flush-to-zero, IEEE division and square root
    "-fmad=false", "-ftz=false", "-prec-div=true", "-prec-sqrt=true",
    "-Xcompiler", "-fPIC,-fvisibility=hidden,-O2", "-shared",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def probe_sources():
    return sorted(glob.glob(os.path.join(CSRC, "probes", "*.cu")))


def _stale(lib, deps) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(d) > t for d in deps)


def _nvcc(out, srcs, verbose):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = out + f".tmp{os.getpid()}"
    cmd = [nvcc, *NVCC_FLAGS, "-I", INCLUDE, "-I", CSRC, "-o", tmp, *srcs]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
        print(" ".join(cmd))
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    if not force and not _stale(LIB, deps):
        return LIB
    return _nvcc(LIB, sources(), verbose)


def build_probes(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale(PROBES_LIB, probe_sources()):
        return PROBES_LIB
    return _nvcc(PROBES_LIB, probe_sources(), verbose)


if __name__ == "__main__":
    v = "-v" in sys.argv
    print(build(force=True, verbose=v))
    print(build_probes(force=True, verbose=v))
