"""Builds libbwla.so (the CUDA library behind the C ABI) for sm_100a with nvcc, in-tree.

Usage: ``python -m paper_2605_00422_b200.build [--force] [--verbose]``.
nvcc cross-compiles without a GPU.  The shared object lands beside this file.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libbwla.so")
INCLUDE = os.path.join(_ROOT, "include")

NVCC_FLAGS = ["-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
              "-Xcompiler", "-fPIC", "-shared", "--use_fast_math=false"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")]
    if verbose:
        flags += ["-Xptxas", "-v"]
    cmd = [nvcc] + flags + ["-I", INCLUDE, "-I", CSRC, "-o", LIB] + sources() + ["-lcudart"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libbwla.so")
    return LIB


def build_microbench() -> str:
    """The instruction-rate probes (stand-alone programs; not part of the library)."""
    nvcc = os.environ.get("NVCC", "nvcc")
    outs = []
    for name in ("issue_rates", "umma_rates"):
        src = os.path.join(_HERE, "microbench", name + ".cu")
        out = os.path.join(_HERE, "microbench", name)
        res = subprocess.run([nvcc, "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a", "-I", INCLUDE,
                              "-I", CSRC, "-o", out, src], capture_output=True, text=True)
        if res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
            raise RuntimeError("nvcc failed building the microbenchmark " + name)
        outs.append(out)
    return " ".join(outs)


if __name__ == "__main__":
    if "--microbench" in sys.argv:
        print(build_microbench())
    else:
        print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
