"""Compile libskipffn.so in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libskipffn.so")
# the same library with per-role cycle counters in the tensor-core GEMM kernels (bench.py --role-cycles)
LIB_ROLE_CYCLES = os.path.join(HERE, "libskipffn_role_cycles.so")
SOURCES = ["api.cu", "compact.cu", "compact_static.cu", "kvcache.cu", "merge.cu", "prenorm.cu", "simt.cu", "summary.cu", "umma.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "skipffn.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def _compile(out: str, extra, verbose: bool) -> None:
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = out + f".{os.getpid()}.tmp"
    cmd = [nvcc] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + \
          ["-I", INCLUDE, "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, out)


def build(force: bool = False, verbose: bool = False) -> str:
    """Build the shared library if it is missing or older than its sources; returns its path."""
    if force or _stale():
        _compile(LIB, [], verbose)
    return LIB


def build_role_cycles() -> str:
    """Build the instrumented variant (per-role wait / busy cycle counters, -DSKIPFFN_ROLE_CYCLES)."""
    _compile(LIB_ROLE_CYCLES, ["-DSKIPFFN_ROLE_CYCLES"], False)
    return LIB_ROLE_CYCLES


if __name__ == "__main__":
    import sys
    if "--role-cycles" in sys.argv:
        print(build_role_cycles())
    else:
        print(build(force=True, verbose=True))
