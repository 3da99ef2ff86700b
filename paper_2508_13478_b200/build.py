"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no torch extension).

Every source is compiled to an object file on its own, the sources side by side, then linked
into libdhq_b200.so next to this file.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
OBJ_DIR = os.path.join(_HERE, "_build")
LIB = os.path.join(_HERE, "libdhq_b200.so")
SOURCES = ["dhq_api.cu", "dhq_prepare.cu", "dhq_layerwise.cu", "dhq_fused.cu", "dhq_fused_w64.cu",
           "dhq_fused_w128.cu", "dhq_fused_w256.cu", "dhq_fused_w512.cu", "dhq_peaks.cu", "dhq_static.cu",
           "dhq_float.cu"]
ARCH_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a"]
NVCC_FLAGS = [*ARCH_FLAGS, "-lineinfo", "-O3", "-std=c++17", "--fmad=false",
              "-Xcompiler", "-fPIC,-fvisibility=hidden"]


def _newest_source() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    inc = os.path.join(os.path.dirname(_HERE), "include")
    paths += [os.path.join(inc, f) for f in os.listdir(inc)]
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, extra=()) -> str:
    """Compile csrc/*.cu into libdhq_b200.so next to this file; returns its path."""
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)

    def compile_one(src: str) -> str:
        obj = os.path.join(OBJ_DIR, os.path.splitext(src)[0] + ".o")
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", "-o", obj, os.path.join(CSRC, src)]
        if verbose:
            print(" ".join(cmd), file=sys.stderr)
        subprocess.run(cmd, check=True)
        return obj

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    link = [nvcc, *ARCH_FLAGS, "-shared", "-cudart", "shared", "-o", LIB, *objs]
    if verbose:
        print(" ".join(link), file=sys.stderr)
    subprocess.run(link, check=True)
    return LIB


if __name__ == "__main__":
    build(force=True, verbose=True, extra=tuple(sys.argv[1:]))
    print(LIB)
