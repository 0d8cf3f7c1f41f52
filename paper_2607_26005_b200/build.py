"""Build libpictura.so (CUDA, sm_100a) in-tree with nvcc.  No torch, no JIT cache."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpictura.so")
SOURCES = ["pic_api.cu", "pic_kernels.cu", "pic_render.cu", "pic_static.cu", "pic_probe.cu", "pic_bvh.cpp"]
HEADERS = ["pic_types.h", "pic_device.cuh", "pic_exhaustive.cuh", "pic_colour.cuh", "pic_coverage.cuh", os.path.join("..", "..", "include", "pictura.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if a source is newer than it.  Returns the path of the .so."""
    if not (force or _stale()):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
           "-Xcompiler", "-fPIC,-Wall", "-shared", "-cudart", "static", "-o", LIB]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, f) for f in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libpictura.so")
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
