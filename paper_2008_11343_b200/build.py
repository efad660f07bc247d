"""Compile the CUDA library in-tree: paper_2008_11343_b200/libapms.so (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
SRC = os.path.join(CSRC, "apms.cu")                      # the one translation unit; it includes the .cuh files
HDR = os.path.join(ROOT, "include", "apms.h")
LIB = os.path.join(HERE, "libapms.so")
LIB_CHECKED = os.path.join(HERE, "libapms_checked.so")   # the same source with -DAPMS_BOUNDS_CHECK (debugging aid)
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-fmad=false", "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "-shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v",
    "-I", os.path.join(ROOT, "include"),
]


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    sources = [HDR] + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh"))]
    return os.path.getmtime(lib) < max(os.path.getmtime(f) for f in sources)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile libapms.so, or with checked=True libapms_checked.so (every kernel access validated on the device)."""
    lib = LIB_CHECKED if checked else LIB
    if not force and not is_stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + f".tmp{os.getpid()}"
    extra = ["-DAPMS_BOUNDS_CHECK"] if checked else []
    proc = subprocess.run([nvcc, *NVCC_FLAGS, *extra, SRC, "-o", tmp], capture_output=True, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
    if proc.returncode != 0:
        raise RuntimeError(f"nvcc failed building {os.path.basename(lib)}")
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose=True))
    if "--checked" in sys.argv:
        print(build(force=True, checked=True))
