"""Compile the C oracle into oracle/libapms_oracle.so (gcc, no CUDA)."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "apms_oracle.c")
LIB = os.path.join(HERE, "libapms_oracle.so")
FLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC", "-std=c99",
         "-Wall", "-Wextra"]


def build(force: bool = False, src: str = SRC, lib: str = LIB, extra=()) -> str:
    if (not force and os.path.exists(lib) and os.path.getmtime(lib) >= os.path.getmtime(src)):
        return lib
    tmp = lib + f".tmp{os.getpid()}"
    subprocess.check_call(["gcc", *FLAGS, *extra, src, "-o", tmp, "-lm"])
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True))
