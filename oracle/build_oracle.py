"""Compile the plain-C oracle into a shared library next to its source (gcc, -O2, OpenMP)."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "tman_oracle.c")
LIB = os.path.join(HERE, "libtman_oracle.so")
SRC_INT = os.path.join(HERE, "tman_oracle_int.c")
LIB_INT = os.path.join(HERE, "libtman_oracle_int.so")


def _compile(src: str, lib: str, force: bool) -> str:
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= os.path.getmtime(src):
        return lib
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-shared", "-fPIC", "-o", lib, src, "-lm"]
    subprocess.run(cmd, check=True)
    return lib


def build(force: bool = False) -> str:
    """The fp oracle (per-block weights, fp16 activations)."""
    return _compile(SRC, LIB, force)


def build_int(force: bool = False) -> str:
    """The integer oracle (per-tensor ternary weights, integer activations)."""
    return _compile(SRC_INT, LIB_INT, force)


if __name__ == "__main__":
    print(build(force=True))
    print(build_int(force=True))
