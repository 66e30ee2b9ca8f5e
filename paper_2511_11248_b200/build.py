"""Build step: compile the CUDA sources into libtman.so next to this file (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libtman.so")
LIB_STAMPS = os.path.join(HERE, "libtman_stamps.so")   # the same library with role time stamps in the prefill kernel
SOURCES = ["api.cu", "pack.cu", "mpgemv.cu", "mpgemv_static.cu", "mpgemm.cu", "mpgemm_i8.cu", "microbench.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "--shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "tman.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, stamps: bool = False) -> str:
    """stamps: build libtman_stamps.so (-DTMAN_ROLE_STAMPS) instead of libtman.so."""
    lib = LIB_STAMPS if stamps else LIB
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + NVCC_FLAGS + (["-DTMAN_ROLE_STAMPS"] if stamps else []) + (["-Xptxas", "-v"] if verbose else []) + \
          [os.path.join(CSRC, s) for s in SOURCES] + ["-o", lib]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed")
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, stamps="--stamps" in sys.argv))
