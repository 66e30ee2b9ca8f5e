"""B200-native table-lookup low-bit matmul (decode mpGEMV, prefill mpGEMM) behind a C ABI.

`binding` holds the ctypes wrappers (same names as include/tman.h); `synth` the seeded input
generators; `build` compiles the CUDA sources.  Nothing is loaded at import time.
"""
__all__ = ["binding", "synth", "build"]
