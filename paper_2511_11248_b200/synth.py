"""Seeded synthetic inputs for the low-bit matmul path.

This module only draws random numbers and rounds them to their storage types.
It holds none of the method's arithmetic (no packing, no tables, no
dequantization), so both the CPU oracle's tests and the CUDA path's tests and
benchmark can be fed from it without sharing any computation.

Shapes and quantization format follow the layer shapes the paper evaluates
(Sec. "Evaluation Setup": per-block asymmetric GPTQ-style codes, scales and
zero-points; fp16 activations).  Values are random because trained weights are
not available offline.

Draw order per case (fixed, so a seed identifies a case):
codes -> zeros -> scales -> activations (-> outlier channels).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterator, List, Tuple

import numpy as np

SEED_BASE = 251111000


@dataclass
class Case:
    """One matmul problem: y[M,N] = x[M,K] . W[K,N], W given by (codes, scales, zeros)."""

    name: str
    M: int
    K: int
    N: int
    bits: int
    group: int
    seed: int
    codes: np.ndarray   # uint8 [K, N], values in [0, 2^bits)
    scales: np.ndarray  # float16 [K/group, N]
    zeros: np.ndarray   # uint8 [K/group, N], values in [0, 2^bits)
    x: np.ndarray       # float16 [M, K]


def make_case(name: str, M: int, K: int, N: int, bits: int, group: int, seed: int,
              scale_lo: float, scale_hi: float, outlier_frac: float = 0.0,
              outlier_mult: float = 20.0) -> Case:
    rng = np.random.Generator(np.random.PCG64(seed))
    levels = 1 << bits
    codes = rng.integers(0, levels, size=(K, N), dtype=np.uint8)
    zeros = rng.integers(0, levels, size=(K // group, N), dtype=np.uint8)
    scales = rng.uniform(scale_lo, scale_hi, size=(K // group, N)).astype(np.float16)
    x = rng.standard_normal(size=(M, K)).astype(np.float32)
    if outlier_frac > 0.0:
        n_out = max(1, int(round(outlier_frac * K)))
        chans = rng.choice(K, size=n_out, replace=False)
        x[:, chans] *= outlier_mult
    return Case(name, M, K, N, bits, group, seed, codes, scales, zeros, x.astype(np.float16))


def scale_range(bits: int) -> Tuple[float, float]:
    """Scale distribution used by the configs: wider steps for 2-bit codes."""
    return (0.01, 0.05) if bits == 2 else (0.005, 0.02)


# ---- the five workload families --------------------------------------------

LLAMA3_8B_PROJ: List[Tuple[str, int, int]] = [
    ("q", 4096, 4096), ("k", 4096, 1024), ("v", 4096, 1024), ("o", 4096, 4096),
    ("gate", 4096, 14336), ("up", 4096, 14336), ("down", 14336, 4096),
]
QWEN25_7B_PROJ: List[Tuple[str, int, int]] = [
    ("gateup", 3584, 18944), ("down", 18944, 3584), ("qkv", 3584, 4608),
]


def config1() -> Case:
    """Decode, M=1, 4096x4096, 4-bit, group 64."""
    return make_case("c1_m1_4096x4096_b4_g64", 1, 4096, 4096, 4, 64,
                     SEED_BASE + 100 * 1, 0.005, 0.02)


def config2_specs() -> List[Tuple[str, int, int, int, int, int, int]]:
    """Decode, M=1, 2-bit, Llama-3-8B MLP shapes: (name, M, K, N, bits, group, seed)."""
    out = []
    for i, (nm, K, N) in enumerate([("gate", 4096, 14336), ("up", 4096, 14336),
                                    ("down", 14336, 4096)]):
        out.append((f"c2_{nm}_m1_{K}x{N}_b2_g64", 1, K, N, 2, 64, SEED_BASE + 100 * 2 + i))
    return out


def config3_specs() -> List[Tuple[str, int, int, int, int, int, int]]:
    """Decode batch sweep: seven projections x bits {2,3,4} x M {1,2,4,8}, group 128."""
    out = []
    idx = 0
    for bits in (2, 3, 4):
        for M in (1, 2, 4, 8):
            for nm, K, N in LLAMA3_8B_PROJ:
                out.append((f"c3_{nm}_m{M}_{K}x{N}_b{bits}_g128", M, K, N, bits, 128,
                            SEED_BASE + 100 * 3 + idx))
                idx += 1
    return out


def config4_specs() -> List[Tuple[str, int, int, int, int, int, int]]:
    """Prefill, M=1024, K=4096, N in {4096, 14336}, 4-bit, group 128."""
    return [(f"c4_m1024_4096x{N}_b4_g128", 1024, 4096, N, 4, 128, SEED_BASE + 100 * 4 + i)
            for i, N in enumerate((4096, 14336))]


def config5_specs() -> List[Tuple[str, int, int, int, int, int, int]]:
    """Prefill sweep on Qwen2.5-7B shapes with 1% outlier channels (x20)."""
    out = []
    idx = 0
    for bits in (2, 4):
        for group in (64, 128):
            for M in (128, 512, 2048, 8192):
                for nm, K, N in QWEN25_7B_PROJ:
                    out.append((f"c5_{nm}_m{M}_{K}x{N}_b{bits}_g{group}", M, K, N, bits, group,
                                SEED_BASE + 100 * 5 + idx))
                    idx += 1
    return out


def case_from_spec(spec, outliers: bool = False) -> Case:
    name, M, K, N, bits, group, seed = spec
    lo, hi = scale_range(bits)
    if name.startswith("c1") or name.startswith("c3") or name.startswith("c4"):
        lo, hi = 0.005, 0.02
    return make_case(name, M, K, N, bits, group, seed, lo, hi,
                     outlier_frac=0.01 if outliers else 0.0)


def iter_config(cfg: int) -> Iterator[Case]:
    if cfg == 1:
        yield config1()
    elif cfg == 2:
        for s in config2_specs():
            yield case_from_spec(s)
    elif cfg == 3:
        for s in config3_specs():
            yield case_from_spec(s)
    elif cfg == 4:
        for s in config4_specs():
            yield case_from_spec(s)
    elif cfg == 5:
        for s in config5_specs():
            yield case_from_spec(s, outliers=True)
    else:
        raise ValueError(f"unknown config {cfg}")


def small_case(M: int, K: int, N: int, bits: int, group: int, seed: int = 7,
               outliers: bool = False) -> Case:
    """A reduced-size case with the same value distributions (for parity tests)."""
    lo, hi = scale_range(bits)
    return make_case(f"small_m{M}_{K}x{N}_b{bits}_g{group}", M, K, N, bits, group,
                     SEED_BASE + seed, lo, hi, outlier_frac=0.01 if outliers else 0.0)
