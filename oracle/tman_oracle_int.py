"""NumPy-facing wrapper of the integer oracle (test infrastructure only): per-tensor ternary weights
with 16-bit (decode) or 8-bit (prefill) integer activations.  The arithmetic lives in
``tman_oracle_int.c``.  Passages followed: Sec. 6.1 (BitNet: per-tensor ternary weights treated as
2-bit, A_INT16), Sec. 2.2 and Fig. 2 (bit-serial table lookup), Sec. 4.3 (integer aggregation inside the
block, floating point after it), Sec. 4.1 / Fig. 7 and Sec. 6.2 (two-level lookup dequantization, to INT8
for per-tensor weights)."""
from __future__ import annotations

import ctypes as C

import numpy as np

from .build_oracle import build_int

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build_int())
    return _lib


def _p(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


def quantize_rows(x: np.ndarray, qmax: int):
    """Per-token symmetric quantization: (a int32 [M, K], s_a fp64 [M])."""
    assert x.dtype == np.float16
    M, K = x.shape
    a = np.empty((M, K), dtype=np.int32)
    s = np.empty(M, dtype=np.float64)
    lib().oracle_quantize_rows(_p(np.ascontiguousarray(x).view(np.uint16)), C.c_int(M), C.c_int(K), C.c_int(qmax),
                               _p(a), _p(s))
    return a, s


def ternary_matmul(a: np.ndarray, q: np.ndarray) -> np.ndarray:
    """The definition, int64 [M, N]: sum_k a[m][k] * (q[k][n] - 1)."""
    M, K = a.shape
    N = q.shape[1]
    acc = np.empty((M, N), dtype=np.int64)
    lib().oracle_ternary_matmul(_p(np.ascontiguousarray(a, dtype=np.int32)), _p(np.ascontiguousarray(q)),
                                C.c_int(M), C.c_int(K), C.c_int(N), _p(acc))
    return acc


def ternary_lut_matmul(a: np.ndarray, q: np.ndarray) -> np.ndarray:
    """The bit-serial table form with integer tables, int64 [M, N]."""
    M, K = a.shape
    N = q.shape[1]
    acc = np.empty((M, N), dtype=np.int64)
    lib().oracle_ternary_lut_matmul(_p(np.ascontiguousarray(a, dtype=np.int32)), _p(np.ascontiguousarray(q)),
                                    C.c_int(M), C.c_int(K), C.c_int(N), _p(acc))
    return acc


def ternary_dequant_int8(q: np.ndarray) -> np.ndarray:
    """Codes -> int8 values through the two tables, int8 [K, N]."""
    K, N = q.shape
    w8 = np.empty((K, N), dtype=np.int8)
    lib().oracle_ternary_dequant_int8(_p(np.ascontiguousarray(q)), C.c_int(K), C.c_int(N), _p(w8))
    return w8


def int8_matmul(a8: np.ndarray, w8: np.ndarray) -> np.ndarray:
    M, K = a8.shape
    N = w8.shape[1]
    acc = np.empty((M, N), dtype=np.int64)
    lib().oracle_int8_matmul(_p(np.ascontiguousarray(a8, dtype=np.int32)), _p(np.ascontiguousarray(w8)),
                             C.c_int(M), C.c_int(K), C.c_int(N), _p(acc))
    return acc


def scale_result(acc: np.ndarray, s_a: np.ndarray, s_w: float) -> np.ndarray:
    M, N = acc.shape
    y = np.empty((M, N), dtype=np.float64)
    lib().oracle_scale_result(_p(np.ascontiguousarray(acc)), _p(np.ascontiguousarray(s_a)), C.c_double(s_w),
                              C.c_int(M), C.c_int(N), _p(y))
    return y


def decode(x: np.ndarray, q: np.ndarray, s_w: float) -> np.ndarray:
    """W_INT2(ternary) A_INT16 decode: quantize rows to 16 bits, integer table lookups, scale."""
    a, s_a = quantize_rows(x, 32767)
    return scale_result(ternary_lut_matmul(a, q), s_a, s_w)


def prefill(x: np.ndarray, q: np.ndarray, s_w: float) -> np.ndarray:
    """Prefill: quantize rows to 8 bits, weights dequantized to INT8 by table lookup, integer matmul, scale."""
    a8, s_a = quantize_rows(x, 127)
    return scale_result(int8_matmul(a8, ternary_dequant_int8(q)), s_a, s_w)
