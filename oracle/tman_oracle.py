"""NumPy-facing wrapper of the plain-C oracle (test infrastructure only).

Every function here marshals NumPy arrays into the C routines of
``tman_oracle.c``; the arithmetic lives there.  Passages followed:
Sec. 2.2 (dequantization formula; bit-serial table lookup, Fig. 2),
Sec. 4.1 (two-level lookup dequantization, Fig. 7), Sec. 4.3 (aggregation
inside a quantization block, scaling, floating-point aggregation across blocks).
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from .build_oracle import build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_packed_bytes.restype = C.c_size_t
        _lib.oracle_packed_bytes.argtypes = [C.c_int] * 4
        _lib.oracle_num_threads.restype = C.c_int
        _lib.oracle_unpack.restype = C.c_int
    return _lib


def _p(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


def _u16(a: np.ndarray) -> np.ndarray:
    assert a.dtype == np.float16
    return np.ascontiguousarray(a).view(np.uint16)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def mpgemm(x, codes, scales, zeros, group: int) -> np.ndarray:
    """y = x . (s * (q - z)) by the definition, fp64 [M, N]."""
    M, K = x.shape
    N = codes.shape[1]
    y = np.empty((M, N), dtype=np.float64)
    lib().oracle_mpgemm(_p(_u16(x)), _p(np.ascontiguousarray(codes)), _p(_u16(scales)),
                        _p(np.ascontiguousarray(zeros)), C.c_int(M), C.c_int(K), C.c_int(N),
                        C.c_int(group), _p(y))
    return y


def mpgemm_rows(x, codes, scales, zeros, group: int, rows) -> np.ndarray:
    """The definition on selected output rows only, fp64 [len(rows), N]."""
    K = x.shape[1]
    N = codes.shape[1]
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int32))
    y = np.empty((len(rows), N), dtype=np.float64)
    lib().oracle_mpgemm_rows(_p(_u16(x)), _p(np.ascontiguousarray(codes)), _p(_u16(scales)),
                             _p(np.ascontiguousarray(zeros)), _p(rows), C.c_int(len(rows)),
                             C.c_int(K), C.c_int(N), C.c_int(group), _p(y))
    return y


def indices(codes, bits: int) -> np.ndarray:
    """4-bit table indices per plane, uint8 [bits, K/4, N]."""
    K, N = codes.shape
    idx = np.empty((bits, K // 4, N), dtype=np.uint8)
    lib().oracle_indices(_p(np.ascontiguousarray(codes)), C.c_int(K), C.c_int(N),
                         C.c_int(bits), _p(idx))
    return idx


def luts(x) -> np.ndarray:
    """Activation tables, fp64 [M, K/4, 16]."""
    M, K = x.shape
    lut = np.empty((M, K // 4, 16), dtype=np.float64)
    lib().oracle_luts(_p(_u16(x)), C.c_int(M), C.c_int(K), _p(lut))
    return lut


def lut_gemv(x, codes, scales, zeros, bits: int, group: int) -> np.ndarray:
    """The bit-serial table-lookup evaluation, step by step, fp64 [M, N]."""
    M, K = x.shape
    N = codes.shape[1]
    idx = indices(codes, bits)
    lut = luts(x)
    y = np.empty((M, N), dtype=np.float64)
    lib().oracle_lut_gemv(_p(idx), _p(lut), _p(_u16(x)), _p(_u16(scales)),
                          _p(np.ascontiguousarray(zeros)), C.c_int(M), C.c_int(K), C.c_int(N),
                          C.c_int(bits), C.c_int(group), _p(y))
    return y


def repack_table(bits: int) -> np.ndarray:
    """Level-1 table, uint16 [bits, 16]."""
    R = np.empty((bits, 16), dtype=np.uint16)
    lib().oracle_repack_table(C.c_int(bits), _p(R))
    return R


def affine_table(scale: np.float16, zero: int, bits: int) -> np.ndarray:
    """Level-2 table of one (block, column), fp64 [2^bits]."""
    T = np.empty(1 << bits, dtype=np.float64)
    s = np.array([scale], dtype=np.float16).view(np.uint16)[0]
    lib().oracle_affine_table(C.c_uint16(int(s)), C.c_uint8(int(zero)), C.c_int(bits), _p(T))
    return T


def dequant_two_level(codes, scales, zeros, bits: int, group: int) -> np.ndarray:
    """Dequantized weights rebuilt through the two tables, fp64 [K, N]."""
    K, N = codes.shape
    idx = indices(codes, bits)
    w = np.empty((K, N), dtype=np.float64)
    lib().oracle_dequant_two_level(_p(idx), _p(_u16(scales)), _p(np.ascontiguousarray(zeros)),
                                   C.c_int(K), C.c_int(N), C.c_int(bits), C.c_int(group), _p(w))
    return w


def packed_bytes(K: int, N: int, bits: int, group: int) -> int:
    return int(lib().oracle_packed_bytes(K, N, bits, group))


def pack(codes, scales, zeros, bits: int, group: int) -> np.ndarray:
    """Packed buffer as uint8 [packed_bytes]."""
    K, N = codes.shape
    out = np.empty(packed_bytes(K, N, bits, group), dtype=np.uint8)
    lib().oracle_pack(_p(np.ascontiguousarray(codes)), _p(_u16(scales)),
                      _p(np.ascontiguousarray(zeros)), C.c_int(K), C.c_int(N), C.c_int(bits),
                      C.c_int(group), _p(out))
    return out


def unpack(packed: np.ndarray, K: int, N: int, group: int):
    """Inverse of pack: (codes uint8 [K,N], scales fp16 [K/G,N], zeros uint8 [K/G,N])."""
    q = np.empty((K, N), dtype=np.uint8)
    s = np.empty((K // group, N), dtype=np.uint16)
    z = np.empty((K // group, N), dtype=np.uint8)
    rc = lib().oracle_unpack(_p(np.ascontiguousarray(packed)), _p(q), _p(s), _p(z))
    if rc != 0:
        raise ValueError(f"bad packed header (code {rc})")
    return q, s.view(np.float16), z
