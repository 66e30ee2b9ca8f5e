"""ctypes binding of libtman.so: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors (PyTorch supplies device memory and streams); every step of the
path runs in the library's kernels.  There is no CPU fallback: if the shared library is missing
the import of any entry point raises.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
# TMAN_LIBRARY selects another build of the same library (e.g. libtman_stamps.so, the build with role time stamps)
LIB_PATH = os.environ.get("TMAN_LIBRARY") or os.path.join(HERE, "libtman.so")

TMAN_OK = 0
STATUS_NAMES = {
    0: "TMAN_OK", 1: "TMAN_ERR_NULL", 2: "TMAN_ERR_SHAPE", 3: "TMAN_ERR_UNSUPPORTED",
    4: "TMAN_ERR_BUFFER_TOO_SMALL", 5: "TMAN_ERR_BAD_PACKED", 6: "TMAN_ERR_CUDA", 7: "TMAN_ERR_TIMEOUT",
}
OP_GEMV, OP_GEMM, OP_AUX, OP_TERNARY = 0, 1, 2, 3

EXPORTS = [
    "tman_status_string", "tman_version", "tman_packed_bytes", "tman_workspace_bytes",
    "tman_workspace_init", "tman_read_status", "tman_pack_weights", "tman_unpack_weights",
    "tman_mpgemv", "tman_mpgemm", "tman_debug_indices", "tman_debug_luts", "tman_debug_gemm_plan", "tman_mpgemv_static", "tman_mpgemv_grouped",
    "tman_debug_microbench", "tman_debug_cluster_capacity", "tman_debug_gemm_plan_for", "tman_debug_gemv_plan", "tman_debug_wait_timeout", "tman_debug_mpgemm_variant", "tman_quantize_rows", "tman_mpgemv_ternary", "tman_dequant_ternary_int8", "tman_debug_role_stamps", "tman_quantize_rows_i8", "tman_mpgemm_ternary_i8",
]

_lib = None


class TmanError(RuntimeError):
    def __init__(self, status: int, where: str):
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")
        self.status = status


def lib() -> C.CDLL:
    """Load libtman.so (built by paper_2511_11248_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2511_11248_b200.build`; "
                "there is no fallback path")
        L = C.CDLL(LIB_PATH)
        L.tman_status_string.restype = C.c_char_p
        L.tman_status_string.argtypes = [C.c_int]
        L.tman_version.restype = C.c_int
        i, sz, vp = C.c_int, C.c_size_t, C.c_void_p
        L.tman_packed_bytes.argtypes = [i, i, i, i, C.POINTER(sz)]
        L.tman_workspace_bytes.argtypes = [i, i, i, i, i, i, C.POINTER(sz)]
        L.tman_workspace_init.argtypes = [vp, sz, vp]
        L.tman_read_status.argtypes = [vp, C.POINTER(i), vp]
        L.tman_pack_weights.argtypes = [vp, vp, vp, i, i, i, i, vp, sz, vp]
        L.tman_unpack_weights.argtypes = [vp, sz, i, i, i, i, vp, vp, vp, vp, sz, vp]
        L.tman_mpgemv.argtypes = [vp, sz, vp, vp, i, i, i, i, i, vp, sz, vp]
        L.tman_mpgemm.argtypes = [vp, sz, vp, vp, i, i, i, i, i, vp, sz, vp]
        L.tman_mpgemv_static.argtypes = [vp, sz, vp, vp, i, i, i, i, i, vp, vp]
        L.tman_mpgemv_grouped.argtypes = [i, C.POINTER(vp), C.POINTER(sz), vp, C.POINTER(vp), i, i, C.POINTER(i), i, i, vp, sz, vp]
        L.tman_debug_indices.argtypes = [vp, i, i, i, i, vp, vp, sz, vp]
        L.tman_debug_luts.argtypes = [vp, i, i, vp, vp]
        L.tman_debug_gemm_plan.argtypes = [i, i, i, i, i, C.POINTER(C.c_int)]
        L.tman_debug_microbench.argtypes = [i, i, vp, sz, vp, sz, vp]
        L.tman_debug_cluster_capacity.argtypes = [i, i, i, C.POINTER(C.c_int)]
        L.tman_debug_gemm_plan_for.argtypes = [i, i, i, i, i, i, i, C.POINTER(C.c_int)]
        L.tman_debug_gemv_plan.argtypes = [i, i, i, i, i, i, sz, C.POINTER(C.c_int)]
        L.tman_debug_wait_timeout.argtypes = [vp, sz, C.c_uint, vp]
        L.tman_quantize_rows_i8.argtypes = [vp, i, i, vp, vp, vp]
        L.tman_mpgemm_ternary_i8.argtypes = [vp, sz, vp, vp, C.c_float, vp, i, i, i, i, vp, sz, vp]
        L.tman_debug_role_stamps.argtypes = [vp, sz, i, vp, vp]
        L.tman_dequant_ternary_int8.argtypes = [vp, sz, i, i, i, vp, vp, sz, vp]
        L.tman_quantize_rows.argtypes = [vp, i, i, i, vp, vp, vp]
        L.tman_mpgemv_ternary.argtypes = [vp, sz, vp, vp, C.c_float, vp, vp, i, i, i, i, vp, sz, vp]
        L.tman_debug_mpgemm_variant.argtypes = [i, vp, sz, vp, vp, i, i, i, i, i, vp, vp, sz, vp]
        for name in EXPORTS[2:]:
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _check(st: int, where: str) -> None:
    if st != TMAN_OK:
        raise TmanError(st, where)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _stream(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def tman_version() -> int:
    return int(lib().tman_version())


def tman_status_string(status: int) -> str:
    return lib().tman_status_string(int(status)).decode()


def tman_packed_bytes(K: int, N: int, bits: int, group: int) -> int:
    out = C.c_size_t(0)
    _check(lib().tman_packed_bytes(K, N, bits, group, C.byref(out)), "tman_packed_bytes")
    return int(out.value)


def tman_workspace_bytes(op: int, M: int, K: int, N: int, bits: int, group: int) -> int:
    out = C.c_size_t(0)
    _check(lib().tman_workspace_bytes(op, M, K, N, bits, group, C.byref(out)), "tman_workspace_bytes")
    return int(out.value)


def tman_workspace_init(workspace, stream=None) -> None:
    _check(lib().tman_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                     _stream(stream)), "tman_workspace_init")


def tman_read_status(workspace, stream=None) -> int:
    out = C.c_int(0)
    _check(lib().tman_read_status(_ptr(workspace), C.byref(out), _stream(stream)), "tman_read_status")
    return int(out.value)


def tman_pack_weights(codes, scales, zeros, K, N, bits, group, packed, stream=None) -> None:
    _check(lib().tman_pack_weights(_ptr(codes), _ptr(scales), _ptr(zeros), K, N, bits, group,
                                   _ptr(packed), packed.numel() * packed.element_size(),
                                   _stream(stream)), "tman_pack_weights")


def tman_unpack_weights(packed, K, N, bits, group, codes, scales, zeros, workspace, stream=None) -> None:
    _check(lib().tman_unpack_weights(_ptr(packed), packed.numel() * packed.element_size(), K, N, bits,
                                     group, _ptr(codes), _ptr(scales), _ptr(zeros), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream(stream)),
           "tman_unpack_weights")


def tman_mpgemv(packed, x, y, M, K, N, bits, group, workspace, stream=None) -> None:
    _check(lib().tman_mpgemv(_ptr(packed), packed.numel() * packed.element_size(), _ptr(x), _ptr(y), M, K, N, bits, group, _ptr(workspace),
                             workspace.numel() * workspace.element_size(), _stream(stream)),
           "tman_mpgemv")


def tman_mpgemv_static(packed, x, y, M, K, N, bits, group, status=None, stream=None) -> None:
    """Decode matmul on the library's built-in scratch array: for callers that cannot allocate a
    workspace.  `status`, if given, is a 4-byte device tensor that receives the device-side status."""
    _check(lib().tman_mpgemv_static(_ptr(packed), packed.numel() * packed.element_size(), _ptr(x), _ptr(y),
                                    M, K, N, bits, group, _ptr(status), _stream(stream)),
           "tman_mpgemv_static")


def tman_mpgemv_grouped(packed_list, x, y_list, M, K, N_list, bits, group, workspace, stream=None) -> None:
    """Decode for several weight matrices that share the activations x, in one launch."""
    n = len(packed_list)
    pk = (C.c_void_p * n)(*[_ptr(t) for t in packed_list])
    pb = (C.c_size_t * n)(*[t.numel() * t.element_size() for t in packed_list])
    ys = (C.c_void_p * n)(*[_ptr(t) for t in y_list])
    ns = (C.c_int * n)(*[int(v) for v in N_list])
    _check(lib().tman_mpgemv_grouped(n, pk, pb, _ptr(x), ys, M, K, ns, bits, group, _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream(stream)),
           "tman_mpgemv_grouped")


def tman_mpgemm(packed, x, y, M, K, N, bits, group, workspace, stream=None) -> None:
    _check(lib().tman_mpgemm(_ptr(packed), packed.numel() * packed.element_size(), _ptr(x), _ptr(y), M, K, N, bits, group, _ptr(workspace),
                             workspace.numel() * workspace.element_size(), _stream(stream)),
           "tman_mpgemm")


def tman_debug_indices(packed, K, N, bits, group, idx, workspace, stream=None) -> None:
    _check(lib().tman_debug_indices(_ptr(packed), K, N, bits, group, _ptr(idx), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _stream(stream)),
           "tman_debug_indices")


def tman_debug_gemm_plan(M, K, N, bits, group) -> dict:
    out = (C.c_int * 8)()
    _check(lib().tman_debug_gemm_plan(M, K, N, bits, group, out), "tman_debug_gemm_plan")
    return dict(zip(("pair", "row_blocks", "tiles_m", "tiles_n", "whole_tiles", "workers", "span_tiles", "pieces"), list(out)))


def tman_debug_gemm_plan_for(M, K, N, bits, group, sms, resident) -> dict:
    out = (C.c_int * 8)()
    _check(lib().tman_debug_gemm_plan_for(M, K, N, bits, group, sms, resident, out), "tman_debug_gemm_plan_for")
    return dict(zip(("pair", "row_blocks", "tiles_m", "tiles_n", "whole_tiles", "workers", "span_tiles", "pieces"), list(out)))


def tman_debug_gemv_plan(M, K, N, bits, group, sms=148, ws_limit=0) -> dict:
    out = (C.c_int * 52)()
    _check(lib().tman_debug_gemv_plan(M, K, N, bits, group, sms, C.c_size_t(ws_limit), out), "tman_debug_gemv_plan")
    keys = ("rows", "variant_rows", "words", "slices", "ctas", "smem_bytes")
    return {"ws_kib": out[1], "cost_us": out[2] / 1000.0,
            "passes": [dict(zip(keys, out[4 + 6 * i: 10 + 6 * i])) for i in range(out[0])]}


def tman_dequant_ternary_int8(packed, K, N, group, w8, ws, stream=None) -> None:
    _check(lib().tman_dequant_ternary_int8(_ptr(packed), packed.numel() * packed.element_size(), K, N, group, _ptr(w8),
                                           _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "tman_dequant_ternary_int8")


def tman_quantize_rows_i8(x, M, K, a, row_scale, stream=None) -> None:
    _check(lib().tman_quantize_rows_i8(_ptr(x), M, K, _ptr(a), _ptr(row_scale), _stream(stream)), "tman_quantize_rows_i8")


def tman_mpgemm_ternary_i8(packed, a, row_scale, w_scale, y, M, K, N, group, ws, stream=None) -> None:
    _check(lib().tman_mpgemm_ternary_i8(_ptr(packed), packed.numel() * packed.element_size(), _ptr(a), _ptr(row_scale),
                                        float(w_scale), _ptr(y), M, K, N, group, _ptr(ws), ws.numel() * ws.element_size(),
                                        _stream(stream)), "tman_mpgemm_ternary_i8")


def tman_quantize_rows(x, M, K, qmax, a, row_scale, stream=None) -> None:
    _check(lib().tman_quantize_rows(_ptr(x), M, K, qmax, _ptr(a), _ptr(row_scale), _stream(stream)), "tman_quantize_rows")


def tman_mpgemv_ternary(packed, a, row_scale, w_scale, y, acc, M, K, N, group, ws, stream=None) -> None:
    _check(lib().tman_mpgemv_ternary(_ptr(packed), packed.numel() * packed.element_size(), _ptr(a), _ptr(row_scale),
                                     float(w_scale), _ptr(y), _ptr(acc), M, K, N, group, _ptr(ws),
                                     ws.numel() * ws.element_size(), _stream(stream)), "tman_mpgemv_ternary")


GEMM_VARIANTS = {"product": 0, "convert_dq": 1, "load_full": 2, "sequential": 3}


def tman_debug_mpgemm_variant(variant, packed, x, y, M, K, N, bits, group, ws, wt=None, stream=None) -> None:
    _check(lib().tman_debug_mpgemm_variant(GEMM_VARIANTS.get(variant, variant), _ptr(packed),
                                           packed.numel() * packed.element_size(), _ptr(x), _ptr(y), M, K, N, bits, group,
                                           _ptr(wt), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "tman_debug_mpgemm_variant")


def tman_debug_role_stamps(ws, ctas, stream=None):
    """int64 array [ctas][26 warps][4]: wait clocks (two kinds), role clocks, tag; needs the stamps build."""
    import numpy as np
    out = np.zeros((ctas, 26, 4), dtype=np.int64)
    _check(lib().tman_debug_role_stamps(_ptr(ws), ws.numel() * ws.element_size(), ctas, out.ctypes.data, _stream(stream)),
           "tman_debug_role_stamps")
    return out


def tman_debug_wait_timeout(ws, polls, stream=None) -> None:
    _check(lib().tman_debug_wait_timeout(_ptr(ws), ws.numel() * ws.element_size(), polls, _stream(stream)),
           "tman_debug_wait_timeout")


def tman_debug_luts(x, M, K, lut, stream=None) -> None:
    _check(lib().tman_debug_luts(_ptr(x), M, K, _ptr(lut), _stream(stream)), "tman_debug_luts")


def tman_debug_microbench(kind, arg, results, buffer=None, stream=None) -> None:
    _check(lib().tman_debug_microbench(kind, arg, _ptr(results), results.numel() * results.element_size(),
                                       _ptr(buffer), 0 if buffer is None else buffer.numel() * buffer.element_size(),
                                       _stream(stream)), "tman_debug_microbench")


def tman_debug_cluster_capacity(threads: int, smem_bytes: int, cluster: int) -> int:
    out = C.c_int(0)
    _check(lib().tman_debug_cluster_capacity(threads, smem_bytes, cluster, C.byref(out)), "tman_debug_cluster_capacity")
    return int(out.value)

