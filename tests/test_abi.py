"""Host-only checks of the C ABI: the library loads, exports every symbol the header declares,
and rejects bad arguments before touching a GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2511_11248_b200 import build, binding
    build.build()
    return binding.lib()


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(tman_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert {"tman_pack_weights", "tman_mpgemv", "tman_mpgemm"} <= names
    for n in names:
        assert hasattr(lib, n), n
    from paper_2511_11248_b200 import binding
    assert set(binding.EXPORTS) <= names
    for n in names:
        assert hasattr(binding, n), f"binding lacks {n}"


def test_version_and_status_strings(lib):
    from paper_2511_11248_b200 import binding as B
    assert B.tman_version() >= 1
    assert B.tman_status_string(0) == "TMAN_OK"
    assert B.tman_status_string(5) == "TMAN_ERR_BAD_PACKED"
    assert B.tman_status_string(99) == "TMAN_ERR_UNKNOWN"


def test_packed_bytes_matches_format_description(lib):
    from paper_2511_11248_b200 import binding as B
    up = lambda v: (v + 255) // 256 * 256
    for K, N, bits, G in [(4096, 4096, 4, 64), (4096, 14336, 2, 64), (14336, 4096, 3, 128), (128, 8, 1, 32)]:
        want = 256 + up(K * N * bits // 8) + up(K // G * N * 2) + up(K // G * (N // 4) * 2)
        assert B.tman_packed_bytes(K, N, bits, G) == want
    # config 1 (K = N = 4096, 4-bit, group 64): planes + scales (zeros are stored as nibbles)
    assert B.tman_packed_bytes(4096, 4096, 4, 64) == 256 + 8388608 + 524288 + 131072


def test_packed_bytes_agrees_with_oracle_format(lib):
    from oracle import tman_oracle as orc
    from paper_2511_11248_b200 import binding as B
    for K, N, bits, G in [(256, 24, 3, 64), (1024, 136, 4, 128), (128, 8, 2, 32)]:
        assert B.tman_packed_bytes(K, N, bits, G) == orc.packed_bytes(K, N, bits, G)


@pytest.mark.parametrize("K,N,bits,G", [(100, 8, 4, 64), (128, 6, 4, 64), (128, 8, 5, 64),
                                         (128, 8, 0, 64), (128, 8, 4, 48), (0, 8, 4, 64)])
def test_bad_shapes_rejected(lib, K, N, bits, G):
    from paper_2511_11248_b200 import binding as B
    with pytest.raises(B.TmanError) as e:
        B.tman_packed_bytes(K, N, bits, G)
    assert e.value.status == 2


def test_null_and_range_errors_before_any_launch(lib):
    out = C.c_size_t(0)
    assert lib.tman_packed_bytes(128, 8, 4, 64, None) == 1
    assert lib.tman_workspace_bytes(7, 1, 128, 8, 4, 64, C.byref(out)) == 3
    assert lib.tman_workspace_bytes(0, 9, 128, 8, 4, 64, C.byref(out)) == 2
    assert lib.tman_workspace_bytes(0, 0, 128, 8, 4, 64, C.byref(out)) == 2
    # null data pointers: rejected on the host
    assert lib.tman_pack_weights(None, None, None, 128, 8, 4, 64, None, 0, None) == 1
    assert lib.tman_mpgemv(None, 0, None, None, 1, 128, 8, 4, 64, None, 0, None) == 1
    assert lib.tman_mpgemm(None, 0, None, None, 1, 128, 8, 4, 64, None, 0, None) == 1
    assert lib.tman_debug_luts(None, 1, 128, None, None) == 1
    # fake non-null pointers (never dereferenced: the size checks fail first)
    fake = C.c_void_p(4096 * 256)
    assert lib.tman_pack_weights(fake, fake, fake, 128, 8, 4, 64, fake, 16, None) == 4
    assert lib.tman_mpgemv(fake, 1 << 30, fake, fake, 9, 128, 8, 4, 64, fake, 1 << 30, None) == 2
    assert lib.tman_mpgemv(fake, 1 << 30, fake, fake, 1, 128, 8, 1, 64, fake, 1 << 30, None) == 3
    assert lib.tman_mpgemv(fake, 1 << 30, fake, fake, 1, 128, 8, 4, 64, fake, 8, None) == 4
    assert lib.tman_mpgemv(fake, 300, fake, fake, 1, 128, 8, 4, 64, fake, 1 << 30, None) == 4
    assert lib.tman_mpgemm(fake, 300, fake, fake, 1, 128, 8, 4, 64, fake, 1 << 30, None) == 4
    assert lib.tman_mpgemm(fake, 1 << 30, fake, fake, 0, 128, 8, 4, 64, fake, 1 << 30, None) == 2
    assert lib.tman_unpack_weights(fake, 16, 128, 8, 4, 64, fake, fake, fake, fake, 256, None) == 4
    assert lib.tman_workspace_init(fake, 8, None) == 4


def test_workspace_sizes(lib):
    from paper_2511_11248_b200 import binding as B
    assert B.tman_workspace_bytes(B.OP_AUX, 1, 128, 8, 4, 64) == 256
    assert B.tman_workspace_bytes(B.OP_GEMM, 1024, 4096, 4096, 4, 128) >= 256
    w = B.tman_workspace_bytes(B.OP_GEMV, 1, 4096, 4096, 4, 64)
    assert w >= 256 + 4096 + 4 * 4096 * 4
