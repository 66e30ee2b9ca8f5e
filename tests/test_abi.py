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
    # every entry point has its argument types declared: ctypes would otherwise pass pointers as 32-bit ints
    for n in names - {"tman_version"}:
        assert getattr(lib, n).argtypes is not None, f"{n} has no argtypes"


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


@pytest.mark.parametrize("offset", [4, 8])
def test_misaligned_buffers_rejected_before_any_launch(lib, offset):
    """Packed buffers and workspaces must start on a 256-byte boundary, activations and outputs on a
    16-byte boundary: every entry point that takes one says TMAN_ERR_SHAPE on the host (the fake
    pointers are never dereferenced)."""
    ok = C.c_void_p(4096 * 256)
    bad = C.c_void_p(4096 * 256 + offset)
    big = 1 << 30
    out = C.c_int(0)
    assert lib.tman_pack_weights(ok, ok, ok, 128, 8, 4, 64, bad, big, None) == 2
    assert lib.tman_unpack_weights(bad, big, 128, 8, 4, 64, ok, ok, ok, ok, big, None) == 2
    assert lib.tman_unpack_weights(ok, big, 128, 8, 4, 64, ok, ok, ok, bad, big, None) == 2
    assert lib.tman_debug_indices(bad, 128, 8, 4, 64, ok, ok, big, None) == 2
    assert lib.tman_debug_indices(ok, 128, 8, 4, 64, ok, bad, big, None) == 2
    assert lib.tman_workspace_init(bad, big, None) == 2
    assert lib.tman_read_status(bad, C.byref(out), None) == 2
    for fn in (lib.tman_mpgemv, lib.tman_mpgemm):
        assert fn(bad, big, ok, ok, 1, 128, 8, 4, 64, ok, big, None) == 2      # packed
        assert fn(ok, big, ok, ok, 1, 128, 8, 4, 64, bad, big, None) == 2      # workspace
        assert fn(ok, big, bad, ok, 1, 128, 8, 4, 64, ok, big, None) == 2      # activations
        assert fn(ok, big, ok, bad, 1, 128, 8, 4, 64, ok, big, None) == 2      # output
    assert lib.tman_mpgemv_static(bad, big, ok, ok, 1, 128, 8, 4, 64, None, None) == 2
    arr = (C.c_void_p * 1)(bad)
    good = (C.c_void_p * 1)(ok)
    sizes = (C.c_size_t * 1)(big)
    ns = (C.c_int * 1)(8)
    assert lib.tman_mpgemv_grouped(1, arr, sizes, ok, good, 1, 128, ns, 4, 64, ok, big, None) == 2
    assert lib.tman_mpgemv_grouped(1, good, sizes, ok, arr, 1, 128, ns, 4, 64, ok, big, None) == 2


def test_prefill_plan_never_launches_more_workers_than_can_be_resident(lib):
    """Workers of a prefill call wait for one another, so the plan is capped by what the device holds
    at once (the library asks the occupancy query; here the numbers are given).  Host arithmetic only."""
    from paper_2511_11248_b200 import binding as B
    shapes = [(1024, 4096, 4096, 4, 128), (1024, 4096, 14336, 4, 128), (8192, 3584, 18944, 2, 64),
              (100, 24576, 2560, 3, 128), (300, 8192, 1024, 4, 128), (64, 4096, 4096, 4, 64)]
    for M, K, N, bits, G in shapes:
        full = B.tman_debug_gemm_plan_for(M, K, N, bits, G, 148, 148)
        ncta = 2 if full["pair"] else 1
        assert 1 <= full["workers"] * ncta <= 148
        for resident in (1, 7, 36, 60):
            p = B.tman_debug_gemm_plan_for(M, K, N, bits, G, 148, resident)
            assert 1 <= p["workers"] <= resident, (M, K, N, resident, p)
            assert p["pair"] == full["pair"] and p["row_blocks"] == full["row_blocks"]
            # every tile is still covered: whole tiles go round the workers, split tiles have their pieces
            assert p["tiles_m"] * p["tiles_n"] >= 1
            if p["pieces"]:
                assert p["tiles_m"] * p["tiles_n"] * p["pieces"] == p["workers"]
    with pytest.raises(B.TmanError):
        B.tman_debug_gemm_plan_for(1024, 4096, 4096, 4, 128, 148, 0)


def test_decode_plan_choices_and_limits(lib):
    """The decode plan (host arithmetic): one pass for every M on the model shapes, fewer rows per pass
    when the workspace or the number of SMs does not admit the wide variants, and every pass within the
    limits it was admitted under."""
    from paper_2511_11248_b200 import binding as B
    K, N, bits, G = 4096, 14336, 4, 128
    want = {1: [1], 2: [2], 3: [4], 4: [4], 6: [8], 7: [8], 8: [8]}
    for M, variants in want.items():
        p = B.tman_debug_gemv_plan(M, K, N, bits, G)
        assert [q["variant_rows"] for q in p["passes"]] == variants, (M, p)
        assert sum(q["rows"] for q in p["passes"]) == M
        assert p["ws_kib"] * 1024 >= B.tman_workspace_bytes(B.OP_GEMV, M, K, N, bits, G) > (p["ws_kib"] - 1) * 1024
        for q in p["passes"]:
            assert q["ctas"] <= 148 and q["slices"] * q["words"] * 32 >= K
            assert q["smem_bytes"] <= 227 * 1024
    # five rows: one 8-row pass or a 4-row and a 1-row pass, whichever the model says; all rows served
    p5 = B.tman_debug_gemv_plan(5, K, N, bits, G)
    assert sum(q["rows"] for q in p5["passes"]) == 5 and len(p5["passes"]) <= 2
    # a workspace that only holds the 4-row variant's partial sums: eight rows go in two passes of four
    ws4 = B.tman_workspace_bytes(B.OP_GEMV, 4, K, N, bits, G)
    p = B.tman_debug_gemv_plan(8, K, N, bits, G, ws_limit=ws4)
    assert [q["variant_rows"] for q in p["passes"]] == [4, 4] and p["ws_kib"] * 1024 <= ws4 + 1023
    # the smallest workspace the call accepts: single rows
    ws1 = B.tman_workspace_bytes(B.OP_GEMV, 1, K, N, bits, G)
    p = B.tman_debug_gemv_plan(3, K, N, bits, G, ws_limit=ws1)
    assert all(q["variant_rows"] <= 2 for q in p["passes"]) and sum(q["rows"] for q in p["passes"]) == 3
    with pytest.raises(B.TmanError) as e:
        B.tman_debug_gemv_plan(3, K, N, bits, G, ws_limit=ws1 - 1024)
    assert e.value.status == 3
    # a long reduction on a small device: the 8-word K-slices would need more CTAs than there are SMs
    p = B.tman_debug_gemv_plan(8, 16384, 4096, 2, 64, sms=40)
    assert all(q["slices"] <= 40 for q in p["passes"]) and sum(q["rows"] for q in p["passes"]) == 8
    assert all(q["variant_rows"] < 8 for q in p["passes"])
    # more rows never cost less, more bits never cost less
    costs = [B.tman_debug_gemv_plan(M, K, N, bits, G)["cost_us"] for M in range(1, 9)]
    assert all(a <= b + 1e-9 for a, b in zip(costs, costs[1:]))
    assert B.tman_debug_gemv_plan(4, K, N, 2, G)["cost_us"] < B.tman_debug_gemv_plan(4, K, N, 4, G)["cost_us"]
