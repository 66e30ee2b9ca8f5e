"""tman_mpgemv_static: the decode matmul for callers that cannot allocate a workspace.

A serving runtime that froze its memory arena, or code running inside another framework's
callback, has no way to produce the scratch buffer tman_mpgemv wants.  The static variant keeps
that scratch inside the library (4 MiB per GPU).  It must give what tman_mpgemv gives, call
after call, although every call reuses the same array and finds the previous call's leftovers
in it.  This file is collected last on purpose: a failure here cannot hide another test's.
"""
import numpy as np
import pytest
import torch

from oracle import tman_oracle as orc
from paper_2511_11248_b200 import binding as B, helpers as H, synth

pytestmark = pytest.mark.gpu
TOL = 5e-3   # same bound as the other decode tests: max|a - b| / max|b|


def _reference(c, dev, packed):
    ws = H.alloc_workspace(B.OP_GEMV, c.M, c.K, c.N, c.bits, c.group)
    y = H.alloc_y(c.M, c.N)
    B.tman_mpgemv(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group, ws)
    assert B.tman_read_status(ws) == 0
    return H.to_f64(y)


def _oracle_err(c, got):
    ref = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, c.group)
    return float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))


def test_two_calls_in_a_row_match_the_workspace_variant():
    # two different problems back to back: the second call starts from the first one's leftovers
    cases = [synth.small_case(3, 2048, 264, 4, 64, seed=31), synth.small_case(1, 4096, 1032, 2, 64, seed=32),
             synth.small_case(7, 2304, 200, 3, 64, seed=34)]
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    for c in cases:
        dev = H.device_case(c)
        packed = H.pack_case(c, dev)
        want = _reference(c, dev, packed)
        y = H.alloc_y(c.M, c.N)
        B.tman_mpgemv_static(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group, status)
        torch.cuda.synchronize()
        H.check_guards()
        got = H.to_f64(y)
        assert int(status.item()) == 0
        assert np.all(np.isfinite(got))
        assert np.array_equal(got, want)        # same kernels, same summation order: the same bits
        assert _oracle_err(c, got) <= TOL


def test_same_problem_twice_gives_the_same_answer():
    c = synth.small_case(2, 4096, 520, 3, 128, seed=33)
    dev = H.device_case(c)
    packed = H.pack_case(c, dev)
    want = _reference(c, dev, packed)
    for _ in range(2):
        y = H.alloc_y(c.M, c.N)
        B.tman_mpgemv_static(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group)
        torch.cuda.synchronize()
        got = H.to_f64(y)
        assert np.array_equal(got, want)
        assert _oracle_err(c, got) <= TOL


def test_no_device_memory_is_allocated_or_freed():
    c = synth.small_case(1, 4096, 1032, 2, 64, seed=35)
    dev = H.device_case(c)
    packed = H.pack_case(c, dev)
    y = H.alloc_y(c.M, c.N)
    B.tman_mpgemv_static(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group)   # the first call may look up the array
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    held0 = torch.cuda.memory_allocated()
    for _ in range(3):
        B.tman_mpgemv_static(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_allocated() == held0


def test_status_word_reaches_the_caller_and_a_good_call_follows_a_refused_one():
    c = synth.small_case(2, 1024, 264, 4, 64, seed=36)
    dev = H.device_case(c)
    packed = H.pack_case(c, dev)
    junk = torch.zeros_like(packed)
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    y = H.alloc_y(c.M, c.N, fill=3.0)
    B.tman_mpgemv_static(junk, dev["x"], y, c.M, c.K, c.N, c.bits, c.group, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 5              # TMAN_ERR_BAD_PACKED
    assert bool((y == 3.0).all())
    H.check_guards()
    B.tman_mpgemv_static(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(H.to_f64(y), _reference(c, dev, packed))


def test_shape_beyond_the_fixed_array_is_refused():
    # scratch for four rows, K = 18944, N = 18944 is far above 4 MiB: refused on the host, nothing enqueued
    M, K, N, bits, G = 4, 18944, 18944, 2, 128
    assert B.tman_workspace_bytes(B.OP_GEMV, M, K, N, bits, G) > (4 << 20)
    packed = torch.empty(B.tman_packed_bytes(K, N, bits, G), dtype=torch.uint8, device="cuda")
    x = torch.zeros((M, K), dtype=torch.float16, device="cuda")
    y = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    with pytest.raises(B.TmanError) as e:
        B.tman_mpgemv_static(packed, x, y, M, K, N, bits, G)
    assert e.value.status == 4   # TMAN_ERR_BUFFER_TOO_SMALL
