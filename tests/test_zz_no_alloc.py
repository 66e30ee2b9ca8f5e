"""tman_mpgemv_static: the decode matmul for callers that cannot allocate a workspace.

A serving runtime that froze its memory arena, or code running inside another framework's
callback, has no way to produce the scratch buffer tman_mpgemv wants.  The static variant keeps
that scratch inside the library (4 KiB per GPU).  It must give what tman_mpgemv gives, call
after call, although every call reuses the same array and finds the previous call's leftovers
in it.  This file is collected last on purpose: a failure here cannot hide another test's.
"""
import numpy as np
import pytest
import torch

from paper_2511_11248_b200 import binding as B, helpers as H, synth

pytestmark = pytest.mark.gpu
TOL = 5e-3   # same bound as the other decode tests: max|a - b| / max|b|


def _reference(c, dev, packed):
    ws = H.alloc_workspace(B.OP_GEMV, c.M, c.K, c.N, c.bits, c.group)
    y = torch.empty((c.M, c.N), dtype=torch.float16, device="cuda")
    B.tman_mpgemv(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group, ws)
    assert B.tman_read_status(ws) == 0
    return H.to_f64(y)


def test_two_calls_in_a_row_match_the_workspace_variant():
    # two different problems back to back: the second call starts from the first one's leftovers
    cases = [synth.small_case(3, 2048, 264, 4, 64, seed=31), synth.small_case(1, 4096, 1032, 2, 64, seed=32)]
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    for c in cases:
        dev = H.device_case(c)
        packed = H.pack_case(c, dev)
        want = _reference(c, dev, packed)
        y = torch.full((c.M, c.N), float("nan"), dtype=torch.float16, device="cuda")
        B.tman_mpgemv_static(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group, status)
        torch.cuda.synchronize()
        got = H.to_f64(y)
        assert int(status.item()) == 0
        assert np.all(np.isfinite(got))
        assert float(np.max(np.abs(got - want)) / np.max(np.abs(want))) <= TOL


def test_same_problem_twice_gives_the_same_answer():
    c = synth.small_case(2, 4096, 520, 3, 128, seed=33)
    dev = H.device_case(c)
    packed = H.pack_case(c, dev)
    want = _reference(c, dev, packed)
    for _ in range(2):
        y = torch.empty((c.M, c.N), dtype=torch.float16, device="cuda")
        B.tman_mpgemv_static(packed, dev["x"], y, c.M, c.K, c.N, c.bits, c.group)
        torch.cuda.synchronize()
        got = H.to_f64(y)
        assert float(np.max(np.abs(got - want)) / np.max(np.abs(want))) <= TOL


def test_no_legal_shape_outgrows_the_fixed_array():
    # the array is 4 KiB; the decode path's global scratch is its status block, whatever the shape, so the
    # size check of the entry point never refuses a legal decode shape
    for M, K, N, bits, G in [(8, 18944, 18944, 2, 128), (1, 4096, 152064, 4, 32), (8, 128, 8, 4, 128)]:
        assert B.tman_workspace_bytes(B.OP_GEMV, M, K, N, bits, G) <= 4096
