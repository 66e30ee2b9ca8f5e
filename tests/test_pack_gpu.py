"""Bit-exactness of packing, unpacking and index extraction: CUDA path vs CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import tman_oracle as orc
from paper_2511_11248_b200 import binding as B, helpers as H, synth

pytestmark = pytest.mark.gpu

SHAPES = [(128, 8, 1, 32), (256, 24, 2, 64), (384, 40, 3, 128), (512, 136, 4, 64), (1024, 1032, 4, 128),
          (128, 8, 4, 128), (4096, 512, 2, 32)]


@pytest.mark.parametrize("K,N,bits,G", SHAPES)
def test_pack_is_bit_exact(K, N, bits, G):
    c = synth.small_case(1, K, N, bits, G, seed=K + N + bits)
    packed = H.pack_case(c)
    torch.cuda.synchronize()
    want = orc.pack(c.codes, c.scales, c.zeros, bits, G)
    got = packed.cpu().numpy()
    assert got.shape == want.shape
    assert np.array_equal(got, want)


@pytest.mark.parametrize("K,N,bits,G", SHAPES)
def test_unpack_roundtrip_and_indices(K, N, bits, G):
    c = synth.small_case(1, K, N, bits, G, seed=3 * K + N + bits)
    dev = H.device_case(c)
    packed = H.pack_case(c, dev)
    ws = H.alloc_workspace(B.OP_AUX, 1, K, N, bits, G)
    q = torch.empty_like(dev["codes"]); s = torch.empty_like(dev["scales"]); z = torch.empty_like(dev["zeros"])
    B.tman_unpack_weights(packed, K, N, bits, G, q, s, z, ws)
    idx = torch.empty((bits, K // 4, N), dtype=torch.uint8, device="cuda")
    B.tman_debug_indices(packed, K, N, bits, G, idx, ws)
    assert B.tman_read_status(ws) == 0
    assert torch.equal(q, dev["codes"]) and torch.equal(z, dev["zeros"])
    assert torch.equal(s.view(torch.int16), dev["scales"].view(torch.int16))
    assert np.array_equal(idx.cpu().numpy(), orc.indices(c.codes, bits))


def test_gpu_unpacks_oracle_packed_buffer():
    K, N, bits, G = 256, 24, 3, 64
    c = synth.small_case(1, K, N, bits, G, seed=99)
    packed = torch.from_numpy(orc.pack(c.codes, c.scales, c.zeros, bits, G)).cuda()
    ws = H.alloc_workspace(B.OP_AUX, 1, K, N, bits, G)
    q = torch.empty((K, N), dtype=torch.uint8, device="cuda")
    s = torch.empty((K // G, N), dtype=torch.float16, device="cuda")
    z = torch.empty((K // G, N), dtype=torch.uint8, device="cuda")
    B.tman_unpack_weights(packed, K, N, bits, G, q, s, z, ws)
    assert B.tman_read_status(ws) == 0
    assert np.array_equal(q.cpu().numpy(), c.codes) and np.array_equal(z.cpu().numpy(), c.zeros)


def test_header_mismatch_sets_status_and_leaves_output():
    K, N, bits, G = 256, 24, 4, 64
    c = synth.small_case(1, K, N, bits, G, seed=5)
    dev = H.device_case(c)
    packed = H.pack_case(c, dev)
    ws = H.alloc_workspace(B.OP_AUX, 1, K, N, bits, G)
    q = torch.full((K, N), 77, dtype=torch.uint8, device="cuda")
    s = torch.empty((K // 128, N), dtype=torch.float16, device="cuda")
    z = torch.empty((K // 128, N), dtype=torch.uint8, device="cuda")
    # same byte size of planes, wrong group: header check must refuse
    big = torch.zeros(B.tman_packed_bytes(K, N, bits, 64), dtype=torch.uint8, device="cuda")
    big[: packed.numel()] = packed
    B.tman_unpack_weights(big, K, N, bits, 128, q, s, z, ws)
    assert B.tman_read_status(ws) == 5
    assert bool((q == 77).all())
    # garbage buffer (no magic)
    B.tman_workspace_init(ws)
    junk = torch.zeros_like(big)
    y = torch.full((1, N), 3.0, dtype=torch.float16, device="cuda")
    wsv = H.alloc_workspace(B.OP_GEMV, 1, K, N, bits, G)
    B.tman_mpgemv(junk, dev["x"], y, 1, K, N, bits, G, wsv)
    assert B.tman_read_status(wsv) == 5
    assert bool((y == 3.0).all())
    wsm = H.alloc_workspace(B.OP_GEMM, 1, K, N, bits, G)
    B.tman_mpgemm(junk, dev["x"], y, 1, K, N, bits, G, wsm)
    assert B.tman_read_status(wsm) == 5
    assert bool((y == 3.0).all())


def test_debug_luts_match_oracle_tables():
    c = synth.small_case(3, 512, 8, 4, 64, seed=6)
    dev = H.device_case(c)
    lut = torch.empty((3, 128, 16), dtype=torch.float32, device="cuda")
    B.tman_debug_luts(dev["x"], 3, 512, lut)
    want = orc.luts(c.x)
    got = lut.cpu().numpy().astype(np.float64)
    # fp32 sums of at most four fp16 values, same order as the oracle: at most a few fp32 ulps
    assert np.max(np.abs(got - want)) <= 4 * 2.0 ** -24 * max(1.0, np.max(np.abs(want)))
