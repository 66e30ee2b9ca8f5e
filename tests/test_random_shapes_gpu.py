"""Seeded random legal shapes through both matmuls and the integer path: every M, bit width and group
size, K any multiple of 128, N any multiple of 8, compared element by element with the oracles."""
import numpy as np
import pytest
import torch

from oracle import tman_oracle as orc
from oracle import tman_oracle_int as oi
from paper_2511_11248_b200 import binding as B, helpers as H, synth
from parity import TOL, rel_err, run

pytestmark = pytest.mark.gpu


def draw_shapes(seed, count, max_m, max_k_blocks, max_n8):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(count):
        M = int(rng.integers(1, max_m + 1))
        K = 128 * int(rng.integers(1, max_k_blocks + 1))
        N = 8 * int(rng.integers(1, max_n8 + 1))
        bits = int(rng.choice([2, 3, 4]))
        G = int(rng.choice([32, 64, 128]))
        out.append((M, K, N, bits, G, 1000 * seed + i))
    return out


@pytest.mark.parametrize("M,K,N,bits,G,seed", draw_shapes(1, 36, 8, 40, 90))
def test_decode_random_shapes(M, K, N, bits, G, seed):
    c = synth.small_case(M, K, N, bits, G, seed=seed, outliers=(seed % 3 == 0))
    y, *_ = run(B.OP_GEMV, c, pack="oracle" if seed % 2 else "library")
    assert rel_err(H.to_f64(y), orc.mpgemm(c.x, c.codes, c.scales, c.zeros, c.group)) <= TOL


@pytest.mark.parametrize("M,K,N,bits,G,seed", draw_shapes(2, 24, 700, 24, 120))
def test_prefill_random_shapes(M, K, N, bits, G, seed):
    c = synth.small_case(M, K, N, bits, G, seed=seed, outliers=(seed % 3 == 0))
    y, *_ = run(B.OP_GEMM, c, pack="oracle" if seed % 2 else "library")
    assert rel_err(H.to_f64(y), orc.mpgemm(c.x, c.codes, c.scales, c.zeros, c.group)) <= TOL


@pytest.mark.parametrize("M,K,N,bits,G,seed", draw_shapes(3, 12, 300, 20, 60))
def test_integer_path_random_shapes(M, K, N, bits, G, seed):
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((M, K)) * float(rng.choice([0.01, 1.0, 50.0]))).astype(np.float16)
    q = rng.integers(0, 3, size=(K, N)).astype(np.uint8)
    packed = H.alloc_packed(K, N, 2, G)
    B.tman_pack_weights(torch.from_numpy(q).cuda(), torch.ones((K // G, N), dtype=torch.float16, device="cuda"),
                        torch.ones((K // G, N), dtype=torch.uint8, device="cuda"), K, N, 2, G, packed)
    xd = torch.from_numpy(x.view(np.int16)).cuda().view(torch.float16)
    s_w = 0.013
    ws = H.alloc_workspace(B.OP_GEMV, 1, K, N, 2, G)
    # decode: first row, 16-bit integers, exact sums
    a16 = H.guarded_bytes(K * 2, "a_i16").view(torch.int16).view(1, K)
    sa = H.guarded_bytes(((M * 4 + 255) // 256) * 256, "row_scale").view(torch.float32)
    acc = H.guarded_bytes(N * 4, "acc").view(torch.int32).view(1, N)
    y1 = H.alloc_y(1, N)
    B.tman_quantize_rows(xd, 1, K, 32767, a16, sa)
    B.tman_mpgemv_ternary(packed, a16, sa, s_w, y1, acc, 1, K, N, G, ws)
    assert B.tman_read_status(ws) == 0
    a_ref, s_ref = oi.quantize_rows(x[:1], 32767)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), oi.ternary_lut_matmul(a_ref, q))
    # prefill: all rows, 8-bit integers
    a8 = H.guarded_bytes(M * K, "a_i8").view(torch.int8).view(M, K)
    y = H.alloc_y(M, N)
    B.tman_quantize_rows_i8(xd, M, K, a8, sa)
    B.tman_mpgemm_ternary_i8(packed, a8, sa, s_w, y, M, K, N, G, ws)
    assert B.tman_read_status(ws) == 0
    H.check_guards()
    ref = oi.prefill(x, q, float(np.float32(s_w)))
    got = H.to_f64(y)
    assert np.all(np.abs(got - ref) <= np.abs(ref) * 2.0 ** -10 + 1e-7)
