"""Parity of the integer decode path (per-tensor ternary weights, 16-bit integer activations) with the
integer oracle, through the C ABI: quantized activations and integer sums bit for bit, y within rounding."""
import numpy as np
import pytest
import torch

from oracle import tman_oracle_int as oi
from paper_2511_11248_b200 import binding as B, helpers as H

pytestmark = pytest.mark.gpu


def ternary_case(M, K, N, seed, spread=1.0):
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((M, K)) * spread).astype(np.float16)
    t = rng.choice(np.array([-1, 0, 1], dtype=np.int8), size=(K, N), p=[0.3, 0.4, 0.3])
    return x, t, (t + 1).astype(np.uint8), 0.0173


def pack_ternary(q, group):
    K, N = q.shape
    codes = torch.from_numpy(q).cuda()
    scales = torch.ones((K // group, N), dtype=torch.float16, device="cuda")
    zeros = torch.ones((K // group, N), dtype=torch.uint8, device="cuda")
    packed = H.alloc_packed(K, N, 2, group)
    B.tman_pack_weights(codes, scales, zeros, K, N, 2, group, packed)
    return packed


@pytest.mark.parametrize("M,K,qmax,spread", [(1, 128, 32767, 1.0), (5, 2560, 32767, 3.0), (3, 6912, 127, 0.01),
                                             (2, 1000, 32767, 200.0), (3, 1001, 127, 1.0), (1, 16384, 32767, 1.0)])
def test_row_quantization_is_bit_exact(M, K, qmax, spread):
    x, *_ = ternary_case(M, K, 8, seed=K + qmax, spread=spread)
    if M > 1:
        x[1, :] = 0                                           # a row of zeros: scale 1, all zeros
    want_a, want_s = oi.quantize_rows(x, qmax)
    xd = torch.from_numpy(x.view(np.int16)).cuda().view(torch.float16)
    a = H.guarded_bytes(M * K * 2, "a_i16").view(torch.int16).view(M, K)
    s = H.guarded_bytes(M * 4, "row_scale").view(torch.float32)
    B.tman_quantize_rows(xd, M, K, qmax, a, s)
    torch.cuda.synchronize()
    H.check_guards()
    assert np.array_equal(a.cpu().numpy().astype(np.int32), want_a)
    assert np.array_equal(s.cpu().numpy().astype(np.float64), want_s)


# the paper's BitNet kernel sizes {2560, 6912} x {2560, 6912}, ragged column counts, one-slice K, both pairings
SHAPES = [(128, 8, 128), (512, 40, 32), (2560, 2560, 128), (2560, 6912, 64), (6912, 2560, 128), (6912, 6912, 128),
          (1152, 264, 64), (16384, 72, 128)]


@pytest.mark.parametrize("K,N,group", SHAPES)
def test_ternary_decode_matches_the_integer_oracle(K, N, group):
    x, t, q, s_w = ternary_case(1, K, N, seed=K + N)
    a_ref, s_ref = oi.quantize_rows(x, 32767)
    acc_ref = oi.ternary_lut_matmul(a_ref, q)
    y_ref = oi.scale_result(acc_ref, s_ref, float(np.float32(s_w)))

    packed = pack_ternary(q, group)
    xd = torch.from_numpy(x.view(np.int16)).cuda().view(torch.float16)
    a = H.guarded_bytes(K * 2, "a_i16").view(torch.int16).view(1, K)
    s = H.guarded_bytes(256, "row_scale").view(torch.float32)
    B.tman_quantize_rows(xd, 1, K, 32767, a, s)
    ws = H.alloc_workspace(B.OP_TERNARY, 1, K, N, 2, group)
    y = H.alloc_y(1, N)
    acc = H.guarded_bytes(N * 4, "acc_i32").view(torch.int32).view(1, N)
    acc.fill_(-12345)
    for _ in range(2):                                        # the second call finds the workspace as the first left it
        B.tman_mpgemv_ternary(packed, a, s, s_w, y, acc, 1, K, N, group, ws)
        assert B.tman_read_status(ws) == 0
        H.check_guards()
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)          # integer work: bit-exact
        got = H.to_f64(y)
        # fp32 product of the two scales and the integer, rounded to fp16: within an fp16 rounding of the fp64 value
        assert np.all(np.abs(got - y_ref) <= np.abs(y_ref) * 2.0 ** -10 + 1e-7)
    # without the integer output
    y2 = H.alloc_y(1, N)
    B.tman_mpgemv_ternary(packed, a, s, s_w, y2, None, 1, K, N, group, ws)
    assert B.tman_read_status(ws) == 0
    assert torch.equal(y, y2)


def test_ternary_closed_forms_and_refusals():
    K, N = 1024, 32
    x, t, q, s_w = ternary_case(1, K, N, seed=3)
    xd = torch.from_numpy(x.view(np.int16)).cuda().view(torch.float16)
    a = H.guarded_bytes(K * 2, "a_i16").view(torch.int16).view(1, K)
    s = H.guarded_bytes(256, "row_scale").view(torch.float32)
    B.tman_quantize_rows(xd, 1, K, 32767, a, s)
    ws = H.alloc_workspace(B.OP_GEMV, 1, K, N, 2, 64)
    y = H.alloc_y(1, N)
    acc = H.guarded_bytes(N * 4, "acc_i32").view(torch.int32).view(1, N)
    asum = int(a.cpu().numpy().astype(np.int64).sum())
    for code, want in ((2, asum), (1, 0), (0, -asum)):        # all +1: the activation sum; all 0; all -1
        packed = pack_ternary(np.full((K, N), code, dtype=np.uint8), 64)
        B.tman_mpgemv_ternary(packed, a, s, s_w, y, acc, 1, K, N, 64, ws)
        assert B.tman_read_status(ws) == 0
        assert bool((acc == want).all())
    with pytest.raises(B.TmanError) as e:                      # at most eight rows
        B.tman_mpgemv_ternary(packed, a, s, s_w, y, acc, 9, K, N, 64, ws)
    assert e.value.status == 2
    junk = torch.zeros_like(packed)
    y.fill_(3.0)
    B.tman_mpgemv_ternary(junk, a, s, s_w, y, acc, 1, K, N, 64, ws)
    assert B.tman_read_status(ws) == 5 and bool((y == 3.0).all())


@pytest.mark.parametrize("K,N,group", [(128, 8, 128), (2560, 2560, 128), (6912, 2560, 64), (1152, 264, 32)])
def test_int8_dequantization_is_bit_exact(K, N, group):
    # Sec. 6.2: per-tensor weights become INT8 through the two lookups; compared with the oracle's tables
    _, t, q, _ = ternary_case(1, K, N, seed=K * 3 + N)
    packed = pack_ternary(q, group)
    ws = H.alloc_workspace(B.OP_AUX, 1, K, N, 2, group)
    w8 = H.guarded_bytes(K * N, "w8").view(torch.int8).view(N, K)
    w8.fill_(55)
    B.tman_dequant_ternary_int8(packed, K, N, group, w8, ws)
    assert B.tman_read_status(ws) == 0
    H.check_guards()
    want = oi.ternary_dequant_int8(q)                         # [K][N]
    assert np.array_equal(w8.cpu().numpy().T, want)
    # a buffer of another shape is refused and the output stays as it was
    w8.fill_(55)
    other = pack_ternary(np.ones((K, N + 8), dtype=np.uint8), group)
    B.tman_dequant_ternary_int8(other, K, N, group, w8, ws)
    assert B.tman_read_status(ws) == 5 and bool((w8 == 55).all())


# one tile, ragged tokens and channels, several k-blocks and tiles per CTA, the paper's BitNet sizes
I8_SHAPES = [(128, 128, 128, 128), (1, 256, 8, 64), (100, 384, 136, 128), (300, 1024, 264, 32), (513, 2560, 2560, 128),
             (1024, 6912, 2560, 128), (2048, 2560, 6912, 64)]


@pytest.mark.parametrize("M,K,N,group", I8_SHAPES)
def test_int8_prefill_matches_the_integer_oracle(M, K, N, group):
    x, t, q, s_w = ternary_case(M, K, N, seed=M + K + N, spread=2.0)
    s_w32 = float(np.float32(s_w))
    a_ref, s_ref = oi.quantize_rows(x, 127)
    y_ref = oi.scale_result(oi.int8_matmul(a_ref, oi.ternary_dequant_int8(q)), s_ref, s_w32)

    packed = pack_ternary(q, group)
    xd = torch.from_numpy(x.view(np.int16)).cuda().view(torch.float16)
    a8 = H.guarded_bytes(M * K, "a_i8").view(torch.int8).view(M, K)
    s = H.guarded_bytes(((M * 4 + 255) // 256) * 256, "row_scale").view(torch.float32)
    B.tman_quantize_rows_i8(xd, M, K, a8, s)
    torch.cuda.synchronize()
    assert np.array_equal(a8.cpu().numpy().astype(np.int32), a_ref)                   # integers: bit-exact
    assert np.array_equal(s[:M].cpu().numpy().astype(np.float64), s_ref)
    ws = H.alloc_workspace(B.OP_AUX, 1, K, N, 2, group)
    y = H.alloc_y(M, N)
    for _ in range(2):
        B.tman_mpgemm_ternary_i8(packed, a8, s, s_w, y, M, K, N, group, ws)
        assert B.tman_read_status(ws) == 0
        H.check_guards()
        got = H.to_f64(y)
        assert np.all(np.isfinite(got))
        # exact integer sums; one fp32 product of scales, one fp32 product with the sum, one rounding to fp16
        assert np.all(np.abs(got - y_ref) <= np.abs(y_ref) * 2.0 ** -10 + 1e-7)
    # a buffer with another header is refused, the output stays
    y.fill_(3.0)
    B.tman_mpgemm_ternary_i8(torch.zeros_like(packed), a8, s, s_w, y, M, K, N, group, ws)
    assert B.tman_read_status(ws) == 5 and bool((y == 3.0).all())


@pytest.mark.parametrize("M,K,N,group", [(2, 1024, 40, 64), (3, 2560, 264, 128), (4, 6912, 2560, 128), (5, 1152, 72, 32),
                                         (8, 2560, 6912, 64), (7, 16384, 16, 128)])
def test_ternary_decode_with_several_rows(M, K, N, group):
    x, t, q, s_w = ternary_case(M, K, N, seed=7 * M + K + N, spread=1.5)
    a_ref, s_ref = oi.quantize_rows(x, 32767)
    acc_ref = oi.ternary_lut_matmul(a_ref, q)
    y_ref = oi.scale_result(acc_ref, s_ref, float(np.float32(s_w)))
    packed = pack_ternary(q, group)
    xd = torch.from_numpy(x.view(np.int16)).cuda().view(torch.float16)
    a = H.guarded_bytes(M * K * 2, "a_i16").view(torch.int16).view(M, K)
    s = H.guarded_bytes(256, "row_scale").view(torch.float32)
    B.tman_quantize_rows(xd, M, K, 32767, a, s)
    ws = H.guarded_bytes(B.tman_workspace_bytes(B.OP_TERNARY, M, K, N, 2, group), "workspace")
    B.tman_workspace_init(ws)
    y = H.alloc_y(M, N)
    acc = H.guarded_bytes(M * N * 4, "acc_i32").view(torch.int32).view(M, N)
    for _ in range(2):
        B.tman_mpgemv_ternary(packed, a, s, s_w, y, acc, M, K, N, group, ws)
        assert B.tman_read_status(ws) == 0
        H.check_guards()
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
        assert np.all(np.abs(H.to_f64(y) - y_ref) <= np.abs(y_ref) * 2.0 ** -10 + 1e-7)
