"""Pins of the integer oracle (per-tensor ternary weights, A_INT16 decode, INT8 prefill) against what the
paper and arithmetic fix: brute force, closed forms, the table form against the definition bit for bit,
the quantization error bound against the fp64 product, and the per-block oracle on the same weights."""
import numpy as np
import pytest

from oracle import tman_oracle as orc
from oracle import tman_oracle_int as oi


def ternary_case(M, K, N, seed, spread=1.0):
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((M, K)) * spread).astype(np.float16)
    t = rng.choice(np.array([-1, 0, 1], dtype=np.int8), size=(K, N), p=[0.3, 0.4, 0.3])
    q = (t + 1).astype(np.uint8)
    return x, t, q, 0.0173


def test_row_quantization_by_hand():
    # Sec. 6.1 (A_INT16): one row by hand: amax = 2 -> s_a = 2 / 32767; ties go to the even integer
    x = np.array([[2.0, -1.0, 0.5, 0.0]], dtype=np.float16)
    a, s = oi.quantize_rows(x, 32767)
    assert s[0] == float(np.float32(2.0) / np.float32(32767))            # the scale is a single-precision value
    assert a.tolist() == [[32767, -16384, 8192, 0]]      # 16383.5 -> 16384 (even), 8191.75 -> 8192
    a8, s8 = oi.quantize_rows(x, 127)
    assert s8[0] == float(np.float32(2.0) / np.float32(127)) and a8.tolist() == [[127, -64, 32, 0]]   # 63.5 -> 64, 31.75 -> 32
    # an exact tie decided in single precision: amax = 127 -> s_a = 1, 2.5 -> 2 and 3.5 -> 4 (to even)
    a8, s8 = oi.quantize_rows(np.array([[127.0, 2.5, 3.5, -2.5]], dtype=np.float16), 127)
    assert s8[0] == 1.0 and a8.tolist() == [[127, 2, 4, -2]]
    # an all-zero row keeps scale 1 and quantizes to zeros
    a0, s0 = oi.quantize_rows(np.zeros((1, 8), dtype=np.float16), 32767)
    assert s0[0] == 1.0 and not a0.any()


@pytest.mark.parametrize("qmax", [32767, 127])
def test_row_quantization_properties(qmax):
    x, *_ = ternary_case(5, 256, 8, seed=1, spread=3.0)
    a, s = oi.quantize_rows(x, qmax)
    xf = x.astype(np.float64)
    assert np.all(np.abs(a) <= qmax) and np.all(np.abs(a).max(axis=1) == qmax)
    s32 = (np.abs(x.astype(np.float32)).max(axis=1) / np.float32(qmax)).astype(np.float32)
    assert np.array_equal(s, s32.astype(np.float64))                           # single-precision scale
    # half a step, plus the single-precision quotient's own rounding (at most 2^-9 of a step near qmax)
    assert np.all(np.abs(xf - a * s[:, None]) <= s[:, None] * (0.5 + 2.0 ** -8))
    assert np.array_equal(a, np.rint(x.astype(np.float32) / s32[:, None]).astype(np.int32))   # fp32 quotient, ties to even


def test_definition_against_brute_force_and_numpy():
    x, t, q, _ = ternary_case(3, 32, 5, seed=2)
    a, _ = oi.quantize_rows(x, 32767)
    want = [[sum(int(a[m, k]) * int(t[k, n]) for k in range(32)) for n in range(5)] for m in range(3)]
    assert oi.ternary_matmul(a, q).tolist() == want
    x, t, q, _ = ternary_case(4, 512, 24, seed=3)
    a, _ = oi.quantize_rows(x, 32767)
    assert np.array_equal(oi.ternary_matmul(a, q), a.astype(np.int64) @ t.astype(np.int64))


@pytest.mark.parametrize("M,K,N,seed", [(1, 128, 8, 4), (3, 2560, 16, 5), (2, 6912, 8, 6)])
def test_table_form_equals_definition_bit_for_bit(M, K, N, seed):
    # Sec. 2.2 / Fig. 2 on integers: planes, 4-bit indices, integer tables, shift-accumulate, minus
    # zero-point (1) x activation sum -- exactly the definition (shapes include the paper's BitNet sizes)
    x, t, q, _ = ternary_case(M, K, N, seed)
    a, _ = oi.quantize_rows(x, 32767)
    assert np.array_equal(oi.ternary_lut_matmul(a, q), oi.ternary_matmul(a, q))


def test_closed_forms():
    x, _, _, _ = ternary_case(2, 256, 8, seed=7)
    a, _ = oi.quantize_rows(x, 32767)
    ones = np.full((256, 8), 2, dtype=np.uint8)            # t = +1 everywhere: the activation sum
    assert np.array_equal(oi.ternary_lut_matmul(a, ones), np.repeat(a.sum(axis=1, dtype=np.int64)[:, None], 8, axis=1))
    zeros = np.full((256, 8), 1, dtype=np.uint8)           # t = 0 everywhere
    assert not oi.ternary_lut_matmul(a, zeros).any()
    minus = np.zeros((256, 8), dtype=np.uint8)             # t = -1 everywhere
    assert np.array_equal(oi.ternary_lut_matmul(a, minus), -oi.ternary_lut_matmul(a, ones))
    onehot = np.zeros((1, 256), dtype=np.int32)            # a one-hot activation reads out a weight row
    onehot[0, 77] = 5
    _, t, q, _ = ternary_case(1, 256, 8, seed=8)
    assert np.array_equal(oi.ternary_lut_matmul(onehot, q)[0], 5 * t[77].astype(np.int64))


def test_dequant_to_int8_through_the_two_tables():
    # Sec. 4.1 / Fig. 7 with an integer second table; Sec. 6.2: per-tensor weights become INT8
    _, t, q, _ = ternary_case(1, 512, 24, seed=9)
    w8 = oi.ternary_dequant_int8(q)
    assert w8.dtype == np.int8 and np.array_equal(w8, t)
    # every aligned group of four codes, exhaustively (3^4 = 81 groups)
    groups = np.array([[(g // 3 ** j) % 3 for j in range(4)] for g in range(81)], dtype=np.uint8)   # [81, 4]
    q_all = np.ascontiguousarray(groups.T.reshape(4, 81))          # K = 4, N = 81
    assert np.array_equal(oi.ternary_dequant_int8(q_all), q_all.astype(np.int8) - 1)


def test_prefill_int8_matmul():
    x, t, q, s_w = ternary_case(6, 256, 16, seed=10)
    a8, s_a = oi.quantize_rows(x, 127)
    acc = oi.int8_matmul(a8, oi.ternary_dequant_int8(q))
    assert np.array_equal(acc, a8.astype(np.int64) @ t.astype(np.int64))
    assert np.array_equal(oi.prefill(x, q, s_w), s_a[:, None] * s_w * acc)


@pytest.mark.parametrize("qmax,fn", [(32767, "decode"), (127, "prefill")])
def test_result_within_the_quantization_error_bound(qmax, fn):
    # |y - s_w * x.t| <= s_w * (s_a / 2) * sum_k |t[k][n]|: each activation moves by at most half a step
    x, t, q, s_w = ternary_case(4, 2560, 32, seed=11, spread=2.0)
    y = getattr(oi, fn)(x, q, s_w)
    exact = s_w * (x.astype(np.float64) @ t.astype(np.float64))
    _, s_a = oi.quantize_rows(x, qmax)
    bound = s_w * (s_a[:, None] / 2) * np.abs(t).sum(axis=0, dtype=np.float64)[None, :]
    assert np.all(np.abs(y - exact) <= bound * (1 + 2.0 ** -7) + 1e-12)
    # and the 16-bit path is far inside the fp path's tolerance, the 8-bit path is not as close
    rel = np.max(np.abs(y - exact)) / np.max(np.abs(exact))
    assert rel < (1e-4 if qmax == 32767 else 2e-2)


def test_per_tensor_ternary_is_a_special_case_of_the_per_block_format():
    # the same weights written as 2-bit codes with zero-point 1 and one scale repeated in every block:
    # the per-block fp oracle on the dequantized integer activations gives the same numbers
    x, t, q, s_w = ternary_case(2, 512, 16, seed=12)
    a, s_a = oi.quantize_rows(x, 2047)                     # 12-bit so that a is exact in fp16
    xa = a.astype(np.float16)
    assert np.array_equal(xa.astype(np.int32), a)
    G = 128
    s16 = np.float16(s_w)
    scales = np.full((512 // G, 16), s16, dtype=np.float16)
    zeros = np.ones((512 // G, 16), dtype=np.uint8)
    ref = orc.mpgemm(xa, q, scales, zeros, G)
    got = oi.scale_result(oi.ternary_lut_matmul(a, q), np.ones(2), float(s16))
    assert np.allclose(got, ref, rtol=1e-12, atol=0)
