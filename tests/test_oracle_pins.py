"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's formula: each compares it with a
closed form, an integer library routine, a brute-force enumeration, a value the
paper prints, or an invariant, chosen so that a dropped term, a wrong sign or
index, or a transposed operand fails at least one of them.
"""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import tman_oracle as orc
from paper_2511_11248_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_case(M, K, N, bits, group, seed=0):
    return synth.small_case(M, K, N, bits, group, seed=seed)


# ---- P1: every one of the 2^g bit patterns on K = g inputs ------------------

def test_lut_entries_equal_bruteforce_dot_products():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((3, 8)).astype(np.float16)
    lut = orc.luts(x)                      # [3, 2, 16]
    for m in range(3):
        for t in range(2):
            for p in range(16):
                bitsv = [(p >> j) & 1 for j in range(4)]
                # fp16 values are dyadic rationals: math.fsum is exact here
                want = math.fsum(float(x[m, 4 * t + j]) * bitsv[j] for j in range(4))
                assert lut[m, t, p] == want


def test_lookup_sum_equals_dot_product_for_all_patterns_K_equals_g():
    # K = g = 4, one column per pattern and per plane: codes enumerate all 16
    # patterns of each bit-plane; s = 1, z = 0.  y must be the plain dot product.
    rng = np.random.default_rng(2)
    K, G = 32, 32            # smallest legal K; only the first 4 rows carry codes
    x = np.zeros((1, K), dtype=np.float16)
    x[0, :4] = rng.standard_normal(4).astype(np.float16)
    for bits in (1, 2, 3, 4):
        N = 16 * bits
        codes = np.zeros((K, N), dtype=np.uint8)
        for i in range(bits):
            for p in range(16):
                for j in range(4):
                    codes[j, 16 * i + p] = ((p >> j) & 1) << i
        scales = np.ones((1, N), dtype=np.float16)
        zeros = np.zeros((1, N), dtype=np.uint8)
        y_lut = orc.lut_gemv(x, codes, scales, zeros, bits, G)
        y_def = orc.mpgemm(x, codes, scales, zeros, G)
        for i in range(bits):
            for p in range(16):
                want = math.fsum(float(x[0, j]) * (((p >> j) & 1) << i) for j in range(4))
                assert y_lut[0, 16 * i + p] == want
                assert y_def[0, 16 * i + p] == want


# ---- P2: pack / unpack round trip ------------------------------------------

@pytest.mark.parametrize("bits", [1, 2, 3, 4])
@pytest.mark.parametrize("group", [32, 64, 128])
def test_pack_unpack_roundtrip(bits, group):
    c = rand_case(1, 256, 24, bits, group, seed=bits * 10 + group)
    packed = orc.pack(c.codes, c.scales, c.zeros, bits, group)
    assert packed.size == orc.packed_bytes(256, 24, bits, group)
    q, s, z = orc.unpack(packed, 256, 24, group)
    assert np.array_equal(q, c.codes)
    assert np.array_equal(s.view(np.uint16), c.scales.view(np.uint16))
    assert np.array_equal(z, c.zeros)


def test_pack_every_code_value_roundtrips():
    for bits in (1, 2, 3, 4):
        K, N, G = 128, 8, 32
        codes = (np.arange(K * N, dtype=np.int64).reshape(K, N) * 7 % (1 << bits)).astype(np.uint8)
        assert set(np.unique(codes)) == set(range(1 << bits))
        scales = np.full((K // G, N), 0.5, dtype=np.float16)
        zeros = (np.arange(K // G * N).reshape(K // G, N) % (1 << bits)).astype(np.uint8)
        q, s, z = orc.unpack(orc.pack(codes, scales, zeros, bits, G), K, N, G)
        assert np.array_equal(q, codes) and np.array_equal(z, zeros)


def plane_bit(r):
    """Bit of a plane word that holds the weight with k % 32 == r (format description: weight
    8*ph + j sits at bit 4*j + ph)."""
    return 4 * (r & 7) + (r >> 3)


def test_plane_bit_is_a_permutation_of_the_word():
    assert sorted(plane_bit(r) for r in range(32)) == list(range(32))
    # nibble j of a word holds the weights j, 8 + j, 16 + j, 24 + j, lowest first
    for j in range(8):
        assert [plane_bit(8 * ph + j) for ph in range(4)] == [4 * j + ph for ph in range(4)]


def test_packed_plane_word_is_a_permuted_bit_plane():
    # a single set bit lands where the format description says: word (strip nb, plane i,
    # v = k/32, c = n%4), bit plane_bit(k%32); planes start at byte 256.
    K, N, G, bits = 128, 8, 32, 3
    for (k, n, code) in [(0, 0, 1), (37, 5, 4), (127, 7, 2), (64, 3, 7)]:
        codes = np.zeros((K, N), dtype=np.uint8)
        codes[k, n] = code
        packed = orc.pack(codes, np.ones((K // G, N), np.float16), np.zeros((K // G, N), np.uint8),
                          bits, G)
        words = packed[256:256 + K * N * bits // 8].view(np.uint32)
        want = np.zeros_like(words)
        for i in range(bits):
            if (code >> i) & 1:
                want[(((n // 4) * bits + i) * (K // 32) + k // 32) * 4 + n % 4] = 1 << plane_bit(k % 32)
        assert np.array_equal(words, want)


def test_packed_indices_can_be_read_out_of_plane_words():
    # bit j of the 4-bit index idx_i[t, n] (activations 4t .. 4t+3) is bit plane_bit(4*(t%8) + j) of
    # the plane word (i, t/8, n)
    c = rand_case(1, 128, 8, 4, 32, seed=3)
    idx = orc.indices(c.codes, 4)
    packed = orc.pack(c.codes, c.scales, c.zeros, 4, 32)
    words = packed[256:256 + 128 * 8 * 4 // 8].view(np.uint32)
    for i in range(4):
        for t in range(32):
            for n in range(8):
                w = int(words[(((n // 4) * 4 + i) * 4 + t // 8) * 4 + n % 4])
                got = sum(((w >> plane_bit(4 * (t % 8) + j)) & 1) << j for j in range(4))
                assert got == idx[i, t, n]


# ---- P3, P10: exact zeros --------------------------------------------------

def test_zero_codes_zero_zero_point_give_zero():
    c = rand_case(2, 256, 16, 4, 64, seed=4)
    codes = np.zeros_like(c.codes)
    zeros = np.zeros_like(c.zeros)
    assert np.all(orc.mpgemm(c.x, codes, c.scales, zeros, 64) == 0.0)
    assert np.all(orc.lut_gemv(c.x, codes, c.scales, zeros, 4, 64) == 0.0)


def test_codes_equal_zero_point_give_zero():
    c = rand_case(2, 256, 16, 3, 64, seed=5)
    codes = np.repeat(c.zeros, 64, axis=0)
    assert np.all(orc.mpgemm(c.x, codes, c.scales, c.zeros, 64) == 0.0)
    y = orc.lut_gemv(c.x, codes, c.scales, c.zeros, 3, 64)
    # the table form cancels A - z*S up to fp64 rounding of the partial sums
    assert np.max(np.abs(y)) < 1e-12


# ---- P4: linearity ---------------------------------------------------------

def test_linearity_in_activations_power_of_two_coefficients():
    c1 = rand_case(1, 256, 16, 4, 64, seed=6)
    c2 = rand_case(1, 256, 16, 4, 64, seed=7)
    x1 = c1.x
    x2 = (c2.x.astype(np.float32) * 0.25).astype(np.float16)   # exact in fp16
    # choose inputs so that 2*x1 + 0.5*x2' stays exactly representable: integers / 8
    x1 = (np.round(x1.astype(np.float32) * 8) / 8).astype(np.float16)
    x2 = (np.round(x2.astype(np.float32) * 8) / 8).astype(np.float16)
    xs = (2.0 * x1.astype(np.float64) + 0.5 * x2.astype(np.float64))
    assert np.array_equal(xs.astype(np.float16).astype(np.float64), xs)
    for fn in (lambda x: orc.mpgemm(x, c1.codes, c1.scales, c1.zeros, 64),
               lambda x: orc.lut_gemv(x, c1.codes, c1.scales, c1.zeros, 4, 64)):
        lhs = fn(xs.astype(np.float16))
        rhs = 2.0 * fn(x1) + 0.5 * fn(x2)
        assert np.allclose(lhs, rhs, rtol=1e-12, atol=1e-12)


# ---- P5-P7: values the paper prints ----------------------------------------

def test_repack_table_worked_example():
    with open(os.path.join(GOLDEN, "repack_table_example.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    for bits, plane, index_b, entry_b in rows:
        R = orc.repack_table(int(bits))
        assert int(R[int(plane), int(index_b, 2)]) == int(entry_b, 2)


def test_repack_or_over_planes_rebuilds_codes_and_counts_ops():
    # one lookup per plane nibble replaces SHIFT+AND+SHIFT for each of 4 weights (12 ops)
    R = orc.repack_table(4)
    for codes4 in itertools.product(range(16), repeat=4):
        if sum(codes4) % 5:       # thin the 65536 cases, deterministic
            continue
        acc = 0
        for i in range(4):
            nib = sum(((codes4[j] >> i) & 1) << j for j in range(4))
            acc |= int(R[i, nib])
        assert [(acc >> (4 * j)) & 0xF for j in range(4)] == list(codes4)
    assert 4 * 3 == 12


def test_affine_table_size_and_values():
    # 2^bits entries per block: INT2 -> 4 float ops, 1/16 of G=64 and 1/32 of G=128
    T = orc.affine_table(np.float16(0.5), 1, 2)
    assert T.shape == (4,)
    assert 64 // T.size == 16 and 128 // T.size == 32
    assert list(T) == [-0.5, 0.0, 0.5, 1.0]
    T4 = orc.affine_table(np.float16(0.25), 9, 4)
    assert list(T4) == [0.25 * (c - 9) for c in range(16)]


def test_vlut_table_fixes_index_width():
    with open(os.path.join(GOLDEN, "vlut_equiv_madds.txt")) as f:
        rows = [tuple(map(int, ln.split())) for ln in f if ln.strip() and not ln.startswith("#")]
    for entries, lookups, madds in rows:
        assert lookups * int(math.log2(entries)) == madds
    # a 16-entry table <=> 4 activations per lookup, which is what the oracle builds
    assert orc.luts(np.zeros((1, 32), np.float16)).shape == (1, 8, 16)


def test_two_level_dequant_equals_formula():
    c = rand_case(1, 256, 16, 4, 64, seed=8)
    w = orc.dequant_two_level(c.codes, c.scales, c.zeros, 4, 64)
    s = np.repeat(c.scales.astype(np.float64), 64, axis=0)
    z = np.repeat(c.zeros.astype(np.int64), 64, axis=0)
    assert np.array_equal(w, s * (c.codes.astype(np.int64) - z))


# ---- P8: special cases that reduce to a library routine ---------------------

@pytest.mark.parametrize("bits", [2, 3, 4])
def test_integer_case_equals_int64_matmul(bits):
    rng = np.random.default_rng(9)
    M, K, N, G = 3, 256, 24, 64
    xi = rng.integers(-8, 9, size=(M, K))
    codes = rng.integers(0, 1 << bits, size=(K, N), dtype=np.uint8)
    ones = np.ones((K // G, N), dtype=np.float16)
    zeros = np.zeros((K // G, N), dtype=np.uint8)
    want = xi.astype(np.int64) @ codes.astype(np.int64)
    x = xi.astype(np.float16)
    assert np.array_equal(orc.mpgemm(x, codes, ones, zeros, G), want.astype(np.float64))
    # P11: bit-serial identity  sum_i 2^i (x . W_i) = x . q, exact for integers
    assert np.array_equal(orc.lut_gemv(x, codes, ones, zeros, bits, G), want.astype(np.float64))
    planes = sum((1 << i) * (xi @ ((codes >> i) & 1).astype(np.int64)) for i in range(bits))
    assert np.array_equal(planes, want)


@pytest.mark.parametrize("bits,group", [(2, 64), (3, 128), (4, 32), (4, 128)])
def test_general_case_against_fp64_matmul(bits, group):
    c = rand_case(4, 512, 40, bits, group, seed=11 + bits)
    B = np.repeat(np.arange(512 // group), group)
    w = c.scales.astype(np.float64)[B] * (c.codes.astype(np.float64) - c.zeros.astype(np.float64)[B])
    want = c.x.astype(np.float64) @ w
    got = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, group)
    scale = np.max(np.abs(want))
    assert np.max(np.abs(got - want)) <= 1e-12 * scale
    got_lut = orc.lut_gemv(c.x, c.codes, c.scales, c.zeros, bits, group)
    assert np.max(np.abs(got_lut - want)) <= 1e-12 * scale


def test_rows_variant_matches_full():
    c = rand_case(6, 256, 16, 4, 64, seed=13)
    full = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, 64)
    part = orc.mpgemm_rows(c.x, c.codes, c.scales, c.zeros, 64, [5, 0, 3])
    assert np.array_equal(part, full[[5, 0, 3]])


# ---- P9: one-hot and all-ones activations -----------------------------------

def test_one_hot_activation_reads_out_each_weight():
    c = rand_case(1, 128, 8, 4, 32, seed=14)
    s64 = c.scales.astype(np.float64)
    for k in range(0, 128, 7):
        x = np.zeros((1, 128), dtype=np.float16)
        x[0, k] = 1.0
        want = s64[k // 32] * (c.codes[k].astype(np.float64) - c.zeros[k // 32])
        assert np.array_equal(orc.mpgemm(x, c.codes, c.scales, c.zeros, 32)[0], want)
        got = orc.lut_gemv(x, c.codes, c.scales, c.zeros, 4, 32)[0]
        assert np.allclose(got, want, rtol=0, atol=1e-15)


def test_ones_activation_gives_column_sums():
    c = rand_case(1, 128, 8, 3, 64, seed=15)
    x = np.ones((1, 128), dtype=np.float16)
    B = np.repeat(np.arange(2), 64)
    w = c.scales.astype(np.float64)[B] * (c.codes.astype(np.float64) - c.zeros.astype(np.float64)[B])
    assert np.allclose(orc.mpgemm(x, c.codes, c.scales, c.zeros, 64)[0], w.sum(axis=0),
                       rtol=1e-14, atol=0)


def test_transposed_operand_would_fail():
    # a non-square problem with distinct rows: y[m] depends only on x[m]
    c = rand_case(3, 128, 8, 4, 64, seed=16)
    y = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, 64)
    for m in range(3):
        ym = orc.mpgemm(c.x[m:m + 1], c.codes, c.scales, c.zeros, 64)
        assert np.array_equal(ym[0], y[m])


def test_group_boundaries_use_their_own_scale_and_zero():
    # two blocks with very different scales: a slip of the block index shows up at once
    K, N, G = 128, 4, 64
    codes = np.full((K, N), 3, dtype=np.uint8)
    scales = np.array([[1.0] * N, [16.0] * N], dtype=np.float16)
    zeros = np.array([[1] * N, [2] * N], dtype=np.uint8)
    x = np.ones((1, K), dtype=np.float16)
    want = 64 * 1.0 * (3 - 1) + 64 * 16.0 * (3 - 2)
    assert np.all(orc.mpgemm(x, codes, scales, zeros, G) == want)
    assert np.all(orc.lut_gemv(x, codes, scales, zeros, 2, G) == want)
