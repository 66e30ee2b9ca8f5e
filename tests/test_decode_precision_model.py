"""Predicted error of the decode path with several activation rows, simulated on the CPU.

With two or more rows the decode kernel stores table entries as fp16 (two rows per 32-bit slot) and
adds the lookups of one 32-activation word -- bits x 4 of them, low plane first, each times 2^plane --
in fp16; the rows of a K-slice are first scaled by a power of two so that the largest magnitude lies in
[1, 2).  Everything after a word's sum is fp32.  This file replays exactly that arithmetic in NumPy
(float16 operations round after every step, as the kernel's do) and checks that the error it predicts
stays several times below the 5e-3 bound the GPU tests use; the GPU tests in test_mpgemv_gpu.py then
hold the kernel to a bound derived from this prediction.
"""
import numpy as np
import pytest

from oracle import tman_oracle as orc
from paper_2511_11248_b200 import synth

PREDICTED_BOUND = 1.5e-3      # what the simulation must stay below (the kernel's tolerance is 5e-3)


def simulate_rows_fp16(c, slice_words):
    M, K, N, bits, G = c.M, c.K, c.N, c.bits, c.group
    x = c.x.astype(np.float32)
    q = c.codes.astype(np.int64)
    s = c.scales.astype(np.float32)
    z = c.zeros.astype(np.float32)
    out = np.zeros((M, N), dtype=np.float32)
    nwords = K // 32
    for m in range(M):
        acc_blocks = np.zeros((K // G, N), dtype=np.float32)      # s * (A - z * S) is linear in the words
        ssum = np.zeros(K // G, dtype=np.float32)
        rs_of_word = np.zeros(nwords, dtype=np.float32)
        for w in range(nwords):
            sl = w // slice_words                                  # the K-slice (one CTA) of this word
            xs = x[m, 32 * sl * slice_words: 32 * min(nwords, (sl + 1) * slice_words)]
            amax = np.abs(xs).max()
            e = np.floor(np.log2(amax)) if amax > 0 else 0.0
            inv, rs = np.float32(2.0 ** -e), np.float32(2.0 ** e)
            rs_of_word[w] = rs
            xw = x[m, 32 * w: 32 * w + 32] * inv
            h = np.zeros(N, dtype=np.float16)
            ss = np.float32(0)
            for i in range(bits):                                  # low plane first
                bit = ((q[32 * w: 32 * w + 32, :] >> i) & 1).astype(np.float32)
                for eb in range(4):                                # index byte eb: activations 8*ph + 2*eb + hi
                    ks = [8 * ph + 2 * eb + hi for hi in range(2) for ph in range(4)]
                    entry = (bit[ks, :] * xw[ks, None]).sum(axis=0, dtype=np.float32).astype(np.float16)
                    h = (entry.astype(np.float32) * np.float32(2 ** i) + h.astype(np.float32)).astype(np.float16)
            for eb in range(4):
                ks = [8 * ph + 2 * eb + hi for hi in range(2) for ph in range(4)]
                ss += np.float32(np.float16(xw[ks].sum(dtype=np.float32)))     # the all-ones entries
            B = (32 * w) // G
            # scaled back per word here (the kernel scales a slice's sum back once; same value: powers of two)
            acc_blocks[B] += h.astype(np.float32) * rs
            ssum[B] += ss * rs
        out[m] = (s * (acc_blocks - z * ssum[:, None])).sum(axis=0, dtype=np.float32)
    return out.astype(np.float16).astype(np.float64)


@pytest.mark.parametrize("M,K,N,bits,G,words,outliers", [
    (2, 2048, 64, 4, 128, 32, False), (2, 2048, 64, 2, 64, 32, False), (4, 2048, 48, 3, 32, 16, False),
    (8, 1024, 48, 4, 64, 8, False), (2, 2048, 64, 4, 128, 32, True),
])
def test_predicted_error_of_fp16_row_tables(M, K, N, bits, G, words, outliers):
    c = synth.small_case(M, K, N, bits, G, seed=5, outliers=outliers)
    ref = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, c.group)
    got = simulate_rows_fp16(c, words)
    err = float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))
    assert err <= PREDICTED_BOUND, err


def test_scaling_makes_the_prediction_independent_of_magnitude():
    # tiny and huge activations (fp16 subnormals would lose bits, sums would overflow) behave like unit ones
    errs = []
    for factor in (2.0 ** -12, 1.0, 2.0 ** 9):
        c = synth.small_case(2, 1024, 32, 4, 64, seed=6)
        c.x[:] = (c.x.astype(np.float32) * factor).astype(np.float16)
        ref = orc.mpgemm(c.x, c.codes, c.scales, c.zeros, c.group)
        errs.append(float(np.max(np.abs(simulate_rows_fp16(c, 32) - ref)) / np.max(np.abs(ref))))
    assert max(errs) <= PREDICTED_BOUND and max(errs) <= 1.5 * min(errs) + 2e-4
