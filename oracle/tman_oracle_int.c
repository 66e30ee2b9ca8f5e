/*
 * CPU oracle for the integer path of the table-lookup matmul (TEST INFRASTRUCTURE): per-tensor
 * ternary weights with integer activations.
 *
 * This file is test infrastructure: only the test-suite, the smoke check and the benchmark's
 * CPU-baseline leg may call it.  It shares no code with the CUDA path; plain loops, exact integers.
 *
 * What it covers (paper Sec. 6.1 "Models and Quantization": BitNet's ternary weights are quantized per
 * tensor and treated as 2-bit, with 16-bit integer activations; Sec. 4.3: low-precision aggregation
 * inside the quantization block, floating point across blocks; Sec. 6.2 "mpGEMM": for prefill the
 * per-tensor weights are dequantized to INT8 for the matrix unit):
 *
 *   weights      w[k][n] = s_w * t[k][n],  t in {-1, 0, +1},  stored as the 2-bit code q = t + 1
 *                (one scale s_w for the whole tensor; zero-point 1)
 *   activations  a[m][k] = round(x[m][k] / s_a[m]),  s_a[m] = max_k |x[m][k]| / QMAX
 *                (QMAX = 32767 for 16-bit decode, 127 for 8-bit prefill; both divisions in single
 *                 precision, x/s_a rounded to nearest, ties to even; a row of zeros has s_a = 1, a = 0)
 *   result       y[m][n] = s_a[m] * s_w * sum_k a[m][k] * t[k][n]      (the sum is an exact integer)
 *
 * Readings taken where the paper is silent: the activation scale is per token (row) and symmetric;
 * the scale and the quotient are single-precision values and rounding is to nearest even; the table entries of the bit-serial form are exact integer sums of four
 * activations; with one block per tensor the "inside the block" aggregation is the whole integer sum.
 *
 * Pins (see tests): the bit-serial table form equals the definition bit for bit; brute force on tiny
 * inputs; all-plus-one / all-zero / one-hot closed forms; the quantization error bound against the
 * fp64 product; the per-block oracle on the same weights written as 2-bit codes with zero-point 1.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

/* exact fp16 (IEEE binary16 bit pattern) -> fp64 */
static double h2d(uint16_t h)
{
    int sign = (h >> 15) & 1, exp = (h >> 10) & 0x1f, man = h & 0x3ff;
    double v;
    if (exp == 0) v = ldexp((double)man, -24);
    else if (exp == 31) v = man ? (0.0 / 0.0) : (1.0 / 0.0);
    else v = ldexp(1.0 + (double)man / 1024.0, exp - 15);
    return sign ? -v : v;
}

/* Per-token symmetric quantization of the activations (Sec. 6.1: A_INT16; INT8 for the matrix unit).
 * The scale and the quotient are computed in single precision (IEEE division, correctly rounded) and the
 * quotient is rounded to the nearest integer, ties to even: floating point decides an integer here, so
 * the precision is part of the definition, and single precision is what an accelerator kernel uses.
 * x: fp16 bits [M][K]; a: int32 [M][K] (values within +-qmax); s_a: fp64 [M] (holding the fp32 value). */
void oracle_quantize_rows(const uint16_t *x, int M, int K, int qmax, int32_t *a, double *s_a)
{
    int m, k;
    for (m = 0; m < M; ++m) {
        float amax = 0.0f, scale;
        for (k = 0; k < K; ++k) {
            float v = fabsf((float)h2d(x[(size_t)m * K + k]));       /* fp16 -> fp32 is exact */
            if (v > amax) amax = v;
        }
        scale = amax > 0.0f ? amax / (float)qmax : 1.0f;
        s_a[m] = (double)scale;
        for (k = 0; k < K; ++k) {
            volatile float quot = (float)h2d(x[(size_t)m * K + k]) / scale;   /* one rounding, to fp32 */
            float r = nearbyintf(quot);                                        /* default mode: ties to even */
            if (r > (float)qmax) r = (float)qmax;
            if (r < -(float)qmax) r = -(float)qmax;
            a[(size_t)m * K + k] = (int32_t)r;
        }
    }
}

/* The definition: acc[m][n] = sum_k a[m][k] * (q[k][n] - 1), exact in int64.  q: codes [K][N] in {0,1,2}. */
void oracle_ternary_matmul(const int32_t *a, const uint8_t *q, int M, int K, int N, int64_t *acc)
{
    int m, n, k;
#pragma omp parallel for private(n, k) schedule(static)
    for (m = 0; m < M; ++m)
        for (n = 0; n < N; ++n) {
            int64_t s = 0;
            for (k = 0; k < K; ++k) s += (int64_t)a[(size_t)m * K + k] * ((int)q[(size_t)k * N + n] - 1);
            acc[(size_t)m * N + n] = s;
        }
}

/* The bit-serial table form with integer tables (Sec. 2.2, Fig. 2, on integer activations):
 *   planes   W_i[k][n] = (q[k][n] >> i) & 1, i in {0, 1}
 *   index    idx_i[t][n] = sum_{j<4} W_i[4t+j][n] << j
 *   table    lut[m][t][p] = sum_{j<4} a[m][4t+j] * bit_j(p)                 (exact integers)
 *   result   acc[m][n] = sum_i 2^i * sum_t lut[m][t][idx_i[t][n]]  -  1 * sum_k a[m][k]
 * the last term being the zero-point (1) times the activation sum of the one block. */
void oracle_ternary_lut_matmul(const int32_t *a, const uint8_t *q, int M, int K, int N, int64_t *acc)
{
    int m, n, t, i, j, p;
    for (m = 0; m < M; ++m) {
        int64_t asum = 0;
        for (t = 0; t < K; ++t) asum += a[(size_t)m * K + t];
        for (n = 0; n < N; ++n) {
            int64_t total = 0;
            for (i = 0; i < 2; ++i) {
                int64_t plane = 0;
                for (t = 0; t < K / 4; ++t) {
                    int64_t lut[16];
                    unsigned idx = 0;
                    for (p = 0; p < 16; ++p) {
                        lut[p] = 0;
                        for (j = 0; j < 4; ++j)
                            if ((p >> j) & 1) lut[p] += a[(size_t)m * K + 4 * t + j];
                    }
                    for (j = 0; j < 4; ++j) idx |= (unsigned)((q[(size_t)(4 * t + j) * N + n] >> i) & 1) << j;
                    plane += lut[idx];
                }
                total += plane * (int64_t)(1 << i);
            }
            acc[(size_t)m * N + n] = total - asum;
        }
    }
}

/* Two-level lookup dequantization to INT8 (Sec. 4.1, Fig. 7, with an integer second table; Sec. 6.2):
 * level 1 places bit i of four weights into their 4-bit fields (the repack table), level 2 maps a code
 * to its value, here T[c] = c - 1 for c in {0, 1, 2} (code 3 does not occur; it maps to 0).
 * w8: int8 [K][N]. */
void oracle_ternary_dequant_int8(const uint8_t *q, int K, int N, int8_t *w8)
{
    static const int8_t T[4] = {-1, 0, 1, 0};
    int t, n, i, j;
    for (t = 0; t < K / 4; ++t)
        for (n = 0; n < N; ++n) {
            unsigned codes4 = 0;
            for (i = 0; i < 2; ++i) {
                unsigned idx = 0, rep = 0;
                for (j = 0; j < 4; ++j) idx |= (unsigned)((q[(size_t)(4 * t + j) * N + n] >> i) & 1) << j;
                for (j = 0; j < 4; ++j) rep |= ((idx >> j) & 1u) << (4 * j + i);      /* repack table entry */
                codes4 |= rep;
            }
            for (j = 0; j < 4; ++j) w8[(size_t)(4 * t + j) * N + n] = T[(codes4 >> (4 * j)) & 3u];
        }
}

/* Prefill on the dequantized INT8 weights: acc[m][n] = sum_k a8[m][k] * w8[k][n], exact. */
void oracle_int8_matmul(const int32_t *a8, const int8_t *w8, int M, int K, int N, int64_t *acc)
{
    int m, n, k;
#pragma omp parallel for private(n, k) schedule(static)
    for (m = 0; m < M; ++m)
        for (n = 0; n < N; ++n) {
            int64_t s = 0;
            for (k = 0; k < K; ++k) s += (int64_t)a8[(size_t)m * K + k] * (int64_t)w8[(size_t)k * N + n];
            acc[(size_t)m * N + n] = s;
        }
}

/* y[m][n] = s_a[m] * s_w * acc[m][n] in fp64 (floating point only after the integer aggregation, Sec. 4.3). */
void oracle_scale_result(const int64_t *acc, const double *s_a, double s_w, int M, int N, double *y)
{
    int m, n;
    for (m = 0; m < M; ++m)
        for (n = 0; n < N; ++n) y[(size_t)m * N + n] = s_a[m] * s_w * (double)acc[(size_t)m * N + n];
}
