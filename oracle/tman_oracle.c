/*
 * CPU oracle for the low-bit-weight x fp16-activation matmul (TEST INFRASTRUCTURE).
 *
 * This file is test infrastructure: only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may call it.  It shares no code with the CUDA
 * path and is deliberately plain: triple loops, fp64, no tables, no blocking.
 *
 * What it computes (paper Sec. 2.2, "Dequantization-based low-bit inference":
 * x_dequantized = (x_quantized - zero_point) * scaling_factor, applied per
 * quantization block of `group` consecutive input channels):
 *
 *     y[m][n] = sum_k  x[m][k] * s[k/G][n] * ( q[k][n] - z[k/G][n] )
 *
 * with x and s converted exactly from fp16 to fp64, q and z integers.
 *
 * It also contains a step-by-step fp64 evaluator of the bit-serial table-lookup
 * form (Sec. 2.2 "Bit-serial table lookup", Fig. 2; Sec. 4.3 two-level tiling:
 * aggregate inside the quantization block, scale, aggregate across blocks) used
 * to check the oracle against itself, and the packed-layout writer/reader that
 * the packed-buffer format description fixes.
 *
 * Pins (see tests): closed forms, integer special cases against an int64
 * matmul, one-hot activations, linearity, zero codes, the paper's worked
 * repack-table entry.  Accumulation order and table precision of the GPU path
 * are "parity unpinned" beyond the 5e-3 relative bound.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* exact fp16 (IEEE binary16 bit pattern) -> fp64 */
static double half_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int exp = (h >> 10) & 0x1f;
    int man = h & 0x3ff;
    double v;
    if (exp == 0) {
        v = (double)man / 1024.0 / 16384.0;              /* subnormal: man * 2^-24 */
    } else if (exp == 31) {
        v = man ? (0.0 / 0.0) : (1.0 / 0.0);
    } else {
        double m = 1.0 + (double)man / 1024.0;
        int e = exp - 15;
        double p = 1.0;
        int i;
        if (e >= 0) for (i = 0; i < e; ++i) p *= 2.0;
        else        for (i = 0; i < -e; ++i) p *= 0.5;
        v = m * p;
    }
    return sign ? -v : v;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* The definition (Sec. 2.2).  x: fp16 bits [M][K]; q: [K][N]; s: fp16 bits [K/G][N];
 * z: [K/G][N]; y: fp64 [M][N].  Threads split the (m, n) outputs; each output is one
 * plain loop over k in increasing order. */
void oracle_mpgemm(const uint16_t *x, const uint8_t *q, const uint16_t *s, const uint8_t *z,
                   int M, int K, int N, int G, double *y)
{
    long mn;
#pragma omp parallel for schedule(static)
    for (mn = 0; mn < (long)M * N; ++mn) {
        int m = (int)(mn / N), n = (int)(mn % N);
        double acc = 0.0;
        int k;
        for (k = 0; k < K; ++k) {
            int B = k / G;
            double w = half_to_double(s[(size_t)B * N + n]) *
                       (double)((int)q[(size_t)k * N + n] - (int)z[(size_t)B * N + n]);
            acc += half_to_double(x[(size_t)m * K + k]) * w;
        }
        y[mn] = acc;
    }
}

/* Same definition restricted to chosen output rows (for sampled parity at large M). */
void oracle_mpgemm_rows(const uint16_t *x, const uint8_t *q, const uint16_t *s, const uint8_t *z,
                        const int *rows, int n_rows, int K, int N, int G, double *y)
{
    long rn;
#pragma omp parallel for schedule(static)
    for (rn = 0; rn < (long)n_rows * N; ++rn) {
        int r = (int)(rn / N), n = (int)(rn % N);
        int m = rows[r];
        double acc = 0.0;
        int k;
        for (k = 0; k < K; ++k) {
            int B = k / G;
            double w = half_to_double(s[(size_t)B * N + n]) *
                       (double)((int)q[(size_t)k * N + n] - (int)z[(size_t)B * N + n]);
            acc += half_to_double(x[(size_t)m * K + k]) * w;
        }
        y[rn] = acc;
    }
}

/* ---- bit-serial table-lookup evaluator, step by step (Sec. 2.2, Fig. 2; Sec. 4.3) ---- */

/* step 1+2: one-bit planes W_i = (q >> i) & 1 and the 4-bit index per plane:
 * idx[i][t][n] = sum_{j<4} W_i[4t+j][n] << j   (Sec. 4.1 "4-bit LUT index") */
void oracle_indices(const uint8_t *q, int K, int N, int bits, uint8_t *idx)
{
    int i, t, n, j;
    for (i = 0; i < bits; ++i)
        for (t = 0; t < K / 4; ++t)
            for (n = 0; n < N; ++n) {
                unsigned v = 0;
                for (j = 0; j < 4; ++j)
                    v |= (unsigned)((q[(size_t)(4 * t + j) * N + n] >> i) & 1) << j;
                idx[((size_t)i * (K / 4) + t) * N + n] = (uint8_t)v;
            }
}

/* step 3: activation tables, lut[m][t][p] = sum_{j<4} x[m][4t+j] * bit_j(p)  (Sec. 2.2) */
void oracle_luts(const uint16_t *x, int M, int K, double *lut)
{
    int m, t, p, j;
    for (m = 0; m < M; ++m)
        for (t = 0; t < K / 4; ++t)
            for (p = 0; p < 16; ++p) {
                double a = 0.0;
                for (j = 0; j < 4; ++j)
                    if ((p >> j) & 1) a += half_to_double(x[(size_t)m * K + 4 * t + j]);
                lut[((size_t)m * (K / 4) + t) * 16 + p] = a;
            }
}

/* steps 4+5: lookups, shift-accumulate inside the block, scale and zero-point per block,
 * fp accumulation across blocks (Sec. 4.3).  idx and lut as produced above. */
void oracle_lut_gemv(const uint8_t *idx, const double *lut, const uint16_t *x,
                     const uint16_t *s, const uint8_t *z,
                     int M, int K, int N, int bits, int G, double *y)
{
    int m, n, B, i, t, k;
    for (m = 0; m < M; ++m)
        for (n = 0; n < N; ++n) {
            double acc = 0.0;
            for (B = 0; B < K / G; ++B) {
                double A = 0.0, S = 0.0;
                for (i = 0; i < bits; ++i) {
                    double P = 0.0;
                    for (t = B * G / 4; t < (B + 1) * G / 4; ++t)
                        P += lut[((size_t)m * (K / 4) + t) * 16 +
                                 idx[((size_t)i * (K / 4) + t) * N + n]];
                    A += (double)(1 << i) * P;
                }
                for (k = B * G; k < (B + 1) * G; ++k)
                    S += half_to_double(x[(size_t)m * K + k]);
                acc += half_to_double(s[(size_t)B * N + n]) *
                       (A - (double)z[(size_t)B * N + n] * S);
            }
            y[(size_t)m * N + n] = acc;
        }
}

/* ---- two-level lookup dequantization (Sec. 4.1, Fig. 7) ---- */

/* level 1: repack table of plane i: a 4-bit slice of plane i (bit i of 4 weights)
 * -> 16-bit word with that bit placed at position i of each weight's 4-bit field. */
void oracle_repack_table(int bits, uint16_t *R /* [bits][16] */)
{
    int i, p, j;
    for (i = 0; i < bits; ++i)
        for (p = 0; p < 16; ++p) {
            unsigned v = 0;
            for (j = 0; j < 4; ++j)
                v |= (unsigned)((p >> j) & 1) << (4 * j + i);
            R[i * 16 + p] = (uint16_t)v;
        }
}

/* level 2: affine table of one (block, column): T[c] = s * (c - z), 2^bits entries. */
void oracle_affine_table(uint16_t s, uint8_t z, int bits, double *T)
{
    int c;
    for (c = 0; c < (1 << bits); ++c)
        T[c] = half_to_double(s) * (double)(c - (int)z);
}

/* rebuild the dequantized weights through the two tables: codes4 = OR_i R_i[idx_i],
 * w[4t+j][n] = T_{B,n}[ nibble j of codes4 ]. */
void oracle_dequant_two_level(const uint8_t *idx, const uint16_t *s, const uint8_t *z,
                              int K, int N, int bits, int G, double *w /* [K][N] */)
{
    uint16_t R[4 * 16];
    double T[16];
    int t, n, i, j;
    oracle_repack_table(bits, R);
    for (t = 0; t < K / 4; ++t)
        for (n = 0; n < N; ++n) {
            unsigned codes4 = 0;
            int B = (4 * t) / G;
            for (i = 0; i < bits; ++i)
                codes4 |= R[i * 16 + idx[((size_t)i * (K / 4) + t) * N + n]];
            oracle_affine_table(s[(size_t)B * N + n], z[(size_t)B * N + n], bits, T);
            for (j = 0; j < 4; ++j)
                w[(size_t)(4 * t + j) * N + n] = T[(codes4 >> (4 * j)) & 0xf];
        }
}

/* ---- packed buffer (format description: 256-byte header, bit-plane words, strip-major
 *      scales, nibble-packed zero-points) ---- */

#define ORACLE_HDR_BYTES 256
static size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

size_t oracle_packed_bytes(int K, int N, int bits, int G)
{
    size_t planes = (size_t)K * N * bits / 8;
    size_t scales = (size_t)(K / G) * N * 2;
    size_t zeros = (size_t)(K / G) * (N / 4) * 2;
    return ORACLE_HDR_BYTES + up256(planes) + up256(scales) + up256(zeros);
}

/* Bit position, inside a plane word, of the weight with k % 32 == r.  The 32 weights of a word are
 * stored permuted (paper Sec. 4.1: weights are permuted offline so that the on-the-fly repacking of
 * the prefill path is cheap): weight r = 8*ph + j sits at bit 4*j + ph, so that the four nibble-packed
 * code words of the repacking step come out in consecutive-k order. */
static int plane_bit(int r) { return 4 * (r & 7) + (r >> 3); }

static void put32(uint8_t *p, uint32_t v) { memcpy(p, &v, 4); }
static void put64(uint8_t *p, uint64_t v) { memcpy(p, &v, 8); }

void oracle_pack(const uint8_t *q, const uint16_t *s, const uint8_t *z,
                 int K, int N, int bits, int G, uint8_t *out)
{
    size_t planes = (size_t)K * N * bits / 8;
    size_t scales = (size_t)(K / G) * N * 2;
    size_t planes_off = ORACLE_HDR_BYTES;
    size_t scales_off = planes_off + up256(planes);
    size_t zeros_off = scales_off + up256(scales);
    size_t total = oracle_packed_bytes(K, N, bits, G);
    int nb, i, v, c, r, B;
    memset(out, 0, total);
    memcpy(out, "TMANB200", 8);
    put32(out + 8, 2);
    put32(out + 12, (uint32_t)K);
    put32(out + 16, (uint32_t)N);
    put32(out + 20, (uint32_t)bits);
    put32(out + 24, (uint32_t)G);
    put32(out + 28, 4);
    put64(out + 32, planes_off);
    put64(out + 40, scales_off);
    put64(out + 48, zeros_off);
    put64(out + 56, total);
    /* plane words: bit plane_bit(r) of word (strip nb, plane i, v, c) = bit i of q[32v + r][4nb + c] */
    for (nb = 0; nb < N / 4; ++nb)
        for (i = 0; i < bits; ++i)
            for (v = 0; v < K / 32; ++v)
                for (c = 0; c < 4; ++c) {
                    uint32_t w = 0;
                    for (r = 0; r < 32; ++r)
                        w |= (uint32_t)((q[(size_t)(32 * v + r) * N + 4 * nb + c] >> i) & 1) << plane_bit(r);
                    put32(out + planes_off +
                          4 * ((((size_t)nb * bits + i) * (K / 32) + v) * 4 + c), w);
                }
    for (nb = 0; nb < N / 4; ++nb)
        for (B = 0; B < K / G; ++B) {
            uint16_t zz = 0;
            for (c = 0; c < 4; ++c) {
                uint16_t sv = s[(size_t)B * N + 4 * nb + c];
                memcpy(out + scales_off + 2 * (((size_t)nb * (K / G) + B) * 4 + c), &sv, 2);
                zz |= (uint16_t)((z[(size_t)B * N + 4 * nb + c] & 0xf) << (4 * c));
            }
            memcpy(out + zeros_off + 2 * ((size_t)nb * (K / G) + B), &zz, 2);
        }
}

/* returns 0 on success, nonzero if the header is not a valid one */
int oracle_unpack(const uint8_t *in, uint8_t *q, uint16_t *s, uint8_t *z)
{
    uint32_t ver, K, N, bits, G;
    uint64_t planes_off, scales_off, zeros_off;
    uint32_t nb, i, v, c, r, B;
    if (memcmp(in, "TMANB200", 8) != 0) return 1;
    memcpy(&ver, in + 8, 4);
    memcpy(&K, in + 12, 4);
    memcpy(&N, in + 16, 4);
    memcpy(&bits, in + 20, 4);
    memcpy(&G, in + 24, 4);
    memcpy(&planes_off, in + 32, 8);
    memcpy(&scales_off, in + 40, 8);
    memcpy(&zeros_off, in + 48, 8);
    if (ver != 2) return 2;
    memset(q, 0, (size_t)K * N);
    for (nb = 0; nb < N / 4; ++nb)
        for (i = 0; i < bits; ++i)
            for (v = 0; v < K / 32; ++v)
                for (c = 0; c < 4; ++c) {
                    uint32_t w;
                    memcpy(&w, in + planes_off +
                           4 * ((((size_t)nb * bits + i) * (K / 32) + v) * 4 + c), 4);
                    for (r = 0; r < 32; ++r)
                        q[(size_t)(32 * v + r) * N + 4 * nb + c] |=
                            (uint8_t)(((w >> plane_bit((int)r)) & 1) << i);
                }
    for (nb = 0; nb < N / 4; ++nb)
        for (B = 0; B < K / G; ++B) {
            uint16_t zz;
            memcpy(&zz, in + zeros_off + 2 * ((size_t)nb * (K / G) + B), 2);
            for (c = 0; c < 4; ++c) {
                memcpy(&s[(size_t)B * N + 4 * nb + c],
                       in + scales_off + 2 * (((size_t)nb * (K / G) + B) * 4 + c), 2);
                z[(size_t)B * N + 4 * nb + c] = (uint8_t)((zz >> (4 * c)) & 0xf);
            }
        }
    return 0;
}
