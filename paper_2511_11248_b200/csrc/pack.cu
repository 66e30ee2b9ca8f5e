// Offline repack into the bit-plane layout, its inverse, and the test-only extractors.
// Pure integer work; every result has exactly one correct value.
#include "common.cuh"
#include <algorithm>
#include <mutex>
#include <vector>

namespace tman {

// One thread per (v, n): reads the 32 codes q[32v .. 32v+31][n] (coalesced across n) and writes
// one word per bit-plane (paper Sec. 2.2: W = sum_i 2^i W_i with one-bit W_i).
__global__ void pack_planes_kernel(const uint8_t *__restrict__ codes, uint32_t *__restrict__ planes,
                                   int K, int N, int bits)
{
    long tid = (long)blockIdx.x * blockDim.x + threadIdx.x;
    long total = (long)(K / 32) * N;
    if (tid >= total) return;
    int n = (int)(tid % N);
    int v = (int)(tid / N);
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    for (int r = 0; r < 32; ++r) {
        uint32_t q = codes[(size_t)(32 * v + r) * N + n];
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] |= ((q >> i) & 1u) << plane_bit(r);
    }
    int nb = n >> 2, c = n & 3;
    for (int i = 0; i < bits; ++i)
        planes[(((size_t)nb * bits + i) * (K / 32) + v) * 4 + c] = w[i];
}

// One thread per (strip, block): four scales and the four zero-point nibbles.
__global__ void pack_scales_kernel(const __half *__restrict__ scales, const uint8_t *__restrict__ zeros,
                                   __half *__restrict__ out_s, uint16_t *__restrict__ out_z,
                                   int K, int N, int group)
{
    long tid = (long)blockIdx.x * blockDim.x + threadIdx.x;
    int nblk = K / group;
    long total = (long)(N / 4) * nblk;
    if (tid >= total) return;
    int B = (int)(tid % nblk);
    int nb = (int)(tid / nblk);
    uint32_t zz = 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        out_s[((size_t)nb * nblk + B) * 4 + c] = scales[(size_t)B * N + 4 * nb + c];
        zz |= (uint32_t)(zeros[(size_t)B * N + 4 * nb + c] & 0xF) << (4 * c);
    }
    out_z[(size_t)nb * nblk + B] = (uint16_t)zz;
}

__global__ void write_header_kernel(uint8_t *packed, int K, int N, int bits, int group)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    Layout L = make_layout(K, N, bits, group);
    uint32_t *h32 = reinterpret_cast<uint32_t *>(packed);
    for (int i = 0; i < (int)(kHeaderBytes / 4); ++i) h32[i] = 0;
    h32[0] = 0x4E414D54u;   // "TMAN"
    h32[1] = 0x30303242u;   // "B200"
    h32[2] = kVersion;
    h32[3] = (uint32_t)K;
    h32[4] = (uint32_t)N;
    h32[5] = (uint32_t)bits;
    h32[6] = (uint32_t)group;
    h32[7] = 4u;
    uint64_t *h64 = reinterpret_cast<uint64_t *>(packed);
    h64[4] = L.planes_off;
    h64[5] = L.scales_off;
    h64[6] = L.zeros_off;
    h64[7] = L.total;
}

// Zero the padding between sections so that the whole buffer is a function of the inputs.
__global__ void zero_padding_kernel(uint8_t *packed, int K, int N, int bits, int group)
{
    Layout L = make_layout(K, N, bits, group);
    size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;   // < 768
    size_t a0 = L.planes_off + L.planes_bytes, a1 = L.scales_off;
    size_t b0 = L.scales_off + L.scales_bytes, b1 = L.zeros_off;
    size_t c0 = L.zeros_off + L.zeros_bytes, c1 = L.total;
    if (tid < 256) { if (a0 + tid < a1) packed[a0 + tid] = 0; }
    else if (tid < 512) { size_t t = tid - 256; if (b0 + t < b1) packed[b0 + t] = 0; }
    else { size_t t = tid - 512; if (c0 + t < c1) packed[c0 + t] = 0; }
}

// Streams on which a packed buffer has been written since the last decode launch.  The decode kernel
// reads weights before it waits for its predecessor when launched with programmatic stream
// serialization, so launch_mpgemv asks here and falls back to plain stream order once after a pack.
static std::mutex g_pending_mutex;
static std::vector<cudaStream_t> g_pending_streams;

void note_packed_write(cudaStream_t s)
{
    std::lock_guard<std::mutex> lock(g_pending_mutex);
    if (std::find(g_pending_streams.begin(), g_pending_streams.end(), s) == g_pending_streams.end())
        g_pending_streams.push_back(s);
}

bool packed_write_pending(cudaStream_t s, bool clear)
{
    std::lock_guard<std::mutex> lock(g_pending_mutex);
    auto it = std::find(g_pending_streams.begin(), g_pending_streams.end(), s);
    if (it == g_pending_streams.end()) return false;
    if (clear) g_pending_streams.erase(it);
    return true;
}

tman_status launch_pack(const uint8_t *codes, const void *scales, const uint8_t *zeros, int K, int N,
                        int bits, int group, void *packed, cudaStream_t s)
{
    Layout L = make_layout(K, N, bits, group);
    uint8_t *p = static_cast<uint8_t *>(packed);
    write_header_kernel<<<1, 32, 0, s>>>(p, K, N, bits, group);
    zero_padding_kernel<<<3, 256, 0, s>>>(p, K, N, bits, group);
    long t1 = (long)(K / 32) * N;
    pack_planes_kernel<<<(unsigned)((t1 + 255) / 256), 256, 0, s>>>(
        codes, reinterpret_cast<uint32_t *>(p + L.planes_off), K, N, bits);
    long t2 = (long)(N / 4) * (K / group);
    pack_scales_kernel<<<(unsigned)((t2 + 255) / 256), 256, 0, s>>>(
        static_cast<const __half *>(scales), zeros, reinterpret_cast<__half *>(p + L.scales_off),
        reinterpret_cast<uint16_t *>(p + L.zeros_off), K, N, group);
    note_packed_write(s);
    return launch_status();
}

// ---- inverse -----------------------------------------------------------------------------
__global__ void unpack_kernel(const uint8_t *__restrict__ packed, uint8_t *__restrict__ codes,
                              __half *__restrict__ scales, uint8_t *__restrict__ zeros,
                              uint32_t *status, int K, int N, int bits, int group)
{
    if (!header_matches(packed, K, N, bits, group)) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(status, 0u, (uint32_t)TMAN_ERR_BAD_PACKED);
        return;
    }
    Layout L = make_layout(K, N, bits, group);
    const uint32_t *planes = reinterpret_cast<const uint32_t *>(packed + L.planes_off);
    long tid = (long)blockIdx.x * blockDim.x + threadIdx.x;
    long total = (long)(K / 32) * N;
    if (tid < total) {
        int n = (int)(tid % N), v = (int)(tid / N);
        int nb = n >> 2, c = n & 3;
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        for (int i = 0; i < bits; ++i) w[i] = planes[(((size_t)nb * bits + i) * (K / 32) + v) * 4 + c];
        for (int r = 0; r < 32; ++r) {
            uint32_t q = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) q |= ((w[i] >> plane_bit(r)) & 1u) << i;
            codes[(size_t)(32 * v + r) * N + n] = (uint8_t)q;
        }
    }
    int nblk = K / group;
    if (tid < (long)nblk * N) {
        int n = (int)(tid % N), B = (int)(tid / N);
        int nb = n >> 2, c = n & 3;
        const __half *ps = reinterpret_cast<const __half *>(packed + L.scales_off);
        const uint16_t *pz = reinterpret_cast<const uint16_t *>(packed + L.zeros_off);
        scales[(size_t)B * N + n] = ps[((size_t)nb * nblk + B) * 4 + c];
        zeros[(size_t)B * N + n] = (uint8_t)((pz[(size_t)nb * nblk + B] >> (4 * c)) & 0xF);
    }
}

tman_status launch_unpack(const void *packed, int K, int N, int bits, int group, uint8_t *codes,
                          void *scales, uint8_t *zeros, uint32_t *status, cudaStream_t s)
{
    long total = (long)(K / 32) * N;   // >= (K/group)*N because group >= 32
    unpack_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(
        static_cast<const uint8_t *>(packed), codes, static_cast<__half *>(scales), zeros, status,
        K, N, bits, group);
    return launch_status();
}

// ---- test-only extractors ------------------------------------------------------------------
// idx[i][t][n] = the 4-bit table index of activations 4t .. 4t+3 (plane i, column n), gathered from
// the bits of plane word (i, t / 8, n) that hold those four weights.
__global__ void debug_indices_kernel(const uint8_t *__restrict__ packed, uint8_t *__restrict__ idx,
                                     uint32_t *status, int K, int N, int bits, int group)
{
    if (!header_matches(packed, K, N, bits, group)) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(status, 0u, (uint32_t)TMAN_ERR_BAD_PACKED);
        return;
    }
    Layout L = make_layout(K, N, bits, group);
    const uint32_t *planes = reinterpret_cast<const uint32_t *>(packed + L.planes_off);
    long tid = (long)blockIdx.x * blockDim.x + threadIdx.x;
    long total = (long)bits * (K / 32) * N;
    if (tid >= total) return;
    int n = (int)(tid % N);
    long r = tid / N;
    int v = (int)(r % (K / 32));
    int i = (int)(r / (K / 32));
    uint32_t w = planes[(((size_t)(n >> 2) * bits + i) * (K / 32) + v) * 4 + (n & 3)];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        uint32_t x = 0;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) x |= ((w >> plane_bit(4 * e + jj)) & 1u) << jj;
        idx[((size_t)i * (K / 4) + 8 * v + e) * N + n] = (uint8_t)x;
    }
}

// ---- per-tensor ternary weights -> INT8 by two table lookups (paper Sec. 4.1 / Fig. 7, Sec. 6.2) -----------
// One thread takes the two plane words of 32 consecutive k of the four columns of a strip.  Level 1 (bit
// repacking): the planes are interleaved into 2-bit codes, eight to a register in k order, one code per
// nibble (the packed format's bit permutation makes a shift and a bit-select do it).  Level 2 (conversion
// table): a four-entry byte table {-1, 0, +1, 0} held in one register, looked up four codes at a time with
// a byte permute whose selector is the codes themselves.  Output: int8 [N][K], 32 bytes per thread and
// column, consecutive threads on consecutive k.
__global__ void dequant_ternary_int8_kernel(const uint8_t *__restrict__ packed, int8_t *__restrict__ w8,
                                            uint32_t *status, int K, int N, int group)
{
    if (!header_matches(packed, K, N, 2, group)) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(status, 0u, (uint32_t)TMAN_ERR_BAD_PACKED);
        return;
    }
    const Layout L = make_layout(K, N, 2, group);
    const int words = K / 32;
    const long tid = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (tid >= (long)(N / 4) * words) return;
    const int nb = (int)(tid / words), v = (int)(tid % words);
    const uint4 *planes = reinterpret_cast<const uint4 *>(packed + L.planes_off);
    const uint4 w0 = __ldg(planes + ((size_t)nb * 2 + 0) * words + v);
    const uint4 w1 = __ldg(planes + ((size_t)nb * 2 + 1) * words + v);
    const uint32_t table = 0x000100FFu;              // byte c = value of code c: -1, 0, +1, (3 does not occur) 0
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const uint32_t p0 = c == 0 ? w0.x : c == 1 ? w0.y : c == 2 ? w0.z : w0.w;
        const uint32_t p1 = c == 0 ? w1.x : c == 1 ? w1.y : c == 2 ? w1.z : w1.w;
        // word bit 4j + ph belongs to weight 8ph + j: a0 holds, in its even bit pairs... interleave planes bit by bit
        const uint32_t a0 = (p0 & 0x55555555u) | ((p1 << 1) & 0xAAAAAAAAu);      // codes of the even word bits
        const uint32_t a1 = ((p0 >> 1) & 0x55555555u) | (p1 & 0xAAAAAAAAu);      // codes of the odd word bits
        uint32_t X[4];                               // X[ph]: nibble j = code of weight 8ph + j
        X[0] = a0 & 0x33333333u;
        X[2] = (a0 >> 2) & 0x33333333u;
        X[1] = a1 & 0x33333333u;
        X[3] = (a1 >> 2) & 0x33333333u;
        uint32_t out[8];
#pragma unroll
        for (int ph = 0; ph < 4; ++ph) {
            out[2 * ph] = __byte_perm(table, 0u, X[ph]);             // weights 8ph .. 8ph+3
            out[2 * ph + 1] = __byte_perm(table, 0u, X[ph] >> 16);   // weights 8ph+4 .. 8ph+7
        }
        uint4 *dst = reinterpret_cast<uint4 *>(w8 + ((size_t)(4 * nb + c) * K + (size_t)32 * v));
        dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
        dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
    }
}

tman_status launch_dequant_ternary_int8(const void *packed, int K, int N, int group, int8_t *w8, uint32_t *status,
                                        cudaStream_t s)
{
    const long total = (long)(N / 4) * (K / 32);
    dequant_ternary_int8_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(static_cast<const uint8_t *>(packed), w8,
                                                                             status, K, N, group);
    return launch_status();
}

tman_status launch_debug_indices(const void *packed, int K, int N, int bits, int group, uint8_t *idx,
                                 uint32_t *status, cudaStream_t s)
{
    long total = (long)bits * (K / 32) * N;
    debug_indices_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(
        static_cast<const uint8_t *>(packed), idx, status, K, N, bits, group);
    return launch_status();
}

__global__ void debug_luts_kernel(const __half *__restrict__ x, float *__restrict__ lut, int M, int K)
{
    long tid = (long)blockIdx.x * blockDim.x + threadIdx.x;
    long total = (long)M * (K / 4);
    if (tid >= total) return;
    const __half *px = x + tid * 4;
    float t[16];
    lut16(__half2float(px[0]), __half2float(px[1]), __half2float(px[2]), __half2float(px[3]), t);
#pragma unroll
    for (int p = 0; p < 16; ++p) lut[tid * 16 + p] = t[p];
}

tman_status launch_debug_luts(const void *x, int M, int K, float *lut, cudaStream_t s)
{
    long total = (long)M * (K / 4);
    debug_luts_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(static_cast<const __half *>(x),
                                                                      lut, M, K);
    return launch_status();
}

}  // namespace tman
