// Decode path: bit-serial table-lookup mpGEMV (paper Sec. 2.2 "Bit-serial table lookup", Fig. 2;
// Sec. 4.3 "Mapping of LUT-based Decoding").
//
// Work split.  The reduction dimension is cut into K-slices of 32/MT plane words (MT = number
// of activation rows a table entry carries).  One CTA owns one K-slice: it builds that slice's
// activation tables in shared memory once and reuses them for every output column it visits
// (the paper's "maximise reuse of cached lookup tables").  Inside a warp a lane owns ONE plane
// word, i.e. 32 consecutive activations = four 8-activation table groups, and one shared-memory
// bank column: tables are stored entry-major so that lane v always reads bank(s) of slot v,
// whatever its index.  Any mix of indices across the warp is therefore conflict-free, which is
// what allows 8-bit indices (two of the paper's 4-bit indices fused: one lookup covers eight
// weights of one bit-plane).
//
// Per lane and column: sum_i 2^i * sum_{4 groups} T[group][index byte]  (shift-accumulate),
// minus zero-point times the lane's activation sum, times the block scale (a lane's 32
// activations never straddle a quantization block since group >= 32); the per-lane partials of
// a column are then reduced across the lanes of the K-slice with warp shuffles, and K-slices
// are combined through fp32 partial sums in the workspace: the last slice to arrive (a counter
// per column group) adds them in slice order and writes fp16.
#include "common.cuh"

namespace tman {

// Optional phase time stamps for experiments (compiled out of the library build).
#ifdef TMAN_PHASE_TIMERS
__device__ unsigned long long *tman_stamp_buf;
#define TMAN_STAMP(i)                                                              \
    do {                                                                           \
        if (threadIdx.x == 0) {                                                    \
            unsigned long long t_;                                                 \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                 \
            tman_stamp_buf[blockIdx.x * 16 + (i)] = t_;                            \
            tman_stamp_buf[blockIdx.x * 16 + 8 + (i)] = (unsigned long long)clock64(); \
        }                                                                          \
    } while (0)
#else
#define TMAN_STAMP(i) do {} while (0)
#endif

constexpr int kGemvThreads = 512;
constexpr int kGemvWarps = kGemvThreads / 32;
constexpr int kGemvTableBytes = 128 * 1024;   // 4 groups x 256 entries x 32 slots x 4 B

struct GemvParams {
    const uint8_t  *packed;
    const uint32_t *planes;
    const __half   *scales;
    const uint16_t *zeros;
    const __half   *x;        // first row of this launch
    __half         *y;        // first row of this launch
    float          *partials;
    uint32_t       *counters;
    uint32_t       *status;
    int M;                    // rows in this launch (<= MT)
    int K, N, bits, group;
    int nkappa;               // K-slices
    int P;                    // CTAs per K-slice
    int units;                // warp-units per K-slice
};

template <int N_, int MASK>
struct LaneReduce {
    // Transpose-reduce N_ values across the lanes selected by MASK, MASK/2, ..., 1: every stage
    // halves the number of values a lane keeps (or, once one is left, plainly adds).
    static __device__ __forceinline__ void run(float *vals, int v, int &base)
    {
        if constexpr (MASK >= 1) {
            if constexpr (N_ >= 2) {
                constexpr int H = N_ / 2;
                const bool up = (v & MASK) != 0;
#pragma unroll
                for (int j = 0; j < H; ++j) {
                    float keep = up ? vals[j + H] : vals[j];
                    float send = up ? vals[j] : vals[j + H];
                    vals[j] = keep + __shfl_xor_sync(0xffffffffu, send, MASK);
                }
                base += up ? H : 0;
                LaneReduce<H, MASK / 2>::run(vals, v, base);
            } else {
                vals[0] += __shfl_xor_sync(0xffffffffu, vals[0], MASK);
                LaneReduce<1, MASK / 2>::run(vals, v, base);
            }
        }
    }
};

template <int MT> struct RowVec;
template <> struct RowVec<1> { using type = float; };
template <> struct RowVec<2> { using type = float2; };
template <> struct RowVec<4> { using type = float4; };

template <int MT>
__device__ __forceinline__ void load_rows(const uint8_t *p, float (&out)[MT])
{
    typename RowVec<MT>::type t = *reinterpret_cast<const typename RowVec<MT>::type *>(p);
    if constexpr (MT == 1) { out[0] = t; }
    else if constexpr (MT == 2) { out[0] = t.x; out[1] = t.y; }
    else { out[0] = t.x; out[1] = t.y; out[2] = t.z; out[3] = t.w; }
}

// byte offset of table entry (group c of the lane's word, index p, slot) inside the table area
__device__ __forceinline__ constexpr uint32_t table_imm(int c) { return (uint32_t)(c >> 1) * 65536u + (uint32_t)(c & 1) * 128u; }

template <int BITS, int MT, int S>
__global__ void __launch_bounds__(kGemvThreads, 1) mpgemv_kernel(const GemvParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    constexpr int W = 32 / MT;            // plane words (lanes) per K-slice
    constexpr int V = 4 * S * MT;         // values a lane produces per warp-unit
    constexpr int NKEEP = (V >= W) ? V / W : 1;

    TMAN_STAMP(0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kappa = blockIdx.x / p.P, j = blockIdx.x % p.P;
    const int words_total = p.K / 32;
    const int word0 = kappa * W;
    const int nwords = min(W, words_total - word0);
    const int sub = lane / W, v = lane % W;
    const bool active = v < nwords;
    const int nstrips = p.N / 4;
    const int nblk = p.K / p.group;
    const int B = active ? ((word0 + v) * 32) / p.group : 0;

    // Let the next kernel in the stream start its own weight streaming while this one drains
    // (programmatic dependent launch); the header words are requested now and checked later.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    uint32_t hdr[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) hdr[q] = __ldg(reinterpret_cast<const uint32_t *>(p.packed) + q);

    uint4    wreg[S][BITS];
    uint2    sreg[S];
    uint32_t zreg[S];

    auto load_unit = [&](int wu) {
#pragma unroll
        for (int s = 0; s < S; ++s) {
            const int nb = (wu * MT + sub) * S + s;
            const bool ok = active && nb < nstrips;
#pragma unroll
            for (int i = 0; i < BITS; ++i) {
                wreg[s][i] = make_uint4(0u, 0u, 0u, 0u);
                if (ok)
                    wreg[s][i] = __ldcs(reinterpret_cast<const uint4 *>(p.planes) +
                                        ((size_t)nb * BITS + i) * words_total + word0 + v);
            }
            sreg[s] = make_uint2(0u, 0u);
            zreg[s] = 0u;
            if (ok) {
                sreg[s] = __ldg(reinterpret_cast<const uint2 *>(p.scales) + (size_t)nb * nblk + B);
                zreg[s] = __ldg(p.zeros + (size_t)nb * nblk + B);
            }
        }
    };

    // Issue the first unit's weight loads before anything else: the packed buffer is constant
    // input and packed_bytes was checked on the host, so these reads are in bounds whatever the
    // header says.  Their latency overlaps the table build.
    int wu = j + p.P * warp;
    if (wu < p.units) load_unit(wu);
    TMAN_STAMP(1);

    // Everything below may depend on the previous kernel in the stream (activations, workspace).
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // The activations of this thread's table slot (one plane word = 32 activations of one row).
    const int vb = lane / MT, mb = lane % MT;
    const bool live = (vb < nwords) && (mb < p.M);
    uint4 xraw[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) xraw[c] = make_uint4(0u, 0u, 0u, 0u);
    if (live) {
        const uint4 *px = reinterpret_cast<const uint4 *>(p.x + (size_t)mb * p.K + (size_t)(word0 + vb) * 32);
#pragma unroll
        for (int c = 0; c < 4; ++c) xraw[c] = __ldg(px + c);
    }
    TMAN_STAMP(2);

    // ---- phase A: activation tables (paper Sec. 2.2; one table per 8 activations, 256 entries,
    // entry = 16-entry table of the low four + sum of the selected high four) -----------------
    {
        // warp w fills the entries whose high index nibble is w, for all four groups of the word
        const int ph = warp;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float xv[8];
            const __half2 *h2 = reinterpret_cast<const __half2 *>(&xraw[c]);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float2 f = __half22float2(h2[q]);
                xv[2 * q] = f.x;
                xv[2 * q + 1] = f.y;
            }
            float lo[16];
            lut16(xv[0], xv[1], xv[2], xv[3], lo);
            float hi = 0.f;
            if (ph & 1) hi += xv[4];
            if (ph & 2) hi += xv[5];
            if (ph & 4) hi += xv[6];
            if (ph & 8) hi += xv[7];
            uint8_t *dst = smem + table_imm(c) + (uint32_t)(ph * 16) * 256u + (uint32_t)lane * 4u;
#pragma unroll
            for (int pl = 0; pl < 16; ++pl)
                *reinterpret_cast<float *>(dst + pl * 256) = lo[pl] + hi;
        }
    }
    __syncthreads();
    TMAN_STAMP(3);

    // header check (uniform over the grid): a mismatch leaves every output untouched
    {
        const bool hdr_ok = (hdr[0] == 0x4E414D54u) && (hdr[1] == 0x30303242u) && (hdr[2] == kVersion) &&
                            (hdr[3] == (uint32_t)p.K) && (hdr[4] == (uint32_t)p.N) &&
                            (hdr[5] == (uint32_t)p.bits) && (hdr[6] == (uint32_t)p.group) && (hdr[7] == 4u);
        if (!hdr_ok) {
            if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_BAD_PACKED);
            return;
        }
    }

    // the lane's activation sum over its 32 activations (all-ones entries), for the zero-point term
    const uint32_t sub_off = (uint32_t)(v * MT * 4);
    float ssum[MT];
    {
#pragma unroll
        for (int m = 0; m < MT; ++m) ssum[m] = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float t[MT];
            load_rows<MT>(smem + table_imm(c) + 255u * 256u + sub_off, t);
#pragma unroll
            for (int m = 0; m < MT; ++m) ssum[m] += t[m];
        }
    }

    bool first = true;
    for (; wu < p.units; wu += p.P * kGemvWarps) {
        if (!first) load_unit(wu);
        first = false;

        // ---- phase B: lookups, shift-accumulate, scale and zero-point (paper Sec. 4.3) --------
        float vals[V];
#pragma unroll
        for (int s = 0; s < S; ++s) {
            const __half2 s01 = *reinterpret_cast<const __half2 *>(&sreg[s].x);
            const __half2 s23 = *reinterpret_cast<const __half2 *>(&sreg[s].y);
            const float sc[4] = {__low2float(s01), __high2float(s01), __low2float(s23), __high2float(s23)};
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                float a[MT];
#pragma unroll
                for (int m = 0; m < MT; ++m) a[m] = 0.f;
#pragma unroll
                for (int i = 0; i < BITS; ++i) {
                    const uint32_t w = (c4 == 0) ? wreg[s][i].x : (c4 == 1) ? wreg[s][i].y
                                     : (c4 == 2) ? wreg[s][i].z : wreg[s][i].w;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        // byte 1 <- index byte c of the word, byte 0 <- the lane's slot offset
                        const uint32_t off = __byte_perm(w, sub_off, 0x7604u | ((uint32_t)c << 4));
                        float t[MT];
                        load_rows<MT>(smem + table_imm(c) + off, t);
#pragma unroll
                        for (int m = 0; m < MT; ++m) a[m] = fmaf(t[m], (float)(1 << i), a[m]);
                    }
                }
                const float zf = (float)((zreg[s] >> (4 * c4)) & 0xFu);
#pragma unroll
                for (int m = 0; m < MT; ++m)
                    vals[(s * 4 + c4) * MT + m] = sc[c4] * fmaf(-zf, ssum[m], a[m]);
            }
        }

        TMAN_STAMP(4);
        // ---- reduce the K-slice's lanes (warp shuffles) -----------------------------------------
        int base = 0;
        LaneReduce<V, W / 2>::run(vals, v, base);
        const bool writer = (V >= W) ? true : ((v & (W / V - 1)) == 0);
        const int col0 = (wu * MT + sub) * S * 4;      // first column of this sub-warp's strips
        TMAN_STAMP(5);

        if (p.nkappa == 1) {
            if (writer) {
#pragma unroll
                for (int e = 0; e < NKEEP; ++e) {
                    const int idx = base + e, m = idx % MT, n = col0 + idx / MT;
                    if (n < p.N && m < p.M) p.y[(size_t)m * p.N + n] = __float2half_rn(vals[e]);
                }
            }
        } else {
            if (writer) {
#pragma unroll
                for (int e = 0; e < NKEEP; ++e) {
                    const int idx = base + e, m = idx % MT, n = col0 + idx / MT;
                    if (n < p.N) p.partials[((size_t)kappa * MT + m) * p.N + n] = vals[e];
                }
            }
            // ---- combine K-slices: the last slice to arrive sums them in slice order ------------
            __threadfence();
            __syncwarp();
            uint32_t old = 0;
            if (lane == 0) old = atomicAdd(p.counters + wu, 1u);
            old = __shfl_sync(0xffffffffu, old, 0);
            TMAN_STAMP(6);
            if (old == (uint32_t)(p.nkappa - 1)) {
                __threadfence();
                constexpr int C = 4 * S * MT;           // columns of the warp-unit
                const int cw0 = wu * C;
                for (int idx = lane; idx < MT * C; idx += 32) {
                    const int m = idx / C, n = cw0 + idx % C;
                    if (n < p.N && m < p.M) {
                        float acc = 0.f;
                        for (int kp = 0; kp < p.nkappa; ++kp)
                            acc += __ldcg(p.partials + ((size_t)kp * MT + m) * p.N + n);
                        p.y[(size_t)m * p.N + n] = __float2half_rn(acc);
                    }
                }
                if (lane == 0) p.counters[wu] = 0u;
            }
        }
    }
    TMAN_STAMP(7);
}

template <int BITS, int MT>
static constexpr int strips_per_unit() { return (BITS == 2 ? 8 : 4) / MT; }

template <int BITS, int MT>
static tman_status launch_one(GemvParams p, int sms, cudaStream_t s)
{
    constexpr int S = strips_per_unit<BITS, MT>();
    constexpr int W = 32 / MT;
    const int words_total = p.K / 32;
    p.nkappa = (words_total + W - 1) / W;
    p.P = sms / p.nkappa;
    if (p.P < 1) p.P = 1;
    const int nstrips = p.N / 4;
    p.units = (nstrips + S * MT - 1) / (S * MT);
    if (p.P > p.units) p.P = p.units;
    auto kern = mpgemv_kernel<BITS, MT, S>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemvTableBytes) != cudaSuccess)
        return TMAN_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.nkappa * p.P));
    cfg.blockDim = dim3(kGemvThreads);
    cfg.dynamicSmemBytes = kGemvTableBytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, p) != cudaSuccess) return TMAN_ERR_CUDA;
    return TMAN_OK;
}

template <int BITS>
static tman_status launch_rows(GemvParams p, int rows, int sms, cudaStream_t s)
{
    p.M = rows;
    if (rows == 1) return launch_one<BITS, 1>(p, sms, s);
    if (rows == 2) return launch_one<BITS, 2>(p, sms, s);
    return launch_one<BITS, 4>(p, sms, s);
}

size_t mpgemv_workspace_bytes(int M, int K, int N)
{
    (void)M;
    // worst case: rows are processed four at a time with K-slices of 8 plane words
    const size_t nkappa = (size_t)(K / 32 + 7) / 8;
    return kWsStatusBytes + ws_counter_bytes(N) + nkappa * 4 * (size_t)N * sizeof(float);
}

// bytes at the start of a workspace that must be zero before a call (status word and counters)
size_t mpgemv_workspace_zero_prefix(int N) { return kWsStatusBytes + ws_counter_bytes(N); }

tman_status launch_mpgemv(const void *packed, const void *x, void *y, int M, int K, int N, int bits,
                          int group, void *ws, size_t ws_bytes, cudaStream_t s)
{
    (void)ws_bytes;
    const int sms = sm_count();
    if (sms <= 0) return TMAN_ERR_CUDA;
    Layout L = make_layout(K, N, bits, group);
    const uint8_t *pk = static_cast<const uint8_t *>(packed);
    uint8_t *w8 = static_cast<uint8_t *>(ws);
    GemvParams p;
    p.packed = pk;
    p.planes = reinterpret_cast<const uint32_t *>(pk + L.planes_off);
    p.scales = reinterpret_cast<const __half *>(pk + L.scales_off);
    p.zeros = reinterpret_cast<const uint16_t *>(pk + L.zeros_off);
    p.status = reinterpret_cast<uint32_t *>(w8);
    p.counters = reinterpret_cast<uint32_t *>(w8 + kWsStatusBytes);
    p.partials = reinterpret_cast<float *>(w8 + kWsStatusBytes + ws_counter_bytes(N));
    p.K = K; p.N = N; p.bits = bits; p.group = group;
    p.M = 0; p.nkappa = 0; p.P = 0; p.units = 0;
    // rows go through in batches of at most four (a table entry carries up to four rows)
    for (int m0 = 0; m0 < M; m0 += 4) {
        const int rows = (M - m0 < 4) ? (M - m0) : 4;
        p.x = static_cast<const __half *>(x) + (size_t)m0 * K;
        p.y = static_cast<__half *>(y) + (size_t)m0 * N;
        tman_status st;
        if (bits == 2) st = launch_rows<2>(p, rows, sms, s);
        else if (bits == 3) st = launch_rows<3>(p, rows, sms, s);
        else st = launch_rows<4>(p, rows, sms, s);
        if (st != TMAN_OK) return st;
    }
    return TMAN_OK;
}

}  // namespace tman
