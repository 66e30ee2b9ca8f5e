// Decode path: bit-serial table-lookup mpGEMV (paper Sec. 2.2 "Bit-serial table lookup", Fig. 2;
// Sec. 4.3 "Mapping of LUT-based Decoding").
//
// Work split.  The reduction dimension is cut into K-slices of 8 to 32 plane words (16 for one
// activation row; 32, 16, 8 for 2, 3-4, 5-8 rows, whose table entries carry the rows as fp16 pairs).  One
// CTA owns one K-slice: it builds that slice's
// activation tables in shared memory once and reuses them for every output column it visits
// (the paper's "maximise reuse of cached lookup tables").  Inside a warp a lane owns ONE plane
// word, i.e. 32 consecutive activations = four 8-activation table groups, and one shared-memory
// bank column: tables are stored entry-major so that lane v always reads bank(s) of slot v,
// whatever its index.  Any mix of indices across the warp is therefore conflict-free, which is
// what allows 8-bit indices (two of the paper's 4-bit indices fused: one lookup covers eight
// weights of one bit-plane).
//
// Per lane and column: sum_i 2^i * sum_{4 groups} T[group][index byte]  (shift-accumulate).
// Lanes whose words share a quantization block are added first (one shuffle stage), then the
// zero-point times the block's activation sum is subtracted and the block scale applied, then the
// remaining lanes of the K-slice are reduced with a transposing shuffle reduction.  K-slices are
// combined through fp32 partial sums in the workspace.  The partial-sum area holds a sentinel bit
// pattern (a NaN no arithmetic produces) wherever no sum is pending; once its lookups are done,
// every CTA polls the sums of its share of the output columns until none of them is the sentinel,
// adds them in a fixed order, writes fp16 and puts the sentinel back.  The data are their own
// "ready" flag, so no fence and no counter sits between the last lookup and the output; the poll
// is bounded and reports TMAN_ERR_TIMEOUT.
//
// Streaming.  A warp works through units (a few strips of four columns).  With up to four activation
// rows every strip's registers are refilled with the next unit's strip as soon as its lookups are done;
// with more rows the next unit sits in a second set of registers.  Either way HBM reads overlap the
// lookups.  The first
// loads (header words, first unit) are issued before the kernel waits for the previous kernel in
// the stream (programmatic dependent launch); the host has checked that every read derived from
// (K, N, bits, group) is in bounds.  That is only sound while the previous kernel does not write the
// packed buffer: the host launches the call that follows a tman_pack_weights on the same stream
// in plain stream order instead (packed_write_pending below), and the header states the rule for
// kernels of the caller's own.
#include "common.cuh"

#include <atomic>

namespace tman {

constexpr int kGemvThreads = 512;
constexpr int kGemvWarps = kGemvThreads / 32;
constexpr int kGemvTableBytes = 128 * 1024;   // 4 groups x 256 entries x 32 slots x 4 B

// "No sum pending": a NaN bit pattern that no floating-point operation returns.
constexpr uint32_t kGemvSentinel = 0x7FA5A5A5u;
constexpr uint32_t kGemvPollLimit = 1u << 21;  // polls of ~0.5 us each: about a second

// Up to kGemvMaxGroup weight matrices that share the activations (same K, bits, group) go through
// one launch: their output columns are concatenated, the tables are built once (paper Sec. 5:
// one table precomputation shared by the projections that read the same input).
constexpr int kGemvMaxGroup = 4;

struct GemvParams {
    const uint8_t  *packed[kGemvMaxGroup];
    const uint4    *planes[kGemvMaxGroup];   // one uint4 = one plane word of the four columns of a strip
    const uint2    *scales[kGemvMaxGroup];   // four fp16 scales of a strip and block
    const uint16_t *zeros[kGemvMaxGroup];    // four zero-point nibbles of a strip and block
    __half         *y[kGemvMaxGroup];        // first row of this launch
    int Ng[kGemvMaxGroup];                   // output columns of each matrix
    int unit0[kGemvMaxGroup];                // first warp-unit of each matrix
    int col0[kGemvMaxGroup];                 // first concatenated column of each matrix
    int count;                               // matrices in this launch
    const __half   *x;          // first row of this launch
    // integer path (per-tensor ternary weights, 16-bit integer activations): quantized activations,
    // their per-row scales, the tensor's weight scale, optional exact integer sums [M][N]
    const int16_t  *xi;
    const float    *row_scale;
    float           w_scale;
    int32_t        *acc_out;
    float          *partials;
    uint32_t       *status;
    int M;                      // rows in this launch (<= MT)
    int K, N, bits, group;      // N = total (concatenated) columns
    int nkappa;                 // K-slices
    int P;                      // CTAs per K-slice
    int units;                  // warp-units per K-slice
    int group_shift;            // log2(group)
    int nblk;                   // K / group
};

// Transposing reduction over the lanes selected by MASK, 2*MASK, ..., below END: every stage
// halves the number of values a lane keeps (or, once one is left, plainly adds).  `base` is the
// logical index of vals[0].
// INTS: the values are 32-bit integers kept in float registers (bit patterns) and are added as integers.
template <int N_, int MASK, int END, bool INTS = false>
struct LaneReduce {
    static __device__ __forceinline__ float add(float a, float b)
    {
        if constexpr (INTS) return __int_as_float(__float_as_int(a) + __float_as_int(b));
        else return a + b;
    }
    static __device__ __forceinline__ void run(float *vals, int v, int &base)
    {
        if constexpr (MASK < END) {
            if constexpr (N_ >= 2) {
                constexpr int H = N_ / 2;
                const bool up = (v & MASK) != 0;
#pragma unroll
                for (int j = 0; j < H; ++j) {
                    const float keep = up ? vals[j + H] : vals[j];
                    const float send = up ? vals[j] : vals[j + H];
                    vals[j] = add(keep, __shfl_xor_sync(0xffffffffu, send, MASK));
                }
                base += up ? H : 0;
                LaneReduce<H, MASK * 2, END, INTS>::run(vals, v, base);
            } else {
                vals[0] = add(vals[0], __shfl_xor_sync(0xffffffffu, vals[0], MASK));
                LaneReduce<1, MASK * 2, END, INTS>::run(vals, v, base);
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

__device__ __forceinline__ float4 ld_volatile_f4(const float4 *p)
{
    float4 v;
    asm volatile("ld.volatile.global.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ bool has_sentinel(const float4 &v)
{
    return __float_as_uint(v.x) == kGemvSentinel || __float_as_uint(v.y) == kGemvSentinel ||
           __float_as_uint(v.z) == kGemvSentinel || __float_as_uint(v.w) == kGemvSentinel;
}

// Bounded wait of the split-K combine: polls up to four partial-sum quads (slices kp, kp + SP, ... below
// nkappa) until none of them holds the "no sum pending" pattern, at most `limit` times.  Returns
// whether they all arrived; the caller reports TMAN_ERR_TIMEOUT otherwise.
__device__ __forceinline__ bool wait_for_sums(const float4 *src, size_t stride4, int kp, int SP, int nkappa,
                                              uint32_t limit, float4 (&t)[4])
{
    bool ready = false;
    for (uint32_t tries = 0; !ready && tries < limit; ++tries) {
        ready = true;
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (kp + q * SP < nkappa) t[q] = ld_volatile_f4(src + (size_t)(kp + q * SP) * stride4);
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (kp + q * SP < nkappa) ready = ready && !has_sentinel(t[q]);
    }
    return ready;
}

// byte offset of table entry (group c of the lane's word, index p, slot) inside the table area
__device__ __forceinline__ constexpr uint32_t table_imm(int c) { return (uint32_t)(c >> 1) * 65536u + (uint32_t)(c & 1) * 128u; }

// The tables start at the first byte of dynamic shared memory.  The kernel has no static shared
// memory, so that byte sits right after the per-CTA reserved region, at shared-window address
// kGemvSmemBase (the host checks cudaDevAttrReservedSharedMemoryPerBlock, the kernel checks its
// own base).  A lookup can then use the byte-permute result (index byte << 8 | slot offset) as
// the address register, with the table's offset folded into the instruction's immediate: no add
// per lookup.
constexpr uint32_t kGemvSmemBase = 1024;

template <int MT, uint32_t IMM>
__device__ __forceinline__ void lookup_rows(uint32_t off, float (&out)[MT])
{
    if constexpr (MT == 1) {
        asm volatile("ld.shared.f32 %0, [%1 + %2];" : "=f"(out[0]) : "r"(off), "n"(IMM));
    } else if constexpr (MT == 2) {
        asm volatile("ld.shared.v2.f32 {%0, %1}, [%2 + %3];" : "=f"(out[0]), "=f"(out[1]) : "r"(off), "n"(IMM));
    } else {
        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4 + %5];"
                     : "=f"(out[0]), "=f"(out[1]), "=f"(out[2]), "=f"(out[3]) : "r"(off), "n"(IMM));
    }
}

// The same lookup returning the raw 32-bit slots (two fp16 rows each).
template <int MT, uint32_t IMM>
__device__ __forceinline__ void lookup_slots(uint32_t off, uint32_t (&out)[MT])
{
    if constexpr (MT == 1) {
        asm volatile("ld.shared.b32 %0, [%1 + %2];" : "=r"(out[0]) : "r"(off), "n"(IMM));
    } else if constexpr (MT == 2) {
        asm volatile("ld.shared.v2.b32 {%0, %1}, [%2 + %3];" : "=r"(out[0]), "=r"(out[1]) : "r"(off), "n"(IMM));
    } else {
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4 + %5];"
                     : "=r"(out[0]), "=r"(out[1]), "=r"(out[2]), "=r"(out[3]) : "r"(off), "n"(IMM));
    }
}

// One unit's worth of a lane's inputs: its plane word of S strips, and the strips' scales and
// zero-points of the lane's quantization block.
template <int BITS, int S>
struct UnitRegs {
    uint4    w[S][BITS];
    uint2    sc[S];
    uint32_t z[S];
    int      g;        // matrix of the unit
    int      col;      // concatenated column of the lane's first strip
};

// BITS planes, MT rows per table entry, S strips per warp-unit and sub-warp, PRE = 1 when the
// lanes v and v^1 share a quantization block (group >= 64): they are added before scaling.
// HALF (MT = 1 only): K-slices of 16 plane words instead of 32, i.e. 64 KB of tables that cost
// half as much to build.  The two half-warps then work on different strips and read the same 64
// tables; entry rows hold all 64 slots (slot = word + 16 * index byte) and the second half-warp
// visits the index bytes of a word in the order 1,0,3,2, so that the 32 lanes still address 32
// different banks.
// GROUPED = 0: one matrix, the matrix index is a compile-time zero.
// HR (more than one activation row): a 32-bit table slot holds two rows as fp16 instead of one as fp32,
// so an entry of MT slots serves 2 * MT rows for the same shared-memory traffic.  Each row of the
// K-slice is first scaled by a power of two that brings its largest magnitude into [1, 2) (undone in
// fp32 at the end), so that entries use fp16's range whatever the activations' size; the bits * 4
// lookups of one plane word are accumulated in fp16 (low plane first), everything after that in fp32.
// INT (one row, HALF): per-tensor ternary weights (2-bit codes, zero-point 1, one scale) with 16-bit integer
// activations (paper Sec. 6.1: BitNet as W_INT2 A_INT16).  Tables hold exact integer sums (as fp32: a sum of
// eight 16-bit values is below 2^24), a word's lookups and the pair sum stay exact in fp32, and from there
// on the sums are 32-bit integers: the slice's lanes, the K-slices and the result are added as integers;
// only the final product with the row's and the tensor's scale is floating point (Sec. 4.3).
// ROLL: one set of unit registers; every strip's registers are refilled with the next unit's strip as
// soon as its lookups are done (larger units, fewer per-unit fixed costs, same bytes in flight).
template <int BITS, int MT, int S, int PRE, int HALF, int GROUPED, int ROLL, int HR, int INT>
__global__ void __launch_bounds__(kGemvThreads, 1) mpgemv_kernel(const GemvParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    static_assert(!HALF || MT == 1, "half slices are for single-row tables");
    static_assert(!INT || (!HR && !GROUPED && BITS == 2), "the integer path is built for ternary weights, fp32-held integer tables");
    static_assert(!HR || !HALF, "fp16 row pairs use whole-warp or sub-warp slices");
    constexpr int R = HR ? 2 * MT : MT;    // activation rows of this launch
    constexpr int W = HALF ? 16 : 32 / MT; // plane words (lanes) per K-slice
    constexpr int SUBS = 32 / W;           // sub-warps, each on its own strips
    constexpr int V = 4 * S * R;          // values a lane produces per warp-unit
    constexpr int V1 = PRE ? V / 2 : V;   // values it still holds when scales are applied
    constexpr int NKEEP = (V >= W) ? V / W : 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kappa = blockIdx.y, j = blockIdx.x;
    const int words_total = p.K >> 5;
    const int word0 = kappa * W;
    const int nwords = min(W, words_total - word0);
    const int sub = lane / W, v = lane % W;
    const bool active = v < nwords;
    const int nblk = p.nblk;
    const int B = ((word0 + (active ? v : 0)) * 32) >> p.group_shift;

    // Let the next kernel in the stream start its own weight streaming while this one drains
    // (programmatic dependent launch); the header words are requested now and checked later.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool hdr_ok = true;
    {
        uint32_t hdr[kGemvMaxGroup][8];
#pragma unroll
        for (int g = 0; g < (GROUPED ? kGemvMaxGroup : 1); ++g)
            if (g < p.count) {
#pragma unroll
                for (int q = 0; q < 8; ++q) hdr[g][q] = __ldg(reinterpret_cast<const uint32_t *>(p.packed[g]) + q);
            }
#pragma unroll
        for (int g = 0; g < (GROUPED ? kGemvMaxGroup : 1); ++g)
            if (g < p.count)
                hdr_ok = hdr_ok && (hdr[g][0] == 0x4E414D54u) && (hdr[g][1] == 0x30303242u) && (hdr[g][2] == kVersion) &&
                         (hdr[g][3] == (uint32_t)p.K) && (hdr[g][4] == (uint32_t)p.Ng[g]) &&
                         (hdr[g][5] == (uint32_t)p.bits) && (hdr[g][6] == (uint32_t)p.group) && (hdr[g][7] == 4u);
    }

    // Loads are unconditional: a unit past the last one re-reads the last unit, a strip past the
    // last one re-reads the last strip, a lane past the end of a ragged last slice re-reads word 0
    // (its tables are all zero); none of those results is ever written.
    const uint32_t lane_word = (uint32_t)(word0 + (active ? v : 0));
    const uint32_t row_bytes = (uint32_t)words_total * 16u;      // one plane of one strip
    const uint32_t strip_bytes = row_bytes * BITS;
    struct UnitAddr { const uint8_t *pw; const uint2 *psc; const uint16_t *pz; int lu, nstrips; };
    auto unit_addr = [&](UnitRegs<BITS, S> &r, int wu) {
        const int u = min(wu, p.units - 1);
        int g = 0;
        if constexpr (GROUPED) {
#pragma unroll
            for (int t = 1; t < kGemvMaxGroup; ++t) g += (t < p.count && u >= p.unit0[t]) ? 1 : 0;
        }
        UnitAddr a;
        a.lu = GROUPED ? u - p.unit0[g] : u;
        a.nstrips = p.Ng[g] >> 2;
        a.pw = reinterpret_cast<const uint8_t *>(p.planes[g] + lane_word);
        a.psc = p.scales[g] + B;
        a.pz = p.zeros[g] + B;
        r.g = g;
        r.col = (GROUPED ? p.col0[g] : 0) + (a.lu * SUBS + sub) * S * 4;
        return a;
    };
    auto load_strip = [&](UnitRegs<BITS, S> &r, int s, const UnitAddr &a) {
        const uint32_t nb = (uint32_t)min((a.lu * SUBS + sub) * S + s, a.nstrips - 1);
        const uint8_t *q = a.pw + (size_t)nb * strip_bytes;
#pragma unroll
        for (int i = 0; i < BITS; ++i) {
            r.w[s][i] = __ldcs(reinterpret_cast<const uint4 *>(q));
            q += row_bytes;
        }
        if constexpr (INT) {
            r.sc[s] = make_uint2(0x3C003C00u, 0x3C003C00u);      // scale 1.0 four times (fp16), zero-point 1 four times
            r.z[s] = 0x1111u;
        } else {
            r.sc[s] = __ldg(a.psc + (size_t)nb * (uint32_t)nblk);
            r.z[s] = __ldg(a.pz + (size_t)nb * (uint32_t)nblk);
        }
    };
    auto load_unit = [&](UnitRegs<BITS, S> &r, int wu) {
        const UnitAddr a = unit_addr(r, wu);
#pragma unroll
        for (int s = 0; s < S; ++s) load_strip(r, s, a);
    };

    // Issue the first unit's weight loads before anything else: packed_bytes was checked on the
    // host, so these reads are in bounds whatever the header says, and no kernel that may still be
    // running writes the packed buffer (see the top of the file).  Their latency overlaps the table build.
    const int wu0 = j + p.P * warp, wstride = p.P * kGemvWarps;
    UnitRegs<BITS, S> regs[ROLL ? 1 : 2];
    load_unit(regs[0], wu0);

    // Everything below may depend on the previous kernel in the stream (activations, workspace).
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if constexpr (HALF) {
        // thread (slot, chunk): slot = word + 16 * index byte of the table it fills, chunk = the
        // three high index bits of its 32 entries
        const int slot = tid & 63, chunk = tid >> 6;
        const int gv = slot & 15, gc = slot >> 4;
        // index bit q of byte gc is word bit 8*gc + q, i.e. the weight 8*(q & 3) + 2*gc + (q >> 2)
        float xv[8];
        if constexpr (INT) {
            short2 raw[4];
#pragma unroll
            for (int ph = 0; ph < 4; ++ph) {
                raw[ph] = make_short2(0, 0);
                if (gv < nwords)
                    raw[ph] = __ldg(reinterpret_cast<const short2 *>(p.xi + (size_t)(word0 + gv) * 32 + 8 * ph + 2 * gc));
            }
#pragma unroll
            for (int ph = 0; ph < 4; ++ph) {
                xv[ph] = (float)raw[ph].x;
                xv[ph + 4] = (float)raw[ph].y;
            }
        } else {
            __half2 raw[4];
#pragma unroll
            for (int ph = 0; ph < 4; ++ph) {
                raw[ph] = __floats2half2_rn(0.f, 0.f);
                if (gv < nwords)
                    raw[ph] = __ldg(reinterpret_cast<const __half2 *>(p.x + (size_t)(word0 + gv) * 32 + 8 * ph + 2 * gc));
            }
            if constexpr (!ROLL) load_unit(regs[1], wu0 + wstride);
#pragma unroll
            for (int ph = 0; ph < 4; ++ph) {
                const float2 f = __half22float2(raw[ph]);
                xv[ph] = f.x;
                xv[ph + 4] = f.y;
            }
        }
        float lo[16];
        lut16(xv[0], xv[1], xv[2], xv[3], lo);
        float hi = 0.f;
        if (chunk & 1) hi += xv[5];
        if (chunk & 2) hi += xv[6];
        if (chunk & 4) hi += xv[7];
        uint8_t *dst = smem + (uint32_t)(chunk * 32) * 256u + (uint32_t)slot * 4u;
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const float base = q ? hi + xv[4] : hi;
#pragma unroll
            for (int e = 0; e < 16; ++e) *reinterpret_cast<float *>(dst + (q * 16 + e) * 256) = lo[e] + base;
        }
    } else if constexpr (HR) {
        // The activations of this thread's table slot: one plane word = 32 activations of rows 2*mb and 2*mb+1.
        const int vb = lane / MT, mb = lane % MT;
        uint4 xraw[2][4];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const bool live = (vb < nwords) && (2 * mb + r < p.M);
#pragma unroll
            for (int c = 0; c < 4; ++c) xraw[r][c] = make_uint4(0u, 0u, 0u, 0u);
            if (live) {
                const uint4 *px = reinterpret_cast<const uint4 *>(p.x + (size_t)(2 * mb + r) * p.K + (size_t)(word0 + vb) * 32);
#pragma unroll
                for (int c = 0; c < 4; ++c) xraw[r][c] = __ldg(px + c);
            }
        }
        if constexpr (!ROLL) load_unit(regs[1], wu0 + wstride);

        // largest magnitude of each row over the K-slice -> power-of-two scale (every warp computes the same)
        float inv[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            __half2 mx = __floats2half2_rn(0.f, 0.f);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const __half2 *h = reinterpret_cast<const __half2 *>(&xraw[r][c]);
#pragma unroll
                for (int q = 0; q < 4; ++q) mx = __hmax2(mx, __habs2(h[q]));
            }
            float amax = fmaxf(__low2float(mx), __high2float(mx));
#pragma unroll
            for (int mask = MT; mask < 32; mask <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, mask));
            const uint32_t e = (__float_as_uint(amax) >> 23) & 0xFFu;      // amax = 1.f * 2^(e - 127)
            inv[r] = __uint_as_float((254u - e) << 23);
            if (warp == 0 && vb == 0)
                reinterpret_cast<float *>(smem + kGemvTableBytes)[2 * mb + r] = __uint_as_float(e << 23);
        }
        {
            // warp w fills, for index byte c = w % 4 of the word, the entries whose high index nibble is
            // 4 * (w / 4) .. 4 * (w / 4) + 3: the low-nibble sums of a byte are then computed once per warp
            const int c = warp & 3;
            float lo[2][16], xh[2][4];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                float xv[8];
#pragma unroll
                for (int qq = 0; qq < 4; ++qq) {
                    // the c-th half2 of quarter qq: four-way select on the warp-uniform c
                    const uint4 q4 = xraw[r][qq];
                    const uint32_t u = c == 0 ? q4.x : c == 1 ? q4.y : c == 2 ? q4.z : q4.w;
                    const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&u));
                    xv[qq] = f.x * inv[r];
                    xv[qq + 4] = f.y * inv[r];
                }
                lut16(xv[0], xv[1], xv[2], xv[3], lo[r]);
#pragma unroll
                for (int qq = 0; qq < 4; ++qq) xh[r][qq] = xv[4 + qq];
            }
#pragma unroll
            for (int pq = 0; pq < 4; ++pq) {
                const int ph = 4 * (warp >> 2) + pq;
                float hi[2];
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    hi[r] = 0.f;
                    if (ph & 1) hi[r] += xh[r][0];
                    if (ph & 2) hi[r] += xh[r][1];
                    if (ph & 4) hi[r] += xh[r][2];
                    if (ph & 8) hi[r] += xh[r][3];
                }
                uint8_t *dst = smem + table_imm(c) + (uint32_t)(ph * 16) * 256u + (uint32_t)lane * 4u;
#pragma unroll
                for (int pl = 0; pl < 16; ++pl)
                    *reinterpret_cast<__half2 *>(dst + pl * 256) = __floats2half2_rn(lo[0][pl] + hi[0], lo[1][pl] + hi[1]);
            }
        }
    } else {
        // The activations of this thread's table slot (one plane word = 32 activations of one row).
        const int vb = lane / MT, mb = lane % MT;
        const bool live = (vb < nwords) && (mb < p.M);
        uint4 xraw[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) xraw[c] = make_uint4(0u, 0u, 0u, 0u);
        if (live) {
            // 16-bit activations either way: fp16, or the integer path's quantized values
            const void *row = INT ? static_cast<const void *>(p.xi + (size_t)mb * p.K + (size_t)(word0 + vb) * 32)
                                  : static_cast<const void *>(p.x + (size_t)mb * p.K + (size_t)(word0 + vb) * 32);
            const uint4 *px = reinterpret_cast<const uint4 *>(row);
#pragma unroll
            for (int c = 0; c < 4; ++c) xraw[c] = __ldg(px + c);
        }
        if constexpr (!ROLL) load_unit(regs[1], wu0 + wstride);

        // ---- phase A: activation tables (paper Sec. 2.2; one table per 8 activations, 256 entries,
        // entry = 16-entry table of the low four + sum of the selected high four) -----------------
        {
            // warp w fills the entries whose high index nibble is w, for all four groups of the word
            const int ph = warp;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                // index bit q of byte c is word bit 8*c + q, i.e. the weight 8*(q & 3) + 2*c + (q >> 2):
                // the c-th pair of each quarter of the word
                float xv[8];
#pragma unroll
                for (int qq = 0; qq < 4; ++qq) {
                    if constexpr (INT) {
                        const short2 q2 = reinterpret_cast<const short2 *>(&xraw[qq])[c];
                        xv[qq] = (float)q2.x;
                        xv[qq + 4] = (float)q2.y;
                    } else {
                        const float2 f = __half22float2(reinterpret_cast<const __half2 *>(&xraw[qq])[c]);
                        xv[qq] = f.x;
                        xv[qq + 4] = f.y;
                    }
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
    }
    __syncthreads();

    // header and layout check (uniform over the grid): a mismatch leaves every output untouched
    const bool base_ok = (uint32_t)__cvta_generic_to_shared(smem) == kGemvSmemBase;
    if (!hdr_ok || !base_ok) {
        if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0)
            atomicCAS(p.status, 0u, (uint32_t)(hdr_ok ? TMAN_ERR_LAYOUT : TMAN_ERR_BAD_PACKED));
        return;
    }

    // the activation sum of the lane's 32 activations (all-ones entries), for the zero-point term;
    // with PRE, of the two lanes that share the block
    const uint32_t sub_off = (uint32_t)(v * MT * 4);
    // HALF: slot offset inside a row = (v + 16 * byte) * 4; the byte visited at step jj is jj for
    // the first half-warp and jj ^ 1 for the second, so 64 * (jj & ~1) goes into the immediate and
    // the rest (0 or 64) into one of two registers
    const uint32_t off_even = (uint32_t)(v * 4 + 64 * sub), off_odd = (uint32_t)(v * 4 + 64 * (1 - sub));
    uint32_t sel_h[4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) sel_h[jj] = 0x7604u | ((uint32_t)(jj ^ sub) << 4);
    float ssum[R];
    {
#pragma unroll
        for (int m = 0; m < R; ++m) ssum[m] = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if constexpr (HR) {
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    const float2 f = __half22float2(
                        *reinterpret_cast<const __half2 *>(smem + table_imm(c) + 255u * 256u + sub_off + 4u * m));
                    ssum[2 * m] += f.x;
                    ssum[2 * m + 1] += f.y;
                }
            } else {
                float t[MT];
                if constexpr (HALF) load_rows<MT>(smem + 255u * 256u + (uint32_t)(v + 16 * c) * 4u, t);
                else load_rows<MT>(smem + table_imm(c) + 255u * 256u + sub_off, t);
#pragma unroll
                for (int m = 0; m < MT; ++m) ssum[m] += t[m];
            }
        }
        if constexpr (PRE) {
#pragma unroll
            for (int m = 0; m < R; ++m) ssum[m] += __shfl_xor_sync(0xffffffffu, ssum[m], 1);
        }
    }

    // ---- phase B: lookups, shift-accumulate, scale and zero-point (paper Sec. 4.3) --------------
    auto compute_unit = [&](UnitRegs<BITS, S> &r, int wu, int next_wu) {
        float vals[V];
        // what the end of the unit needs survives the refill of the strip registers
        uint2 sc_s[S];
        uint32_t z_s[S];
#pragma unroll
        for (int s = 0; s < S; ++s) { sc_s[s] = r.sc[s]; z_s[s] = r.z[s]; }
        const int g_u = r.g, col_u = r.col;
        UnitAddr nxt;
        if constexpr (ROLL) nxt = unit_addr(r, next_wu);
#pragma unroll
        for (int s = 0; s < S; ++s) {
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                float a[MT];
                __half2 a2[MT];
#pragma unroll
                for (int m = 0; m < MT; ++m) { a[m] = 0.f; a2[m] = __floats2half2_rn(0.f, 0.f); }
#pragma unroll
                for (int i = 0; i < BITS; ++i) {
                    const uint32_t w = (c4 == 0) ? r.w[s][i].x : (c4 == 1) ? r.w[s][i].y
                                     : (c4 == 2) ? r.w[s][i].z : r.w[s][i].w;
                    const __half2 pw = __floats2half2_rn((float)(1 << i), (float)(1 << i));
                    // byte 1 <- index byte c of the word, byte 0 <- the lane's slot offset
#define TMAN_LOOKUP(c)                                                                          \
    if constexpr (HR) {                                                                         \
        uint32_t t[MT];                                                                         \
        const uint32_t off = __byte_perm(w, sub_off, 0x7604u | ((uint32_t)(c) << 4));           \
        lookup_slots<MT, kGemvSmemBase + table_imm(c)>(off, t);                                 \
        _Pragma("unroll") for (int m = 0; m < MT; ++m)                                          \
            a2[m] = __hfma2(*reinterpret_cast<const __half2 *>(&t[m]), pw, a2[m]);              \
    } else {                                                                                    \
        float t[MT];                                                                            \
        if constexpr (HALF) {                                                                   \
            const uint32_t off = __byte_perm(w, ((c) & 1) ? off_odd : off_even, sel_h[c]);      \
            lookup_rows<MT, kGemvSmemBase + 64u * ((c) & ~1)>(off, t);                          \
        } else {                                                                                \
            const uint32_t off = __byte_perm(w, sub_off, 0x7604u | ((uint32_t)(c) << 4));       \
            lookup_rows<MT, kGemvSmemBase + table_imm(c)>(off, t);                              \
        }                                                                                       \
        _Pragma("unroll") for (int m = 0; m < MT; ++m) a[m] = fmaf(t[m], (float)(1 << i), a[m]); \
    }
                    TMAN_LOOKUP(0) TMAN_LOOKUP(1) TMAN_LOOKUP(2) TMAN_LOOKUP(3)
#undef TMAN_LOOKUP
                }
                if constexpr (HR) {
#pragma unroll
                    for (int m = 0; m < MT; ++m) {
                        const float2 f = __half22float2(a2[m]);
                        vals[(s * 4 + c4) * R + 2 * m] = f.x;
                        vals[(s * 4 + c4) * R + 2 * m + 1] = f.y;
                    }
                } else {
#pragma unroll
                    for (int m = 0; m < MT; ++m) vals[(s * 4 + c4) * MT + m] = a[m];
                }
            }
            if constexpr (ROLL) load_strip(r, s, nxt);
        }

        // lanes v and v^1 hold the two words of one block: add them first, keeping half the columns
        int base = 0;
        LaneReduce<V, 1, PRE ? 2 : 1>::run(vals, v, base);
        const bool up = PRE && (v & 1);
        // scales and zero-points of the columns this lane still holds
        if constexpr (S >= 2 || !PRE) {
            constexpr int S1 = PRE ? S / 2 : S;
#pragma unroll
            for (int s = 0; s < S1; ++s) {
                const uint2 scq = up ? sc_s[s + (PRE ? S1 : 0)] : sc_s[s];
                const uint32_t zq = up ? z_s[s + (PRE ? S1 : 0)] : z_s[s];
                const __half2 s01 = *reinterpret_cast<const __half2 *>(&scq.x);
                const __half2 s23 = *reinterpret_cast<const __half2 *>(&scq.y);
                const float sc[4] = {__low2float(s01), __high2float(s01), __low2float(s23), __high2float(s23)};
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    const float zf = (float)((zq >> (4 * c4)) & 0xFu);
#pragma unroll
                    for (int m = 0; m < R; ++m) {
                        float &val = vals[(s * 4 + c4) * R + m];
                        val = sc[c4] * fmaf(-zf, ssum[m], val);
                    }
                }
            }
        } else {
            // one strip, two of its four columns left
            const uint32_t scq = up ? sc_s[0].y : sc_s[0].x;
            const uint32_t zq = up ? (z_s[0] >> 8) : z_s[0];
            const __half2 s01 = *reinterpret_cast<const __half2 *>(&scq);
            const float sc[2] = {__low2float(s01), __high2float(s01)};
#pragma unroll
            for (int c2 = 0; c2 < 2; ++c2) {
                const float zf = (float)((zq >> (4 * c2)) & 0xFu);
#pragma unroll
                for (int m = 0; m < R; ++m) {
                    float &val = vals[c2 * R + m];
                    val = sc[c2] * fmaf(-zf, ssum[m], val);
                }
            }
        }
        // the other lanes of the K-slice (integer path: exact integers so far, added as integers from here on)
        if constexpr (INT) {
#pragma unroll
            for (int e = 0; e < V1; ++e) vals[e] = __int_as_float(__float2int_rn(vals[e]));
        }
        LaneReduce<V1, PRE ? 2 : 1, W, INT != 0>::run(vals, v, base);
        const bool writer = (V >= W) ? true : (v < V);
        if (writer && wu < p.units) {
            const int g = GROUPED ? g_u : 0;
            const int lim = GROUPED ? p.col0[g] + p.Ng[g] : p.N;   // end of this matrix's columns
#pragma unroll
            for (int e = 0; e < NKEEP; ++e) {
                const int idx = base + e, m = idx % R, n = col_u + idx / R;
                if (n < lim && m < p.M) {
                    float out = vals[e];
                    if constexpr (HR) out *= reinterpret_cast<const float *>(smem + kGemvTableBytes)[m];   // undo the row's scale
                    if (p.nkappa == 1) {
                        if constexpr (INT) {
                            const int acc = __float_as_int(out);
                            if (p.acc_out) p.acc_out[(size_t)m * p.N + n] = acc;
                            out = (float)acc * (__ldg(p.row_scale + m) * p.w_scale);
                        }
                        p.y[g][(size_t)m * p.Ng[g] + (n - (GROUPED ? p.col0[g] : 0))] = __float2half_rn(out);
                    } else {
                        p.partials[((size_t)kappa * R + m) * p.N + n] = out;     // integer path: the integer's bit pattern
                    }
                }
            }
        }
    };

    if constexpr (ROLL) {
        for (int wu = wu0; wu < p.units; wu += wstride) compute_unit(regs[0], wu, wu + wstride);
    } else {
        for (int wu = wu0; wu < p.units; wu += 2 * wstride) {
            compute_unit(regs[0], wu, 0);
            load_unit(regs[0], wu + 2 * wstride);
            if (wu + wstride >= p.units) break;        // uniform over the warp
            compute_unit(regs[1], wu + wstride, 0);
            load_unit(regs[1], wu + 3 * wstride);
        }
    }

    // ---- combine K-slices: every CTA polls the partial sums of its share of the columns ----------
    if (p.nkappa > 1) {
        const int cta = blockIdx.y * gridDim.x + blockIdx.x, G = gridDim.x * gridDim.y;
        const int ng = p.N >> 2;
        const int g_lo = (int)(((long long)ng * cta) / G), g_hi = (int)(((long long)ng * (cta + 1)) / G);
        const int col_lo = g_lo * 4;
        const int ngrp = g_hi - g_lo;
        const int items = ngrp * p.M;                       // one item = four columns of one row
        const size_t stride4 = (size_t)R * p.N / 4;
        // SP adjacent lanes share an item and split the slices among them (slice kp goes to lane
        // kp % SP); their sums are added in a fixed order, so the result does not depend on timing
        int SP = 1;
        while (SP < 8 && 2 * SP <= p.nkappa && items * 2 * SP <= kGemvThreads) SP *= 2;
        const int part = tid & (SP - 1);
        const float sv = __uint_as_float(kGemvSentinel);
        using RED = LaneReduce<1, 1, 1, INT != 0>;          // its add(): floats, or integers kept in float registers
        bool gave_up = false;
        for (int item0 = 0; item0 < items; item0 += kGemvThreads / SP) {
            const int item = item0 + tid / SP;
            const bool alive = item < items;
            const int m = alive ? item / ngrp : 0, n = col_lo + 4 * (alive ? item % ngrp : 0);
            float4 *src = reinterpret_cast<float4 *>(p.partials + (size_t)m * p.N + n);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);      // also the bit pattern of integer zero
            for (int kp = part; alive && kp < p.nkappa; kp += 4 * SP) {
                float4 t[4];
                if (!wait_for_sums(src, stride4, kp, SP, p.nkappa, kGemvPollLimit, t)) { gave_up = true; break; }
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (kp + q * SP < p.nkappa) {
                        acc.x = RED::add(acc.x, t[q].x); acc.y = RED::add(acc.y, t[q].y);
                        acc.z = RED::add(acc.z, t[q].z); acc.w = RED::add(acc.w, t[q].w);
                        src[(size_t)(kp + q * SP) * stride4] = make_float4(sv, sv, sv, sv);
                    }
            }
            for (int mask = 1; mask < SP; mask <<= 1) {
                acc.x = RED::add(acc.x, __shfl_xor_sync(0xffffffffu, acc.x, mask));
                acc.y = RED::add(acc.y, __shfl_xor_sync(0xffffffffu, acc.y, mask));
                acc.z = RED::add(acc.z, __shfl_xor_sync(0xffffffffu, acc.z, mask));
                acc.w = RED::add(acc.w, __shfl_xor_sync(0xffffffffu, acc.w, mask));
            }
            gave_up = __any_sync(0xffffffffu, gave_up);
            if constexpr (INT) {
                if (alive && part == 0 && !gave_up) {
                    const int4 ia = make_int4(__float_as_int(acc.x), __float_as_int(acc.y), __float_as_int(acc.z), __float_as_int(acc.w));
                    if (p.acc_out) *reinterpret_cast<int4 *>(p.acc_out + (size_t)m * p.N + n) = ia;
                    const float sc = __ldg(p.row_scale + m) * p.w_scale;
                    acc = make_float4((float)ia.x * sc, (float)ia.y * sc, (float)ia.z * sc, (float)ia.w * sc);
                }
            }
            if (alive && part == 0 && !gave_up) {
                const __half2 h01 = __floats2half2_rn(acc.x, acc.y), h23 = __floats2half2_rn(acc.z, acc.w);
                uint2 o;
                o.x = *reinterpret_cast<const uint32_t *>(&h01);
                o.y = *reinterpret_cast<const uint32_t *>(&h23);
                int g = 0;
                if constexpr (GROUPED) {
#pragma unroll
                    for (int t = 1; t < kGemvMaxGroup; ++t) g += (t < p.count && n >= p.col0[t]) ? 1 : 0;
                }
                *reinterpret_cast<uint2 *>(p.y[g] + (size_t)m * p.Ng[g] + (n - p.col0[g])) = o;
            }
        }
        if (gave_up) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_TIMEOUT);
    }
}

template <int BITS, int MT, int S, int PRE, int HALF, int GROUPED, int ROLL, int HR, int INT = 0>
static tman_status launch_one(GemvParams p, int sms, cudaStream_t s)
{
    constexpr int W = HALF ? 16 : 32 / MT;
    constexpr int SUBS = 32 / W;
    // fp16 row pairs: the rows' scales follow the tables
    constexpr int kSmem = HALF ? kGemvTableBytes / 2 : kGemvTableBytes + (HR ? 64 : 0);
    const int words_total = p.K / 32;
    p.nkappa = (words_total + W - 1) / W;
    p.P = sms / p.nkappa;
    if (p.P < 1) p.P = 1;
    p.units = 0;
    for (int g = 0; g < p.count; ++g) {
        p.unit0[g] = p.units;
        p.units += (p.Ng[g] / 4 + S * SUBS - 1) / (S * SUBS);
    }
    for (int g = p.count; g < kGemvMaxGroup; ++g) p.unit0[g] = p.units;
    if (p.P > p.units) p.P = p.units;
    // every CTA must be resident while it polls for the others' partial sums
    if ((long long)p.nkappa * p.P > (long long)sms) return TMAN_ERR_UNSUPPORTED;
    int dev = 0, reserved = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&reserved, cudaDevAttrReservedSharedMemoryPerBlock, dev) != cudaSuccess)
        return TMAN_ERR_CUDA;
    if ((uint32_t)reserved != kGemvSmemBase) return TMAN_ERR_UNSUPPORTED;
    auto kern = mpgemv_kernel<BITS, MT, S, PRE, HALF, GROUPED, ROLL, HR, INT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess)
        return TMAN_ERR_CUDA;
    // the grid has at most one CTA per SM; the occupancy query says whether an SM can hold one at all
    // (asked once per device and variant)
    {
        constexpr int kMaxDevices = 64;
        static std::atomic<int> fits[kMaxDevices];          // 0 = not asked, 1 = fits, -1 = does not
        if (dev < 0 || dev >= kMaxDevices) return TMAN_ERR_CUDA;
        int f = fits[dev].load(std::memory_order_relaxed);
        if (f == 0) {
            int per_sm = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kGemvThreads, kSmem) != cudaSuccess)
                return TMAN_ERR_CUDA;
            f = per_sm >= 1 ? 1 : -1;
            fits[dev].store(f, std::memory_order_relaxed);
        }
        if (f < 0) return TMAN_ERR_UNSUPPORTED;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.P, (unsigned)p.nkappa);
    cfg.blockDim = dim3(kGemvThreads);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = s;
    // The kernel reads weights before it waits for its predecessor, so the call that follows a weight
    // packing on this stream keeps plain stream order.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = packed_write_pending(s, /*clear=*/true) ? 0 : 1;
    if (cudaLaunchKernelEx(&cfg, kern, p) != cudaSuccess) return TMAN_ERR_CUDA;
    return TMAN_OK;
}

template <int BITS, int MT, int PRE, int HR>
static tman_status launch_mt(GemvParams p, int sms, cudaStream_t s)
{
    // one row: fp32 tables over half-warp slices, large units; more rows: fp16 row pairs, smaller units
    // (measured: 2 strips per unit for up to four rows, 1 for eight).  All on one rolling set of registers.
    constexpr int ROLL = 1;
    constexpr int S = (HR && MT == 4) ? 1 : (HR && MT == 2) ? 2 : ((BITS == 2) ? 4 : 2);
    constexpr int HALF = HR ? 0 : 1;
    if (p.count > 1) return launch_one<BITS, MT, S, PRE, HALF, 1, ROLL, HR>(p, sms, s);
    return launch_one<BITS, MT, S, PRE, HALF, 0, ROLL, HR>(p, sms, s);
}

// ---- the plan: which kernel variants serve a call (host arithmetic only) -------------------------
// A variant carries up to `rows` activation rows per pass over the weights in K-slices of `words` plane
// words; its table entries have `slots` 32-bit slots (one fp32 row, or two fp16 rows each).  The time of a
// pass is modelled as fixed + per_mb x megabytes of bit planes; the constants were fitted to calls timed
// in a CUDA graph on a B200 (K = 4096, N = 14336; 2- and 4-bit for one row, 4-bit for the others):
//   rows 1: 6.9 / 9.7 us   rows 2: 10.7 us   rows 4: 14.9 us   rows 8: 23.6 us.
// The slope grows with the rows because an entry of 2 / 4 / 8 fp16 rows takes 1 / 2 / 4 shared-memory
// wavefronts per lookup.
struct GemvVariant { int rows, words, slots, half_slices; double fixed_us, us_per_mb; };
static const GemvVariant kGemvVariants[kGemvVariantCount] = {
    {1, 16, 1, 1, 4.10, 0.190},
    {2, 32, 1, 0, 4.35, 0.216},
    {4, 16, 2, 0, 4.85, 0.341},
    {8, 8, 4, 0, 5.85, 0.605},
};

static size_t variant_ws_bytes(const GemvVariant &v, int K, int N)
{
    // one fp32 partial sum per K-slice, row of the variant and column
    const size_t nkappa = (size_t)(K / 32 + v.words - 1) / (size_t)v.words;
    return kWsStatusBytes + nkappa * (size_t)v.rows * (size_t)N * sizeof(float);
}

// Limits a variant must meet on this device and call: its K-slices times at least one CTA each must be
// resident together (the CTAs poll one another's partial sums), its tables must fit the shared memory of
// an SM, and its partial sums must fit the caller's workspace.
static bool variant_feasible(const GemvVariant &v, int K, int N, int sms, size_t ws_limit)
{
    const int nkappa = (K / 32 + v.words - 1) / v.words;
    const int smem = (v.half_slices ? kGemvTableBytes / 2 : kGemvTableBytes) + 64;
    return nkappa <= sms && smem <= kGemvSmemLimit && variant_ws_bytes(v, K, N) <= ws_limit;
}

GemvPlan plan_gemv(int M, int K, int N, int bits, int sms, size_t ws_limit)
{
    // best[m]: least modelled time for m rows; a pass with variant v takes min(rows_v, m) of them
    const double plane_mb = (double)K * (double)N * bits / 8.0 / 1e6;
    double best[kGemvMaxRows + 1];
    int pick[kGemvMaxRows + 1];
    for (int m = 0; m <= kGemvMaxRows; ++m) { best[m] = 1e300; pick[m] = -1; }
    best[0] = 0.0;
    for (int m = 1; m <= M && m <= kGemvMaxRows; ++m) {
        best[m] = 1e300;
        pick[m] = -1;
        for (int vi = 0; vi < kGemvVariantCount; ++vi) {
            const GemvVariant &v = kGemvVariants[vi];
            if (!variant_feasible(v, K, N, sms, ws_limit)) continue;
            const int take = v.rows < m ? v.rows : m;
            if (take < v.rows && vi > 0 && kGemvVariants[vi - 1].rows >= take &&
                variant_feasible(kGemvVariants[vi - 1], K, N, sms, ws_limit))
                continue;                                   // a narrower variant carries these rows as well
            const double c = v.fixed_us + v.us_per_mb * plane_mb + best[m - take];
            if (c < best[m] - 1e-9) { best[m] = c; pick[m] = vi; }
        }
        if (pick[m] < 0) break;
    }
    GemvPlan g = {};
    if (M < 1 || M > kGemvMaxRows || pick[M] < 0) return g;      // npass == 0: no feasible plan
    g.cost_us = best[M];
    // widest passes first
    int left = M;
    while (left > 0) {
        const int vi = pick[left];
        const GemvVariant &v = kGemvVariants[vi];
        const int take = v.rows < left ? v.rows : left;
        GemvPass &ps = g.pass[g.npass++];
        ps.variant = vi;
        ps.rows = take;
        ps.variant_rows = v.rows;
        ps.words = v.words;
        ps.nkappa = (K / 32 + v.words - 1) / v.words;
        ps.ctas_per_slice = sms / ps.nkappa;
        ps.smem_bytes = v.half_slices ? kGemvTableBytes / 2 : kGemvTableBytes + 64;
        const size_t need = variant_ws_bytes(v, K, N);
        if (need > g.ws_bytes) g.ws_bytes = need;
        left -= take;
    }
    return g;
}

template <int BITS>
static tman_status launch_rows(GemvParams p, int rows, int variant, int sms, cudaStream_t s)
{
    p.M = rows;
    const bool pre = p.group >= 64;
    if (variant == 0) return pre ? launch_mt<BITS, 1, 1, 0>(p, sms, s) : launch_mt<BITS, 1, 0, 0>(p, sms, s);
    if (variant == 1) return pre ? launch_mt<BITS, 1, 1, 1>(p, sms, s) : launch_mt<BITS, 1, 0, 1>(p, sms, s);
    if (variant == 2) return pre ? launch_mt<BITS, 2, 1, 1>(p, sms, s) : launch_mt<BITS, 2, 0, 1>(p, sms, s);
    return pre ? launch_mt<BITS, 4, 1, 1>(p, sms, s) : launch_mt<BITS, 4, 0, 1>(p, sms, s);
}

__global__ void ws_fill_kernel(uint32_t *ws, size_t words)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < words) ws[i] = (i < kWsStatusBytes / 4) ? 0u : kGemvSentinel;
}

// One CTA waits, with the combine's own bounded wait, for partial sums that nothing will ever write (the
// workspace holds "no sum pending" after tman_workspace_init), gives up after `limit` polls and reports
// it the way the decode kernel does.  For testing that a wait that runs out ends cleanly.
__global__ void wait_timeout_kernel(float *partials, uint32_t *status, uint32_t limit)
{
    float4 t[4];
    const bool ready = wait_for_sums(reinterpret_cast<const float4 *>(partials) + threadIdx.x, 0, 0, 1, 1, limit, t);
    const bool gave_up = __any_sync(0xffffffffu, !ready);
    if (gave_up && threadIdx.x == 0) atomicCAS(status, 0u, (uint32_t)TMAN_ERR_TIMEOUT);
}

tman_status launch_wait_timeout(void *ws, size_t ws_bytes, uint32_t limit, cudaStream_t s)
{
    if (ws_bytes < kWsStatusBytes + 32 * sizeof(float4)) return TMAN_ERR_BUFFER_TOO_SMALL;
    uint8_t *w8 = static_cast<uint8_t *>(ws);
    wait_timeout_kernel<<<1, 32, 0, s>>>(reinterpret_cast<float *>(w8 + kWsStatusBytes), reinterpret_cast<uint32_t *>(w8), limit);
    return launch_status();
}

// status word (and its padding) zero, everything after it "no sum pending"
tman_status launch_workspace_init(void *ws, size_t ws_bytes, cudaStream_t s)
{
    const size_t words = ws_bytes / 4;
    ws_fill_kernel<<<(unsigned)((words + 255) / 256), 256, 0, s>>>(static_cast<uint32_t *>(ws), words);
    return launch_status();
}

size_t mpgemv_workspace_bytes(int M, int K, int N, int bits)
{
    // what the preferred plan needs (on the reference device size: the choice of variants depends on the
    // SM count only through the limit on K-slices); a smaller workspace makes the call fall back to
    // variants with fewer rows per pass, down to what one row needs
    const GemvPlan g = plan_gemv(M, K, N, bits, kGemvPlanSms, (size_t)-1);
    return g.npass ? g.ws_bytes : (size_t)-1;
}

tman_status launch_mpgemv_grouped(int count, const void *const *packed, const void *x, void *const *y, int M, int K,
                                  const int *Ns, int bits, int group, void *ws, size_t ws_bytes, cudaStream_t s)
{
    const int sms = sm_count();
    if (sms <= 0) return TMAN_ERR_CUDA;
    int ntot = 0;
    for (int g = 0; g < count; ++g) ntot += Ns[g];
    const GemvPlan plan = plan_gemv(M, K, ntot, bits, sms, ws_bytes);
    if (plan.npass == 0) return TMAN_ERR_UNSUPPORTED;
    uint8_t *w8 = static_cast<uint8_t *>(ws);
    GemvParams p;
    p.count = count;
    p.N = 0;
    for (int g = 0; g < kGemvMaxGroup; ++g) {
        const int gg = g < count ? g : 0;
        Layout L = make_layout(K, Ns[gg], bits, group);
        const uint8_t *pk = static_cast<const uint8_t *>(packed[gg]);
        p.packed[g] = pk;
        p.planes[g] = reinterpret_cast<const uint4 *>(pk + L.planes_off);
        p.scales[g] = reinterpret_cast<const uint2 *>(pk + L.scales_off);
        p.zeros[g] = reinterpret_cast<const uint16_t *>(pk + L.zeros_off);
        p.Ng[g] = g < count ? Ns[g] : 0;
        p.col0[g] = p.N;
        p.unit0[g] = 0;
        if (g < count) p.N += Ns[g];
    }
    p.status = reinterpret_cast<uint32_t *>(w8);
    p.partials = reinterpret_cast<float *>(w8 + kWsStatusBytes);
    p.xi = nullptr; p.row_scale = nullptr; p.w_scale = 0.f; p.acc_out = nullptr;
    p.K = K; p.bits = bits; p.group = group;
    p.M = 0; p.nkappa = 0; p.P = 0; p.units = 0;
    p.group_shift = (group == 32) ? 5 : (group == 64) ? 6 : 7;
    p.nblk = K / group;
    // a table entry carries up to eight rows (four fp16 pairs): normally one pass over the weights
    int m0 = 0;
    for (int ps = 0; ps < plan.npass; ++ps) {
        const int rows = plan.pass[ps].rows, variant = plan.pass[ps].variant;
        p.x = static_cast<const __half *>(x) + (size_t)m0 * K;
        for (int g = 0; g < kGemvMaxGroup; ++g)
            p.y[g] = static_cast<__half *>(y[g < count ? g : 0]) + (size_t)m0 * p.Ng[g];
        tman_status st;
        if (bits == 2) st = launch_rows<2>(p, rows, variant, sms, s);
        else if (bits == 3) st = launch_rows<3>(p, rows, variant, sms, s);
        else st = launch_rows<4>(p, rows, variant, sms, s);
        if (st != TMAN_OK) return st;
        m0 += rows;
    }
    return TMAN_OK;
}

// ---- integer path: per-tensor ternary weights, 16-bit integer activations ---------------------------
// Per-row symmetric quantization of the activations (paper Sec. 6.1, A_INT16; 8 bits for the matrix unit):
// s_a = max|x| / qmax and a = round(x / s_a), both in single precision with correctly rounded division and
// rounding to nearest even, so that the integers are the same on any IEEE machine.  One CTA per row.
template <typename OUT>      // int16_t or int8_t
__global__ void __launch_bounds__(1024) quantize_rows_kernel(const __half *__restrict__ x, int K, int qmax,
                                                             OUT *__restrict__ a, float *__restrict__ s_a)
{
    __shared__ float red[32];
    const __half *row = x + (size_t)blockIdx.x * K;
    OUT *out = a + (size_t)blockIdx.x * K;
    // eight values per thread and step when the row allows 16-byte accesses (K % 8 == 0, checked by the host)
    const bool vec = (K & 7) == 0;
    const int nvec = vec ? K >> 3 : 0;
    float amax = 0.f;
    for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
        const uint4 q = __ldg(reinterpret_cast<const uint4 *>(row) + i);
        const __half2 *h = reinterpret_cast<const __half2 *>(&q);
        __half2 m = __hmax2(__hmax2(__habs2(h[0]), __habs2(h[1])), __hmax2(__habs2(h[2]), __habs2(h[3])));
        amax = fmaxf(amax, fmaxf(__low2float(m), __high2float(m)));
    }
    for (int k = 8 * nvec + threadIdx.x; k < K; k += blockDim.x) amax = fmaxf(amax, fabsf(__half2float(row[k])));
    for (int mask = 16; mask > 0; mask >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, mask));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x < 32) {
        float v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
        for (int mask = 16; mask > 0; mask >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, mask));
        if (threadIdx.x == 0) red[0] = v;
    }
    __syncthreads();
    amax = red[0];
    const float scale = amax > 0.f ? __fdiv_rn(amax, (float)qmax) : 1.f;
    if (threadIdx.x == 0) s_a[blockIdx.x] = scale;
    auto quant = [&](__half v) {
        const int r = __float2int_rn(__fdiv_rn(__half2float(v), scale));
        return (int)max(-qmax, min(qmax, r));
    };
    for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
        const uint4 q = __ldg(reinterpret_cast<const uint4 *>(row) + i);        // second read: from L1/L2
        const __half *h = reinterpret_cast<const __half *>(&q);
        if constexpr (sizeof(OUT) == 2) {
            uint4 o;
            o.x = (uint32_t)(quant(h[0]) & 0xFFFF) | ((uint32_t)quant(h[1]) << 16);
            o.y = (uint32_t)(quant(h[2]) & 0xFFFF) | ((uint32_t)quant(h[3]) << 16);
            o.z = (uint32_t)(quant(h[4]) & 0xFFFF) | ((uint32_t)quant(h[5]) << 16);
            o.w = (uint32_t)(quant(h[6]) & 0xFFFF) | ((uint32_t)quant(h[7]) << 16);
            reinterpret_cast<uint4 *>(out)[i] = o;
        } else {
            uint2 o;
            o.x = (uint32_t)(quant(h[0]) & 0xFF) | ((uint32_t)(quant(h[1]) & 0xFF) << 8) |
                  ((uint32_t)(quant(h[2]) & 0xFF) << 16) | ((uint32_t)quant(h[3]) << 24);
            o.y = (uint32_t)(quant(h[4]) & 0xFF) | ((uint32_t)(quant(h[5]) & 0xFF) << 8) |
                  ((uint32_t)(quant(h[6]) & 0xFF) << 16) | ((uint32_t)quant(h[7]) << 24);
            reinterpret_cast<uint2 *>(out)[i] = o;
        }
    }
    for (int k = 8 * nvec + threadIdx.x; k < K; k += blockDim.x) out[k] = (OUT)quant(row[k]);
}

tman_status launch_quantize_rows(const void *x, int M, int K, int qmax, int16_t *a, float *s_a, cudaStream_t s)
{
    const int threads = K >= 8192 ? 1024 : (K >= 2048 ? 512 : 256);
    quantize_rows_kernel<int16_t><<<(unsigned)M, threads, 0, s>>>(static_cast<const __half *>(x), K, qmax, a, s_a);
    return launch_status();
}

tman_status launch_quantize_rows_i8(const void *x, int M, int K, int8_t *a, float *s_a, cudaStream_t s)
{
    const int threads = K >= 8192 ? 1024 : (K >= 2048 ? 512 : 256);
    quantize_rows_kernel<int8_t><<<(unsigned)M, threads, 0, s>>>(static_cast<const __half *>(x), K, 127, a, s_a);
    return launch_status();
}

// Rows of 16-bit integer activations times ternary weights packed as 2-bit codes (zero-point 1; the
// packed buffer's scales and zero-points are not read).  y = fp16(s_a[m] * s_w * sum), acc_out (may be NULL)
// receives the exact integer sums.  Integer table entries are held exactly in fp32, one per row: passes of
// one row (K-slices of 16 plane words), two rows (16 words) or four rows (8 words) per table entry.
static void ternary_variant(int rows, int *mt, int *words)
{
    if (rows <= 1) { *mt = 1; *words = 16; }
    else if (rows == 2) { *mt = 2; *words = 16; }
    else { *mt = 4; *words = 8; }
}

size_t mpgemv_ternary_workspace_bytes(int M, int K, int N)
{
    int mt = 1, words = 16;
    ternary_variant(M < 4 ? M : 4, &mt, &words);
    const size_t nkappa = (size_t)(K / 32 + words - 1) / (size_t)words;
    return kWsStatusBytes + nkappa * (size_t)mt * (size_t)N * sizeof(float);
}

tman_status launch_mpgemv_ternary(const void *packed, const int16_t *a, const float *s_a, float s_w, void *y,
                                  int32_t *acc_out, int M, int K, int N, int group, void *ws, size_t, cudaStream_t s)
{
    const int sms = sm_count();
    if (sms <= 0) return TMAN_ERR_CUDA;
    uint8_t *w8 = static_cast<uint8_t *>(ws);
    GemvParams p = {};
    p.count = 1;
    Layout L = make_layout(K, N, 2, group);
    const uint8_t *pk = static_cast<const uint8_t *>(packed);
    for (int g = 0; g < kGemvMaxGroup; ++g) {
        p.packed[g] = pk;
        p.planes[g] = reinterpret_cast<const uint4 *>(pk + L.planes_off);
        p.scales[g] = reinterpret_cast<const uint2 *>(pk + L.scales_off);
        p.zeros[g] = reinterpret_cast<const uint16_t *>(pk + L.zeros_off);
        p.Ng[g] = g == 0 ? N : 0;
        p.col0[g] = g == 0 ? 0 : N;
    }
    p.N = N;
    p.x = nullptr;
    p.w_scale = s_w;
    p.status = reinterpret_cast<uint32_t *>(w8);
    p.partials = reinterpret_cast<float *>(w8 + kWsStatusBytes);
    p.K = K; p.bits = 2; p.group = group;
    p.group_shift = (group == 32) ? 5 : (group == 64) ? 6 : 7;
    p.nblk = K / group;
    const bool pre = group >= 64;
    for (int m0 = 0; m0 < M; m0 += 4) {
        const int rows = (M - m0 < 4) ? (M - m0) : 4;
        int mt = 1, words = 16;
        ternary_variant(rows, &mt, &words);
        if ((K / 32 + words - 1) / words > sms) return TMAN_ERR_UNSUPPORTED;      // every K-slice needs a resident CTA
        p.M = rows;
        p.xi = a + (size_t)m0 * K;
        p.row_scale = s_a + m0;
        p.acc_out = acc_out ? acc_out + (size_t)m0 * N : nullptr;
        for (int g = 0; g < kGemvMaxGroup; ++g) p.y[g] = static_cast<__half *>(y) + (size_t)m0 * N;
        tman_status st;
        if (mt == 1) st = pre ? launch_one<2, 1, 4, 1, 1, 0, 1, 0, 1>(p, sms, s) : launch_one<2, 1, 4, 0, 1, 0, 1, 0, 1>(p, sms, s);
        else if (mt == 2) st = pre ? launch_one<2, 2, 2, 1, 0, 0, 1, 0, 1>(p, sms, s) : launch_one<2, 2, 2, 0, 0, 0, 1, 0, 1>(p, sms, s);
        else st = pre ? launch_one<2, 4, 1, 1, 0, 0, 1, 0, 1>(p, sms, s) : launch_one<2, 4, 1, 0, 0, 0, 1, 0, 1>(p, sms, s);
        if (st != TMAN_OK) return st;
    }
    return TMAN_OK;
}

tman_status launch_mpgemv(const void *packed, const void *x, void *y, int M, int K, int N, int bits,
                          int group, void *ws, size_t ws_bytes, cudaStream_t s)
{
    return launch_mpgemv_grouped(1, &packed, x, &y, M, K, &N, bits, group, ws, ws_bytes, s);
}

}  // namespace tman
