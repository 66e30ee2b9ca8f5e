// Prefill path: two-level lookup dequantization fused into a tcgen05 GEMM
// (paper Sec. 4.1 "Unified Layout through Fused LUT-based Dequantization", Fig. 7;
//  Sec. 4.2 "Pipelining to Hide Dequantization Overhead", Fig. 9).
//
// The output is cut into tiles of up to 256 channels x 128*MH tokens (one CTA, at most 128 tokens) or
// 256*MH tokens (a pair of CTAs on two SMs).  A tile's work is its K/64 k-blocks.  The host chooses
// how many column tiles there are and deals the tiles to the workers (CTAs or pairs, at most one per
// SM or SM pair), whole as far as they go round; where whole tiles would leave SMs idle, the
// k-blocks of the last tiles are laid end to end and dealt in equal spans, and a tile whose
// k-blocks fall into several spans is summed through fp32 partial tiles in the workspace (see
// "split of the work").
// Four kinds of agents run concurrently on a ring of shared-memory stages guarded by mbarriers (the
// paper's DMA / vector-core / matrix-core stages):
//   * warp 0, one lane : TMA loads of the fp16 activation tile (128-byte swizzle) and of the packed
//                        bit-plane words of the weight tile (one box per plane);
//   * warps 2..17      : read the staged plane words of their column, rebuild the codes
//                        (level 1: bit-serial -> bit-parallel), look every code up in the
//                        per-(block, column) conversion table kept in registers and addressed
//                        with byte-permute instructions (level 2: scale and zero-point baked in),
//                        and write the fp16 weight tile in the K-major swizzled layout the
//                        tensor core reads;
//   * warp 1, one lane : tcgen05.mma (fp16 x fp16 -> fp32 in tensor memory), one per row block and
//                        16 k; tcgen05.commit hands the stage back;
//   * warps 18..25     : epilogue (tcgen05.ld, round to fp16, stage in shared memory, TMA tile store).
// CTA pairs (more than 128 tokens): each CTA holds its own 128*MH token rows and dequantizes half of
// the tile's channels, and the pair multiplies with tcgen05.mma.cta_group::2 (M = 256), issued by the
// pair's first CTA: every weight is rebuilt once per 256*MH tokens and each SM reads half of the
// weight tile per MMA.  Barriers that both CTAs feed (weight tile ready, accumulator drained) live in
// the first CTA; the MMA's commits arrive in both.  No TMA multicast: each CTA loads its own tiles.
// Every wait is bounded: when a bound is hit the kernel records TMAN_ERR_TIMEOUT, stops issuing
// work, and still reaches the common tear-down that frees tensor memory.
#include "common.cuh"

#include <mutex>

#include <cuda.h>

#include "sm100_ptx.cuh"

namespace tman {
namespace {

constexpr int BM = 128, BK = 64, BN = 256;      // token rows of a row block, k-block, channels of a tile
constexpr int A_HALF_BYTES = BM * BK * 2;
constexpr int NUM_DEQ_WARPS = 16;               // each fills 16 columns of a weight tile
constexpr int NUM_EPI_WARPS = 8;                // two per quarter of the tensor-memory lanes (alternate 32-column chunks)
constexpr int GEMM_THREADS = 32 * (2 + NUM_DEQ_WARPS + NUM_EPI_WARPS);
constexpr int OUT_TILE_BYTES = 32 * 32 * 2;     // an epilogue warp's output staging: 32 tokens x 32 channels
constexpr int CHUNK_BYTES = 32 * 32 * 4;        // the same chunk as fp32 partial sums
constexpr int PART_RING = 4;                    // partial chunks an epilogue warp keeps in flight when it sums a split tile
constexpr int kMaxGemmCtas = 160;               // the workspace is sized for at most this many CTAs

template <int MH, bool PAIR> struct Cfg {
    static constexpr int NCTA = PAIR ? 2 : 1;
    static constexpr int BN_CTA = BN / NCTA;                          // channels a CTA dequantizes
    static constexpr int NSTAGE = PAIR ? 4 : 3;
    static constexpr int A_STAGE_BYTES = MH * A_HALF_BYTES;
    static constexpr int B_STAGE_BYTES = BN_CTA * BK * 2;
    static constexpr int P_PLANE_BYTES = (BN_CTA / 4) * (BK / 32) * 16;   // one plane of a CTA's packed tile
    static constexpr int TMEM_COLS = MH * BN;                         // one fp32 accumulator of BN columns per row block
    static constexpr int smem_bytes(int bits)
    {
        // stages (multiples of 1 KB, so the staging tiles stay 1 KB aligned), staging, barriers.  The kernel
        // has no static shared memory, so the dynamic part starts 1 KB aligned (checked in the kernel).
        return NSTAGE * (A_STAGE_BYTES + B_STAGE_BYTES + bits * P_PLANE_BYTES) + NUM_EPI_WARPS * OUT_TILE_BYTES + 512;
    }
};

// Workspace: status word (kWsStatusBytes), one flag per epilogue warp of every CTA (spans), one flag
// per (epilogue warp of a CTA, sending piece) (even split), then one fp32 partial tile per CTA (spans: a
// worker writes at most one per launch; even split: the chunks the other pieces send to this CTA).
constexpr int kMaxSplit = 8;                    // pieces of a tile in the even split
constexpr size_t kGemmFlagsOff = kWsStatusBytes;
constexpr size_t kGemmFlags2Off = kWsStatusBytes + 8192;
constexpr size_t kGemmPartialOff = kGemmFlags2Off + 40960;
constexpr uint32_t kFlagEmpty = 0x7FA5A5A5u;    // what tman_workspace_init leaves behind
// Role time stamps (only in a library built with -DTMAN_ROLE_STAMPS; the workspace has room for them in
// every build so that its layout does not depend on the flag): per CTA and warp four 64-bit words --
// clocks spent in the role's first kind of wait, in its second kind, in the whole role, and a tag.
//   warp 0 (TMA producer): waits for a free stage            warp 1 (MMA issuer): accumulator free / stage dequantized
//   warps 2..17 (dequantization): stage loaded               warps 18..25 (epilogue): accumulators complete
constexpr int kStampWordsPerWarp = 4;
constexpr int kGemmWarps = 2 + NUM_DEQ_WARPS + NUM_EPI_WARPS;
constexpr size_t kStampBytesPerCta = (size_t)kGemmWarps * kStampWordsPerWarp * sizeof(long long);
#ifdef TMAN_ROLE_STAMPS
#define TMAN_STAMPED_WAIT(acc, call) ([&]() { const long long t_ = clock64(); const bool r_ = (call); (acc) += clock64() - t_; return r_; }())
#else
#define TMAN_STAMPED_WAIT(acc, call) (call)
#endif
constexpr size_t kPartialBytesPerCta = (size_t)NUM_EPI_WARPS * 2 * (BN / 64) * CHUNK_BYTES;   // 256 KB, whatever MH

struct GemmParams {
    const uint8_t  *packed;
    const uint32_t *planes;
    const __half   *scales;
    const uint16_t *zeros;
    uint32_t       *status;
    uint32_t       *flags;
    uint32_t       *flags2;
    float          *partial;
    int M, K, N, bits, group;
    int tiles_m, tiles_n;
    int span_tiles;            // the last span_tiles tiles are dealt as equal spans of k-blocks (0: every tile whole)
    int split_s;               // even split: every tile's k-blocks go to split_s workers (0: off)
    int col_fastest;           // tile number = row tile * tiles_n + column tile (else column tile * tiles_m + row tile)
    long long *stamps;         // role time stamps (written only by a build with TMAN_ROLE_STAMPS)
};

// (PTX wrappers: sm100_ptx.cuh)

// ---- level 2: per-(block, column) conversion table in registers ------------------------------
// Entry c holds fp16( s * (c - z) ) (paper Sec. 4.1: integer-to-float conversion with scale and
// zero-point pre-applied, 2^bits entries per quantization block).  Low and high bytes of the
// entries are kept in separate byte tables so that one byte-permute looks up four codes.
template <int BITS>
struct ConvTable {
    static constexpr int NQ = (BITS == 4) ? 4 : ((BITS == 3) ? 2 : 1);
    uint32_t lo[NQ], hi[NQ];

    // entry c = fp16(s * (c - z)): c - z is a small integer (exact in fp16), so one half-precision
    // multiply rounds once, like the fp32 product rounded to fp16 would
    __device__ __forceinline__ void build(__half s, uint32_t z)
    {
        const __half2 s2 = __half2half2(s);
        const __half2 z2 = __half2half2(__ushort2half_rn((unsigned short)z));
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            const __half2 c01 = __floats2half2_rn((float)(4 * q + 0), (float)(4 * q + 1));
            const __half2 c23 = __floats2half2_rn((float)(4 * q + 2), (float)(4 * q + 3));
            const __half2 e01 = __hmul2(s2, __hsub2(c01, z2));
            const __half2 e23 = __hmul2(s2, __hsub2(c23, z2));
            const uint32_t h01 = *reinterpret_cast<const uint32_t *>(&e01);
            const uint32_t h23 = *reinterpret_cast<const uint32_t *>(&e23);
            lo[q] = __byte_perm(h01, h23, 0x6420);
            hi[q] = __byte_perm(h01, h23, 0x7531);
        }
    }

    // sel: four codes in the four low nibbles.  Returns the four low bytes / high bytes.
    __device__ __forceinline__ void lookup(uint32_t sel, uint32_t &lb, uint32_t &hb) const
    {
        if constexpr (BITS <= 2) {
            lb = __byte_perm(lo[0], lo[0], sel);
            hb = __byte_perm(hi[0], hi[0], sel);
        } else if constexpr (BITS == 3) {
            lb = __byte_perm(lo[0], lo[1], sel);
            hb = __byte_perm(hi[0], hi[1], sel);
        } else {
            const uint32_t sel7 = sel & 0x7777u;
            // byte mask: 0xFF where the code's top bit is set (sign-replicating selectors)
            const uint32_t mask = prmt(sel, sel << 4, 0x9D8Cu);
            const uint32_t la = __byte_perm(lo[0], lo[1], sel7), lc = __byte_perm(lo[2], lo[3], sel7);
            const uint32_t ha = __byte_perm(hi[0], hi[1], sel7), hc = __byte_perm(hi[2], hi[3], sel7);
            lb = (la & ~mask) | (lc & mask);
            hb = (ha & ~mask) | (hc & mask);
        }
    }
};

// Ablation variants of the kernel (paper Sec. 6.5 "Ablation Study"): what replaces the table lookup of the
// dequantization, or the pipelining.  Every variant computes the same numbers.
constexpr int kGemmProduct = 0;      // two-level lookup dequantization, pipelined (the product path)
constexpr int kGemmConvertDq = 1;    // codes converted to floating point one by one, then subtract and multiply
constexpr int kGemmLoadFull = 2;     // fp16 weights prepared in memory and loaded by TMA, no dequantization
constexpr int kGemmSequential = 3;   // the product's dequantization with a ring of one stage: load, dequantize, multiply in turn

// The same 32 weights without the conversion table: every code is extracted, converted to fp16 by an
// integer-to-float conversion, the zero-point subtracted and the scale multiplied (rounds like the table's
// entries do, so the result is the same bits).
template <int BITS>
__device__ __forceinline__ void dequant_word_convert(const uint32_t (&w)[BITS], __half s, uint32_t z, uint32_t (&out)[16])
{
    const __half2 s2 = __half2half2(s);
    const __half2 z2 = __half2half2(__ushort2half_rn((unsigned short)z));
#pragma unroll
    for (int ph = 0; ph < 4; ++ph)
#pragma unroll
        for (int jp = 0; jp < 4; ++jp) {
            // weights 8*ph + 2*jp and 8*ph + 2*jp + 1 sit at word bits 4*(2*jp) + ph and 4*(2*jp + 1) + ph
            uint32_t c0 = 0u, c1 = 0u;
#pragma unroll
            for (int i = 0; i < BITS; ++i) {
                c0 |= ((w[i] >> (8 * jp + ph)) & 1u) << i;
                c1 |= ((w[i] >> (8 * jp + 4 + ph)) & 1u) << i;
            }
            const __half2 c = __halves2half2(__ushort2half_rn((unsigned short)c0), __ushort2half_rn((unsigned short)c1));
            const __half2 e = __hmul2(s2, __hsub2(c, z2));
            out[4 * ph + jp] = *reinterpret_cast<const uint32_t *>(&e);
        }
}

// 32 weights of one column (one plane word per bit) -> 16 half2 in k order.
template <int BITS>
__device__ __forceinline__ void dequant_word(const uint32_t (&w)[BITS], const ConvTable<BITS> &T, uint32_t (&out)[16])
{
    // level 1 (bit repacking): X[ph] nibble j = code of the weight at word bit 4j + ph, which the
    // packed format makes weight 8*ph + j: X[ph] holds weights 8ph .. 8ph+7 in order.  A 4 x 4
    // bit-block transpose of the plane words: first planes 0/1 and 2/3 are interleaved bit by bit,
    // then the two results two bits by two bits (each step is one shift and one bit-select).
    auto bsel = [](uint32_t m, uint32_t a, uint32_t b) { return (a & m) | (b & ~m); };
    uint32_t X[4];
    {
        const uint32_t w0 = w[0], w1 = w[1];
        const uint32_t a0 = bsel(0x55555555u, w0, w1 << 1), a1 = bsel(0x55555555u, w0 >> 1, w1);
        if constexpr (BITS > 2) {
            const uint32_t w2 = w[2], w3 = (BITS > 3) ? w[BITS - 1] : 0u;
            const uint32_t b0 = bsel(0x55555555u, w2, w3 << 1), b1 = bsel(0x55555555u, w2 >> 1, w3);
            X[0] = bsel(0x33333333u, a0, b0 << 2);
            X[2] = bsel(0x33333333u, a0 >> 2, b0);
            X[1] = bsel(0x33333333u, a1, b1 << 2);
            X[3] = bsel(0x33333333u, a1 >> 2, b1);
        } else {
            X[0] = a0 & 0x33333333u;
            X[2] = (a0 >> 2) & 0x33333333u;
            X[1] = a1 & 0x33333333u;
            X[3] = (a1 >> 2) & 0x33333333u;
        }
    }
    // level 2 (conversion table): four codes per lookup, then low and high bytes are interleaved
    // into two half2 of adjacent weights
#pragma unroll
    for (int ph = 0; ph < 4; ++ph)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t lb, hb;
            T.lookup(X[ph] >> (16 * h), lb, hb);
            out[4 * ph + 2 * h]     = __byte_perm(lb, hb, 0x5140);    // weights k0, k0+1   (k0 = 8ph + 4h)
            out[4 * ph + 2 * h + 1] = __byte_perm(lb, hb, 0x7362);    // weights k0+2, k0+3
        }
}

// ---- split of the work ----------------------------------------------------------------------
// T tiles (row tile fastest), W workers.  The first `whole` tiles (a multiple of W) are dealt whole,
// round-robin.  The k-blocks of the remaining tiles (fewer than 2 W), laid end to end in units of two
// k-blocks (a 128-wide quantization block is never cut), are dealt in equal contiguous spans, so
// every worker is busy to the end whatever the shape.  A span is shorter than two tiles: at most
// the end of one tile, one whole tile and the start of the next.  A tile cut into several pieces
// ("split tile") is summed by the worker that owns its last unit: the others, which all have lower
// numbers, write their fp32 accumulators to the workspace and raise a flag.  A worker's walk: first
// the piece that it only contributes (so that it is ready long before it is needed), then its whole
// tiles, last the piece of the tile that it finishes.
// Even split (outputs with fewer tiles than half the workers): every tile's k-blocks are cut into S
// equal pieces for S workers with consecutive numbers.  They finish together; each sends the fp32 chunks
// that another piece sums into that piece's inbox in the workspace, raises one flag per receiver, then
// fetches what it was sent and adds it to its own accumulators in piece order: the summing and its
// traffic are shared by all S workers instead of falling on one.
struct Segment { int tile, kb0, kb1; bool whole, finishes; };

struct Span {
    long long full, Ur;        // tiles dealt whole round-robin; units of the remaining tiles
    long long next_whole;      // next round-robin tile of this worker
    int nu, W, w;
    Segment early, mid, late;  // the piece this worker only contributes; a whole tile of its span; the piece it finishes
    bool has_early, has_mid, has_late;
    __device__ Span(const GemmParams &p, int worker, int nworkers)
        : nu(p.K / (2 * BK)), W(nworkers), w(worker), has_early(false), has_mid(false), has_late(false)
    {
        const long long T = (long long)p.tiles_m * p.tiles_n;
        if (p.split_s) {
            // even split: worker w has piece w % S of tile w / S and nothing else
            full = 0;
            Ur = 0;
            next_whole = 0;
            const int S = p.split_s, piece = worker % S;
            late.tile = worker / S;
            late.kb0 = 2 * (int)((long long)nu * piece / S);
            late.kb1 = 2 * (int)((long long)nu * (piece + 1) / S);
            late.whole = false;
            late.finishes = true;
            has_late = true;
            return;
        }
        full = T - p.span_tiles;
        Ur = (long long)p.span_tiles * nu;
        next_whole = worker;
        long long lo = Ur * worker / nworkers, hi = Ur * (worker + 1) / nworkers;
        for (int i = 0; i < 3 && hi > lo; ++i) {       // from the last tile of the span to the first
            const long long tile = (hi - 1) / nu, t0 = tile * nu;
            const long long k0 = (lo > t0) ? lo - t0 : 0, k1 = hi - t0;
            Segment s;
            s.tile = (int)(full + tile);
            s.kb0 = 2 * (int)k0;
            s.kb1 = 2 * (int)k1;
            s.whole = (k0 == 0 && k1 == nu);
            s.finishes = (k1 == nu);
            if (s.whole) { mid = s; has_mid = true; }
            else if (s.finishes) { late = s; has_late = true; }
            else { early = s; has_early = true; }
            hi = t0 + k0;
        }
    }
    __device__ bool next(Segment &s)
    {
        if (has_early) { s = early; has_early = false; return true; }
        if (next_whole < full) {
            s.tile = (int)next_whole;
            s.kb0 = 0;
            s.kb1 = 2 * nu;
            s.whole = s.finishes = true;
            next_whole += W;
            return true;
        }
        if (has_mid) { s = mid; has_mid = false; return true; }
        if (has_late) { s = late; has_late = false; return true; }
        return false;
    }
    // the worker that owns unit u of tile `tile` (one of the remaining tiles)
    __device__ int owner(int tile, int u) const
    {
        const long long g = (long long)(tile - full) * nu + u;
        return (int)(((g + 1) * W - 1) / Ur);
    }
};

template <int BITS, int MH, bool PAIR, int V>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
mpgemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
              const __grid_constant__ CUtensorMap tmap_y, const __grid_constant__ CUtensorMap tmap_wf, const GemmParams p)
{
    using C = Cfg<MH, PAIR>;
    constexpr int RING = (V == kGemmSequential) ? 1 : C::NSTAGE;      // stages of the ring in use
    constexpr int NCTA = C::NCTA, NSTAGE = C::NSTAGE, A_STAGE_BYTES = C::A_STAGE_BYTES, B_STAGE_BYTES = C::B_STAGE_BYTES;
    constexpr int P_PLANE_BYTES = C::P_PLANE_BYTES, P_STAGE_BYTES = BITS * P_PLANE_BYTES, TMEM_COLS = C::TMEM_COLS;
    constexpr int ROWS_CTA = BM * MH;                  // token rows of a tile held by one CTA
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;   // in a pair, CTA 0 issues the MMAs and owns the shared barriers
    if (!header_matches(p.packed, p.K, p.N, p.bits, p.group)) {   // same answer in every CTA
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_BAD_PACKED);
        return;
    }
    if ((smem_u32(smem) & 1023u) != 0u) {              // the swizzled tiles need 1 KB alignment (same in every CTA)
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_LAYOUT);
        return;
    }
    uint8_t *a_tiles = smem;
    uint8_t *b_tiles = smem + NSTAGE * A_STAGE_BYTES;
    uint8_t *p_tiles = smem + NSTAGE * (A_STAGE_BYTES + B_STAGE_BYTES);
    uint8_t *out_tiles = smem + NSTAGE * (A_STAGE_BYTES + B_STAGE_BYTES + P_STAGE_BYTES);
    uint64_t *bars = reinterpret_cast<uint64_t *>(out_tiles + NUM_EPI_WARPS * OUT_TILE_BYTES);
    // bars[0..NSTAGE) loaded (own TMA), [NSTAGE..2NSTAGE) full (dequantized; in a pair both CTAs' warps
    // arrive in CTA 0), [2NSTAGE..3NSTAGE) empty (MMA commit), then accumulator full (commit) and
    // accumulator empty (epilogue warps; in a pair both CTAs' warps arrive in CTA 0)
    // and PART_RING barriers per epilogue warp for the partial chunks it fetches
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * NSTAGE + 2 + NUM_EPI_WARPS * PART_RING);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = p.K / BK;
    const uint32_t loaded0 = smem_u32(bars), full0 = smem_u32(bars + NSTAGE), empty0 = smem_u32(bars + 2 * NSTAGE),
                   accf = smem_u32(bars + 3 * NSTAGE), acce = smem_u32(bars + 3 * NSTAGE + 1),
                   ring0 = smem_u32(bars + 3 * NSTAGE + 2);

    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(loaded0 + 8 * s, 1);
            mbar_init(full0 + 8 * s, NCTA * NUM_DEQ_WARPS);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accf, 1);
        mbar_init(acce, NCTA * NUM_EPI_WARPS);
        for (int b = 0; b < NUM_EPI_WARPS * PART_RING; ++b) mbar_init(ring0 + 8 * b, 1);
        *tmem_slot = 0xFFFFFFFFu;
        fence_barrier_init();
    }
    __syncthreads();
    if (warp == 1) {
        if constexpr (PAIR) {
            tcgen05_alloc2(smem_u32(tmem_slot), TMEM_COLS);
            tcgen05_relinquish2();
        } else {
            tcgen05_alloc(smem_u32(tmem_slot), TMEM_COLS);
            tcgen05_relinquish();
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();            // both CTAs' barriers and tensor memory are set up
    tcgen05_fence_after();
    uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(tmem_slot);
    if constexpr (PAIR)
        if (tmem_base == 0xFFFFFFFFu) tmem_base = ld_shared_cluster_u32(mapa_u32(smem_u32(tmem_slot), rank ^ 1u));

    bool ok = tmem_base != 0xFFFFFFFFu;
    long long wait_a = 0, wait_b = 0;                  // clocks in this thread's waits (time-stamp builds only)
#ifdef TMAN_ROLE_STAMPS
    const long long role_t0 = clock64();
#endif
    const int worker = (int)blockIdx.x / NCTA, nworkers = (int)gridDim.x / NCTA;
    Span span(p, worker, nworkers);
    Segment sg;
    // a tile's place in the output, the channels this CTA dequantizes (a pair halves the tile's channels;
    // the last tile of a row may be narrower: a multiple of 32 channels that reaches N)
    // Tiles with consecutive numbers run at the same time; the host numbers them so that a round of
    // tiles touches the fewest bytes (row tiles of activations, column tiles of packed weights).
    auto tile_tm = [&](int tile) { return p.col_fastest ? tile / p.tiles_n : tile % p.tiles_m; };
    auto tile_ct = [&](int tile) { return p.col_fastest ? tile % p.tiles_n : tile / p.tiles_m; };
    auto tile_rows = [&](int tile) { return tile_tm(tile) * (NCTA * ROWS_CTA) + (int)rank * ROWS_CTA; };
    // (the N/32 column units are cut into tiles_n column tiles of almost equal width, at most BN)
    const int n32 = (p.N + 31) / 32;
    auto tile_unit0 = [&](int ct) { return (int)(((long long)n32 * ct) / p.tiles_n); };
    auto tile_col0 = [&](int tile) { return 32 * tile_unit0(tile_ct(tile)); };
    auto tile_bn = [&](int tile) { const int ct = tile_ct(tile); return 32 * (tile_unit0(ct + 1) - tile_unit0(ct)); };
    const uint32_t full_lead = PAIR ? mapa_u32(full0, 0) : full0, acce_lead = PAIR ? mapa_u32(acce, 0) : acce;
    auto arrive_lead = [&](uint32_t bar) {
        if constexpr (PAIR) mbar_arrive_cluster(bar);
        else mbar_arrive(bar);
    };

    if (warp == 0) {
        // ---- stage 1: this CTA's activation rows and packed channels by TMA ---------------------
        if (lane == 0) {
            uint32_t it = 0;
            while (ok && span.next(sg)) {
                const int row0 = tile_rows(sg.tile);
                const int strip0 = (tile_col0(sg.tile) + (int)rank * (tile_bn(sg.tile) / NCTA)) / 4;
                for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++it) {
                    const int s = (int)(it % RING);
                    const uint32_t ph = (it / RING) & 1u;
                    if (!TMAN_STAMPED_WAIT(wait_a, mbar_wait(empty0 + 8 * s, ph ^ 1u))) { ok = false; break; }
                    if constexpr (V == kGemmLoadFull) {
                        // the fp16 weight tile itself: this CTA's channels x one k-block, 128-byte swizzle
                        mbar_expect_tx(loaded0 + 8 * s, A_STAGE_BYTES + B_STAGE_BYTES);
                        tma_load_2d(smem_u32(a_tiles + s * A_STAGE_BYTES), &tmap_x, kb * BK, row0, loaded0 + 8 * s);
                        tma_load_2d(smem_u32(b_tiles + s * B_STAGE_BYTES), &tmap_wf, kb * BK, strip0 * 4, loaded0 + 8 * s);
                    } else {
                        mbar_expect_tx(loaded0 + 8 * s, A_STAGE_BYTES + P_STAGE_BYTES);
                        tma_load_2d(smem_u32(a_tiles + s * A_STAGE_BYTES), &tmap_x, kb * BK, row0, loaded0 + 8 * s);
#pragma unroll
                        for (int i = 0; i < BITS; ++i)
                            tma_load_3d(smem_u32(p_tiles + s * P_STAGE_BYTES + i * P_PLANE_BYTES), &tmap_w, kb * (BK / 8), i,
                                        strip0, loaded0 + 8 * s);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---- stage 3: tensor-core MMA (in a pair: issued by CTA 0 for both) ----------------------
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, ti = 0;
            while (ok && span.next(sg)) {
                if (!TMAN_STAMPED_WAIT(wait_a, mbar_wait(acce, (ti & 1u) ^ 1u))) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t idesc = (1u << 4) | ((uint32_t)(tile_bn(sg.tile) >> 3) << 17) | ((uint32_t)((NCTA * BM) >> 4) << 24);
                for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++it) {
                    const int s = (int)(it % RING);
                    const uint32_t ph = (it / RING) & 1u;
                    if (!TMAN_STAMPED_WAIT(wait_b, mbar_wait(full0 + 8 * s, ph))) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint64_t bdesc = make_kmajor_sw128_desc(smem_u32(b_tiles + s * B_STAGE_BYTES));
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j)
#pragma unroll
                        for (int h = 0; h < MH; ++h) {
                            const uint64_t adesc = make_kmajor_sw128_desc(smem_u32(a_tiles + s * A_STAGE_BYTES + h * A_HALF_BYTES));
                            const uint32_t acc = (kb > sg.kb0 || j > 0) ? 1u : 0u;
                            if constexpr (PAIR) tcgen05_mma2_f16(tmem_base + (uint32_t)(h * BN), adesc + 2 * j, bdesc + 2 * j, idesc, acc);
                            else tcgen05_mma_f16(tmem_base + (uint32_t)(h * BN), adesc + 2 * j, bdesc + 2 * j, idesc, acc);
                        }
                    if constexpr (PAIR) tcgen05_commit2_both(empty0 + 8 * s);
                    else tcgen05_commit(empty0 + 8 * s);
                }
                if (ok) {
                    if constexpr (PAIR) tcgen05_commit2_both(accf);
                    else tcgen05_commit(accf);
                }
                ++ti;
            }
        }
    } else if (warp < 2 + NUM_DEQ_WARPS) {
        // ---- stage 2: two-level lookup dequantization of this CTA's channels ----------------------
        // A warp owns 16 channels and both plane words of a k-block: lane = (strip of the warp, word,
        // column of the strip).  With this split the 32 lanes read 32 different banks of the staged
        // plane words and write eight different 16-byte bank groups per quarter-warp.  When a CTA has at
        // most 128 channels of a tile (always in a pair), eight warps cover them: the two halves of the
        // sixteen warps then take turns, two k-blocks each.
        const int wd16 = warp - 2;
        const int sl = lane >> 3, v = (lane >> 2) & 1, c = lane & 3;
        const int nblk = p.K / p.group;
        const int gshift = (p.group == 32) ? 5 : (p.group == 64) ? 6 : 7;
        auto block_of = [&](int kb) { return ((2 * kb + v) * 32) >> gshift; };

        uint32_t it = 0;
        while (ok && span.next(sg)) {
            const int chans = tile_bn(sg.tile) / NCTA;
            const int ngroup = (PAIR || chans <= BN / 2) ? 2 : 1;
            const int wd = wd16 % (NUM_DEQ_WARPS / ngroup), grp = wd16 / (NUM_DEQ_WARPS / ngroup);
            const int n_local = wd * 16 + sl * 4 + c;
            const uint32_t p_off = (uint32_t)(wd * 4 + sl) * 32u + (uint32_t)v * 16u + (uint32_t)c * 4u;
            const uint32_t row_off = (uint32_t)(n_local >> 3) * 1024u + (uint32_t)(n_local & 7) * 128u;
            const uint32_t xr = (uint32_t)(n_local & 7);
            const uint32_t p_base = smem_u32(p_tiles) + p_off, b_base = smem_u32(b_tiles) + row_off;
            // k-blocks this warp works on, by pipeline position (segments start at even k-blocks)
            auto mine = [&](uint32_t i) { return ngroup == 1 || (int)((i >> 1) & 1u) == grp; };
            const int n = tile_col0(sg.tile) + (int)rank * chans + n_local;
            const bool valid = n_local < chans && n < p.N;   // channels past the tile are not used by the MMA
            const int nb = n >> 2;
            const __half *ps = p.scales + (size_t)nb * nblk * 4 + c;
            const uint16_t *pz = p.zeros + (size_t)nb * nblk;
            auto fetch_sz = [&](int B, __half &sv, uint32_t &zz) {
                sv = __float2half(0.f);
                zz = 0u;
                if (valid && B < nblk) {
                    sv = __ldg(ps + (size_t)B * 4);
                    zz = ((uint32_t)__ldg(pz + B) >> (4 * c)) & 0xFu;
                }
            };
            ConvTable<BITS> T;
            int cur_B = -1, next_B = -1;
            __half sv_next = __float2half(0.f), sv_cur = __float2half(0.f);
            uint32_t zz_next = 0u, zz_cur = 0u;
            for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++it) {
                const int s = (int)(it % RING);
                const uint32_t ph = (it / RING) & 1u;
                const bool work = (V != kGemmLoadFull) && valid && mine(it);
                if (work) {
                    const int Bk = block_of(kb);
                    if (Bk != cur_B) {
                        if (next_B != Bk) fetch_sz(Bk, sv_next, zz_next);
                        cur_B = Bk;
                        sv_cur = sv_next;
                        zz_cur = zz_next;
                        if constexpr (V != kGemmConvertDq) T.build(sv_next, zz_next);
                    }
                    // scale and zero-point of the block after this one are fetched one k-block ahead
                    const int kn = (ngroup == 1 || !(kb & 1)) ? kb + 1 : kb + 3;
                    const int Bn = block_of(kn);
                    if (kn < sg.kb1 && Bn != cur_B && Bn != next_B) {
                        next_B = Bn;
                        fetch_sz(Bn, sv_next, zz_next);
                    }
                }
                if (!TMAN_STAMPED_WAIT(wait_a, mbar_wait(loaded0 + 8 * s, ph))) { ok = false; break; }
                if (work) {
                    uint32_t w[BITS];
                    const uint32_t pp = p_base + (uint32_t)s * P_STAGE_BYTES;
#pragma unroll
                    for (int i = 0; i < BITS; ++i)
                        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w[i]) : "r"(pp + i * P_PLANE_BYTES) : "memory");
                    uint32_t out[16];
                    if constexpr (V == kGemmConvertDq) dequant_word_convert<BITS>(w, sv_cur, zz_cur, out);
                    else dequant_word<BITS>(w, T, out);
                    const uint32_t row = b_base + (uint32_t)s * B_STAGE_BYTES;
#pragma unroll
                    for (int cj = 0; cj < 4; ++cj) {
                        const uint32_t chunk = ((uint32_t)(4 * v + cj)) ^ xr;
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(row + chunk * 16u), "r"(out[4 * cj]),
                                     "r"(out[4 * cj + 1]), "r"(out[4 * cj + 2]), "r"(out[4 * cj + 3]) : "memory");
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) arrive_lead(full_lead + 8 * s);
            }
        }
    } else {
        // ---- epilogue: this CTA's rows of a segment's accumulators ------------------------------------
        // A warp reads chunks of 32 tokens x 32 channels (one token per lane; a warp may only read its
        // quarter of the tensor-memory lanes).  Whole tiles and the finishing segment of a split tile:
        // round to fp16, write 64-byte rows into the warp's staging tile in the 64-byte swizzle (16-byte
        // chunk index ^ bits 1..2 of the row: no bank conflicts), one lane stores the tile (tokens >= M
        // and channels >= N are clipped by the store).  Split tiles: the other segments write the fp32
        // chunks to this CTA's partial tile and raise the warp's flag.  The finishing segment, always
        // the last of its worker's walk, waits for the flags of the same warp in the workers before it,
        // fetches their chunks with bulk copies into the pipeline's stage buffers (free by then; a ring
        // of PART_RING chunks per warp keeps enough bytes in flight) and adds them in worker order.
        const int quarter = warp & 3;
        const int ew = warp - 2 - NUM_DEQ_WARPS, epart = ew >> 2;
        const uint32_t stage = smem_u32(out_tiles + ew * OUT_TILE_BYTES);
        const uint32_t my_row = stage + (uint32_t)lane * 64u, xr = ((uint32_t)lane >> 1) & 3u;
        const uint32_t ring_buf = smem_u32(smem) + (uint32_t)ew * (PART_RING * CHUNK_BYTES);
        const uint32_t ring_bar = ring0 + 8u * (uint32_t)(ew * PART_RING);
        constexpr size_t WARP_PARTIAL_FLOATS = (size_t)MH * (BN / 64) * (CHUNK_BYTES / 4);
        static_assert(NUM_EPI_WARPS * PART_RING * CHUNK_BYTES <= NSTAGE * A_STAGE_BYTES + NSTAGE * B_STAGE_BYTES, "ring fits in the stages");
        auto warp_partial = [&](int cta) { return p.partial + (size_t)cta * (kPartialBytesPerCta / 4) + (size_t)ew * WARP_PARTIAL_FLOATS; };
        auto warp_flag = [&](int cta) { return p.flags + (size_t)cta * NUM_EPI_WARPS + ew; };
        uint32_t ti = 0;
        while (ok && span.next(sg)) {
            const int bn = tile_bn(sg.tile), col0 = tile_col0(sg.tile), rows0 = tile_rows(sg.tile);
            // this warp's chunks: nch column chunks for each of the hv row blocks that reach below M
            const int nch = (bn - 32 * epart + 63) / 64;
            int hv = 0;
            for (int h = 0; h < MH; ++h) hv += (rows0 + h * BM + quarter * 32 < p.M) ? 1 : 0;
            const int nq = hv * nch;
            // split tile: the workers before this one that hold the tile's other segments
            int first_w = worker;
            if (!p.split_s && sg.finishes && !sg.whole) first_w = span.owner(sg.tile, 0);
            const int ncontrib = worker - first_w;
            if (!TMAN_STAMPED_WAIT(wait_a, mbar_wait(accf, ti & 1u))) { ok = false; break; }
            tcgen05_fence_after();
            if (p.split_s) {
                // ---- even split: the S workers of a tile finish together and share the summing -----------
                // Chunk q of this warp is summed by piece q % S.  A piece first sends the chunks that
                // others sum (fp32, into their CTA's inbox, slot = (sender, chunk)) and raises one flag
                // per receiver; then it fetches what the others sent for its own chunks and adds them to
                // its accumulators in piece order.
                const int S = p.split_s, me = worker % S, w0 = worker - me;
                const int CH = (MH * (BN / 64) + S - 1) / S;           // chunks a piece sums, at most
                auto inbox = [&](int cta, int sender, int slot) {
                    const int sidx = sender < (cta / NCTA) % S ? sender : sender - 1;
                    return p.partial + (size_t)cta * (kPartialBytesPerCta / 4) +
                           ((size_t)(sidx * CH + slot) * NUM_EPI_WARPS + ew) * (CHUNK_BYTES / 4);
                };
                auto flag2 = [&](int cta, int sender) { return p.flags2 + ((size_t)cta * NUM_EPI_WARPS + ew) * kMaxSplit + sender; };
#pragma unroll 1
                for (int q = 0; q < nq; ++q) {
                    if (q % S == me) continue;
                    uint32_t r[32];
                    tcgen05_ld_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) +
                                          (uint32_t)((q / nch) * BN + 32 * epart + 64 * (q % nch)), r);
                    tcgen05_wait_ld();
                    float4 *dst = reinterpret_cast<float4 *>(inbox((w0 + q % S) * NCTA + (int)rank, me, q / S)) + lane;
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        __stcg(dst + 32 * e, make_float4(__uint_as_float(r[4 * e]), __uint_as_float(r[4 * e + 1]),
                                                         __uint_as_float(r[4 * e + 2]), __uint_as_float(r[4 * e + 3])));
                }
                __threadfence();
                __syncwarp();
                if (lane == 0)
                    for (int o = 0; o < S; ++o)
                        if (o != me)
                            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(flag2((w0 + o) * NCTA + (int)rank, me)), "r"(1u) : "memory");
                // own chunks: items (own chunk c, other piece o) in that order
                const int nown = (nq > me) ? (nq - me + S - 1) / S : 0, nitem = nown * (S - 1);
                auto other = [&](int i) { return i < me ? i : i + 1; };      // i-th other piece
                auto fetch2 = [&](int jj) {
                    const int c = jj / (S - 1), o = other(jj % (S - 1));
                    const uint32_t b = (uint32_t)(jj % PART_RING);
                    mbar_expect_tx(ring_bar + 8 * b, CHUNK_BYTES);
                    bulk_load(ring_buf + b * CHUNK_BYTES, inbox((int)blockIdx.x, o, c), CHUNK_BYTES, ring_bar + 8 * b);
                };
                if (lane == 0) {
                    for (int i = 0; i < S - 1 && ok; ++i) {
                        const uint32_t *f = flag2((int)blockIdx.x, other(i));
                        uint64_t t0 = 0;
                        for (uint32_t spin = 0;; ++spin) {
                            uint32_t fv;
                            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(fv) : "l"(f) : "memory");
                            if (fv == 1u) break;
                            if ((spin & 255u) == 255u) {
                                const uint64_t now = global_timer_ns();
                                if (t0 == 0) t0 = now;
                                else if (now - t0 > 1000000000ull) { ok = false; break; }
                            }
                        }
                    }
                    if (ok) {
                        asm volatile("fence.proxy.async.global;" ::: "memory");
                        for (int jj = 0; jj < PART_RING && jj < nitem; ++jj) fetch2(jj);
                    }
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                int jj = 0;
#pragma unroll 1
                for (int c = 0; c < nown; ++c) {
                    const int q = me + c * S;
                    const int h = q / nch, col = 32 * epart + 64 * (q % nch);
                    const int m0 = rows0 + h * BM + quarter * 32;
                    uint32_t r[32];
                    tcgen05_ld_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(h * BN + col), r);
                    tcgen05_wait_ld();
#pragma unroll 1
                    for (int i = 0; i < S - 1; ++i, ++jj) {
                        const uint32_t b = (uint32_t)(jj % PART_RING);
                        if (!mbar_wait(ring_bar + 8 * b, (uint32_t)(jj / PART_RING) & 1u)) { ok = false; break; }
                        const uint32_t src = ring_buf + b * CHUNK_BYTES + (uint32_t)lane * 16u;
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            float4 a;
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w)
                                         : "r"(src + 512u * e) : "memory");
                            r[4 * e]     = __float_as_uint(__uint_as_float(r[4 * e]) + a.x);
                            r[4 * e + 1] = __float_as_uint(__uint_as_float(r[4 * e + 1]) + a.y);
                            r[4 * e + 2] = __float_as_uint(__uint_as_float(r[4 * e + 2]) + a.z);
                            r[4 * e + 3] = __float_as_uint(__uint_as_float(r[4 * e + 3]) + a.w);
                        }
                        __syncwarp();
                        if (lane == 0 && jj + PART_RING < nitem) fetch2(jj + PART_RING);
                    }
                    if (!ok) break;
                    uint32_t hv16[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const __half2 hh = __floats2half2_rn(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1]));
                        hv16[e] = *reinterpret_cast<const uint32_t *>(&hh);
                    }
                    if (lane == 0) tma_store_wait_read();
                    __syncwarp();
#pragma unroll
                    for (uint32_t cj = 0; cj < 4; ++cj)
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(my_row + ((cj ^ xr) << 4)), "r"(hv16[4 * cj]),
                                     "r"(hv16[4 * cj + 1]), "r"(hv16[4 * cj + 2]), "r"(hv16[4 * cj + 3]) : "memory");
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) tma_store_2d(&tmap_y, stage, col0 + col, m0);
                }
                if (!ok) break;
                // the accumulators are read; the received flags go back to "empty" for the next launch
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) {
                    arrive_lead(acce_lead);
                    for (int i = 0; i < S - 1; ++i) *flag2((int)blockIdx.x, other(i)) = kFlagEmpty;
                }
                ++ti;
                continue;
            }
            // issue the fetch of item j = (chunk q, contributor c) into the ring (lane 0)
            auto fetch = [&](int j) {
                const int q = j / ncontrib, cw = first_w + j % ncontrib;
                const size_t off = (size_t)((q / nch) * (BN / 64) + (q % nch)) * (CHUNK_BYTES / 4);
                const uint32_t b = (uint32_t)(j % PART_RING);
                mbar_expect_tx(ring_bar + 8 * b, CHUNK_BYTES);
                bulk_load(ring_buf + b * CHUNK_BYTES, warp_partial(cw * NCTA + (int)rank) + off, CHUNK_BYTES, ring_bar + 8 * b);
            };
            if (ncontrib > 0) {
                // their partial tiles were written at the start of their walks; bounded wait all the same
                if (lane == 0) {
                    for (int cw = first_w; cw < worker && ok; ++cw) {
                        const uint32_t *f = warp_flag(cw * NCTA + (int)rank);
                        uint64_t t0 = 0;
                        for (uint32_t spin = 0;; ++spin) {
                            uint32_t fv;
                            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(fv) : "l"(f) : "memory");
                            if (fv == 1u) break;
                            if ((spin & 255u) == 255u) {
                                const uint64_t now = global_timer_ns();
                                if (t0 == 0) t0 = now;
                                else if (now - t0 > 1000000000ull) { ok = false; break; }
                            }
                        }
                    }
                    if (ok) {
                        asm volatile("fence.proxy.async.global;" ::: "memory");
                        for (int j = 0; j < PART_RING && j < nq * ncontrib; ++j) fetch(j);
                    }
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
            }
            float *mine_partial = warp_partial((int)blockIdx.x);
            if (nq == 0) {                             // a warp without a chunk in this tile
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) arrive_lead(acce_lead);
            }
            int j = 0;                                 // next item of the ring to consume
#pragma unroll 1
            for (int q = 0; q < nq; ++q) {
                const int h = q / nch, col = 32 * epart + 64 * (q % nch);
                const int m0 = rows0 + h * BM + quarter * 32;
                uint32_t r[32];
                tcgen05_ld_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(h * BN + col), r);
                tcgen05_wait_ld();
                if (q == nq - 1) {                     // the accumulators are read: the next segment's MMAs may start
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) arrive_lead(acce_lead);
                }
                if (!sg.finishes) {
                    // chunk as eight rows of 32 float4: coalesced, and fetched back as one 4 KB block
                    float4 *dst = reinterpret_cast<float4 *>(mine_partial + (size_t)(h * (BN / 64) + (q % nch)) * (CHUNK_BYTES / 4)) + lane;
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        __stcg(dst + 32 * e, make_float4(__uint_as_float(r[4 * e]), __uint_as_float(r[4 * e + 1]),
                                                         __uint_as_float(r[4 * e + 2]), __uint_as_float(r[4 * e + 3])));
                    continue;
                }
#pragma unroll 1
                for (int c = 0; c < ncontrib; ++c, ++j) {
                    const uint32_t b = (uint32_t)(j % PART_RING);
                    if (!mbar_wait(ring_bar + 8 * b, (uint32_t)(j / PART_RING) & 1u)) { ok = false; break; }
                    const uint32_t src = ring_buf + b * CHUNK_BYTES + (uint32_t)lane * 16u;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        float4 a;
                        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w)
                                     : "r"(src + 512u * e) : "memory");
                        r[4 * e]     = __float_as_uint(__uint_as_float(r[4 * e]) + a.x);
                        r[4 * e + 1] = __float_as_uint(__uint_as_float(r[4 * e + 1]) + a.y);
                        r[4 * e + 2] = __float_as_uint(__uint_as_float(r[4 * e + 2]) + a.z);
                        r[4 * e + 3] = __float_as_uint(__uint_as_float(r[4 * e + 3]) + a.w);
                    }
                    __syncwarp();                      // every lane has read the buffer: it may be refilled
                    if (lane == 0 && j + PART_RING < nq * ncontrib) fetch(j + PART_RING);
                }
                if (!ok) break;
                uint32_t hv16[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const __half2 hh = __floats2half2_rn(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1]));
                    hv16[e] = *reinterpret_cast<const uint32_t *>(&hh);
                }
                if (lane == 0) tma_store_wait_read();              // the staging tile is free again
                __syncwarp();
#pragma unroll
                for (uint32_t cj = 0; cj < 4; ++cj)
                    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(my_row + ((cj ^ xr) << 4)), "r"(hv16[4 * cj]),
                                 "r"(hv16[4 * cj + 1]), "r"(hv16[4 * cj + 2]), "r"(hv16[4 * cj + 3]) : "memory");
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) tma_store_2d(&tmap_y, stage, col0 + col, m0);
            }
            if (!ok) break;
            if (!sg.finishes) {
                // partial tile complete: every lane's stores, then the flag
                __threadfence();
                __syncwarp();
                if (lane == 0) asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(warp_flag((int)blockIdx.x)), "r"(1u) : "memory");
            } else if (ncontrib > 0) {
                // the partial tiles are consumed: their flags go back to "empty" for the next launch
                __syncwarp();
                if (lane == 0)
                    for (int cw = first_w; cw < worker; ++cw) *warp_flag(cw * NCTA + (int)rank) = kFlagEmpty;
            }
            ++ti;
        }
        if (lane == 0) tma_store_wait_all();
    }

    if (!ok) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_TIMEOUT);
    tcgen05_fence_before();
#ifdef TMAN_ROLE_STAMPS
    if (lane == 0 && p.stamps != nullptr) {
        long long *st = p.stamps + ((size_t)blockIdx.x * kGemmWarps + warp) * kStampWordsPerWarp;
        st[0] = wait_a;
        st[1] = wait_b;
        st[2] = clock64() - role_t0;
        st[3] = 0x5354414D50ll;                        // "STAMP": this build writes time stamps
    }
#else
    (void)wait_a; (void)wait_b;
#endif
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();            // nobody touches the peer's memory after this
    if (warp == 1 && tmem_base != 0xFFFFFFFFu) {
        tcgen05_fence_after();
        if constexpr (PAIR) tcgen05_dealloc2(tmem_base, TMEM_COLS);
        else tcgen05_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---- host side ---------------------------------------------------------------------------
// Row blocks per CTA and single CTAs or pairs, from the number of tokens: one CTA up to 128 tokens,
// pairs of one row block each up to 256, pairs of two row blocks each beyond.
inline int gemm_mh(int M) { return M > 2 * BM ? 2 : 1; }
inline bool gemm_pair(int M) { return M > BM; }

// How a call's work is cut (host).  One worker per SM (pair of SMs), fewer when there is less work
// than that.  The channels are cut into column tiles of almost equal width (multiples of 32, at
// most 256) and the tiles dealt whole; the number of column tiles is the one with the least
// estimated time for the longest worker: rounds of tiles x k-blocks x time of a k-block, which for
// a pair hardly falls below 192 channels (the MMA's activation operand bounds it) and for a single
// CTA is a latency chain plus the dequantization's share, in proportion to the width (measured
// figures, microseconds: pair 0.74 / 0.76 / 0.87 at 128 / 192 / 256 channels, single CTA 0.51 / 0.59 /
// 0.77 / 1.11 at 32 / 64 / 128 / 256).  The
// alternative: the widest tiles, whole as far as they go round and the rest in equal spans, whose
// split tiles cost their workers a partial tile written to and read back from the workspace (an SM
// writes about 50 GB/s; the more pieces per tile, the more to read back).
struct GemmPlan { int pair, mh, tiles_m, tiles_n, span_tiles, workers, col_fastest, split_s; };

// `resident`: how many workers (CTAs, or CTA pairs) of the chosen kernel the device can hold at the
// same time.  Workers wait for one another's partial tiles, so no more than that may be launched.
GemmPlan plan_gemm(int M, int K, int N, int bits, int sms, int resident)
{
    GemmPlan g;
    g.pair = gemm_pair(M) ? 1 : 0;
    g.mh = gemm_mh(M);
    const int ncta = g.pair ? 2 : 1, rows = ncta * BM * g.mh;
    g.tiles_m = (M + rows - 1) / rows;
    const long long nu = K / (2 * BK);
    long long workers = (sms < kMaxGemmCtas ? sms : kMaxGemmCtas) / ncta;
    if (workers > resident) workers = resident;
    if (workers < 1) workers = 1;
    const int n32 = (N + 31) / 32, tn_min = (n32 + BN / 32 - 1) / (BN / 32);
    const bool pair = g.pair != 0;
    auto kb_us = [pair](int width) {
        const double w = (double)width;
        if (pair) return w <= 192 ? 0.70 + 0.0003 * w : 0.7576 + 0.00175 * (w - 192);
        return 0.42 + 0.0027 * w;
    };
    double best = 1e300;
    g.span_tiles = 0;
    g.tiles_n = tn_min;
    for (int tn = tn_min; tn <= n32 && tn <= 8 * tn_min; ++tn) {
        const long long rounds = ((long long)g.tiles_m * tn + workers - 1) / workers;
        const int wmax = 32 * ((n32 + tn - 1) / tn);
        const double cost = (double)rounds * (2.0 * nu * kb_us(wmax) + 3.0);
        if (cost <= best + 1e-9) { best = cost; g.tiles_n = tn; }     // ties: more, narrower tiles
    }
    {
        // widest tiles; the remainder of the last round is cut into spans, together with one whole
        // round when the remainder alone would be cut into many pieces per tile
        const long long t = (long long)g.tiles_m * tn_min, rest = t % workers;
        const long long span = (rest != 0 && rest < workers / 2 && t > workers) ? rest + workers : rest;
        const double cost = (double)((t - span) / workers) * (2.0 * nu * kb_us(BN) + 3.0) +
                            (double)((span * nu + workers - 1) / workers) * 2.0 * kb_us(BN) +
                            (span ? (pair ? 24.0 : 16.0) + 3.0 * (double)workers / (double)span : 0.0);
        if (span != 0 && cost < best) {
            best = cost;
            g.span_tiles = (int)span;
            g.tiles_n = tn_min;
        }
    }
    g.split_s = 0;
    {
        // fewer widest tiles than half the workers: every tile's k-blocks to S workers (even pieces), which
        // finish together and share the summing
        const long long t = (long long)g.tiles_m * tn_min;
        const int nq_warp = g.mh * (BN / 64);           // chunks an epilogue warp holds
        for (int S = 2; S <= kMaxSplit; ++S) {
            if (t * S > workers || nu < S) break;
            if ((S - 1) * ((nq_warp + S - 1) / S) > 8) continue;    // what the pieces send to one CTA must fit its inbox
            const double cost = (double)((nu + S - 1) / S) * 2.0 * kb_us(BN) + 3.0 +
                                (pair ? 9.0 + 3.0 * (S - 1) : 8.0 + 1.3 * (S - 1));   // measured exchange times
            if (cost < best) {
                best = cost;
                g.split_s = S;
                g.span_tiles = 0;
                g.tiles_n = tn_min;
            }
        }
    }
    const long long tiles = (long long)g.tiles_m * g.tiles_n;
    if (g.split_s) workers = tiles * g.split_s;
    else if (tiles < workers) {                        // fewer tiles than workers: as many workers as units at most
        const long long units = g.span_tiles ? tiles * nu : tiles;
        if (workers > units) workers = units;
    }
    g.workers = (int)workers;
    // tile numbering: bytes a round of `workers` consecutive tiles touches, either way
    {
        const double a_tile = (double)rows * K * 2.0, b_tile = (double)N / g.tiles_n * K * bits / 8.0;
        const long long rows_r = g.tiles_m < workers ? g.tiles_m : workers, cols_r = (workers + g.tiles_m - 1) / g.tiles_m;
        const long long cols_c = g.tiles_n < workers ? g.tiles_n : workers, rows_c = (workers + g.tiles_n - 1) / g.tiles_n;
        g.col_fastest = (rows_c * a_tile + cols_c * b_tile < rows_r * a_tile + cols_r * b_tile) ? 1 : 0;
    }
    return g;
}

template <int BITS, int MH, bool PAIR, int V>
tman_status launch_cfg(const CUtensorMap &tmap_x, const CUtensorMap &tmap_w, const CUtensorMap &tmap_y, const CUtensorMap &tmap_wf,
                       const GemmParams &p, int workers, cudaStream_t s)
{
    using C = Cfg<MH, PAIR>;
    auto kern = mpgemm_kernel<BITS, MH, PAIR, V>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::smem_bytes(BITS)) != cudaSuccess)
        return TMAN_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(workers * C::NCTA));
    cfg.blockDim = dim3(GEMM_THREADS);
    cfg.dynamicSmemBytes = C::smem_bytes(BITS);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C::NCTA;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, tmap_x, tmap_w, tmap_y, tmap_wf, p) != cudaSuccess) return TMAN_ERR_CUDA;
    return TMAN_OK;
}

template <int BITS, int V>
tman_status launch_bits(const CUtensorMap &tmap_x, const CUtensorMap &tmap_w, const CUtensorMap &tmap_y, const CUtensorMap &tmap_wf,
                        const GemmParams &p, const GemmPlan &g, cudaStream_t s)
{
    if (!g.pair) return launch_cfg<BITS, 1, false, V>(tmap_x, tmap_w, tmap_y, tmap_wf, p, g.workers, s);
    if (g.mh == 1) return launch_cfg<BITS, 1, true, V>(tmap_x, tmap_w, tmap_y, tmap_wf, p, g.workers, s);
    return launch_cfg<BITS, 2, true, V>(tmap_x, tmap_w, tmap_y, tmap_wf, p, g.workers, s);
}

// Workers of one kernel variant that can be resident together on the current device (occupancy query,
// once per device and variant).
template <int BITS, int MH, bool PAIR>
int resident_cfg(int sms)
{
    using C = Cfg<MH, PAIR>;
    auto kern = mpgemm_kernel<BITS, MH, PAIR, kGemmProduct>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::smem_bytes(BITS)) != cudaSuccess) return -1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(sms / C::NCTA * C::NCTA));
    cfg.blockDim = dim3(GEMM_THREADS);
    cfg.dynamicSmemBytes = C::smem_bytes(BITS);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C::NCTA;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) return -1;
    return n;
}

int resident_workers(int M, int bits, int sms)
{
    constexpr int kMaxDevices = 64;
    static std::mutex lock;
    static int cache[kMaxDevices][3][3];     // [device][bits - 2][variant], 0 = not asked yet
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices || bits < 2 || bits > 4) return -1;
    const int variant = !gemm_pair(M) ? 0 : (gemm_mh(M) == 1 ? 1 : 2);
    std::lock_guard<std::mutex> guard(lock);
    int &slot = cache[dev][bits - 2][variant];
    if (slot == 0) {
        int n = -1;
        if (bits == 2) n = variant == 0 ? resident_cfg<2, 1, false>(sms) : variant == 1 ? resident_cfg<2, 1, true>(sms) : resident_cfg<2, 2, true>(sms);
        if (bits == 3) n = variant == 0 ? resident_cfg<3, 1, false>(sms) : variant == 1 ? resident_cfg<3, 1, true>(sms) : resident_cfg<3, 2, true>(sms);
        if (bits == 4) n = variant == 0 ? resident_cfg<4, 1, false>(sms) : variant == 1 ? resident_cfg<4, 1, true>(sms) : resident_cfg<4, 2, true>(sms);
        if (n < 1) return -1;                 // not cached: asked again next time
        slot = n;
    }
    return slot;
}

}  // namespace

tman_status mpgemm_plan_for(int M, int K, int N, int bits, int sms, int resident, int *out8)
{
    const GemmPlan g = plan_gemm(M, K, N, bits, sms, resident);
    out8[0] = g.pair; out8[1] = g.mh; out8[2] = g.tiles_m; out8[3] = g.tiles_n; out8[4] = (g.span_tiles || g.split_s) ? 0 : 1; out8[5] = g.workers;
    out8[6] = g.span_tiles; out8[7] = g.split_s;
    return TMAN_OK;
}

tman_status mpgemm_plan(int M, int K, int N, int bits, int *out8)
{
    const int sms = sm_count();
    if (sms <= 0) return TMAN_ERR_CUDA;
    const int resident = resident_workers(M, bits, sms);
    if (resident < 1) return TMAN_ERR_CUDA;
    return mpgemm_plan_for(M, K, N, bits, sms, resident, out8);
}

size_t mpgemm_workspace_bytes(int M, int, int)
{
    (void)M;
    return kGemmPartialOff + (size_t)kMaxGemmCtas * (kPartialBytesPerCta + kStampBytesPerCta);
}

// Copies the role time stamps of the last prefill call out of the workspace (host buffer of
// ctas x 26 warps x 4 words).  Only a library built with TMAN_ROLE_STAMPS writes them.
tman_status mpgemm_read_stamps(const void *ws, int ctas, long long *out_host, cudaStream_t s)
{
#ifdef TMAN_ROLE_STAMPS
    if (ctas < 1 || ctas > kMaxGemmCtas) return TMAN_ERR_SHAPE;
    const uint8_t *src = static_cast<const uint8_t *>(ws) + kGemmPartialOff + (size_t)kMaxGemmCtas * kPartialBytesPerCta;
    if (cudaMemcpyAsync(out_host, src, (size_t)ctas * kStampBytesPerCta, cudaMemcpyDeviceToHost, s) != cudaSuccess) return TMAN_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return TMAN_ERR_CUDA;
    return TMAN_OK;
#else
    (void)ws; (void)ctas; (void)out_host; (void)s;
    return TMAN_ERR_UNSUPPORTED;
#endif
}

tman_status launch_mpgemm(const void *packed, const void *x, void *y, int M, int K, int N, int bits,
                          int group, void *ws, size_t ws_bytes, cudaStream_t s)
{
    return launch_mpgemm_variant(kGemmProduct, packed, x, y, M, K, N, bits, group, nullptr, ws, ws_bytes, s);
}

// variant: one of kGemmProduct .. kGemmSequential; wt_f16: for kGemmLoadFull the dequantized weights as fp16
// [N][K] (channel-major), otherwise unused.  The variants other than the product path exist for 4-bit only.
tman_status launch_mpgemm_variant(int variant, const void *packed, const void *x, void *y, int M, int K, int N, int bits,
                                  int group, const void *wt_f16, void *ws, size_t, cudaStream_t s)
{
    if (variant < kGemmProduct || variant > kGemmSequential) return TMAN_ERR_UNSUPPORTED;
    if (variant != kGemmProduct && bits != 4) return TMAN_ERR_UNSUPPORTED;
    if (variant == kGemmLoadFull && (!wt_f16 || (reinterpret_cast<uintptr_t>(wt_f16) & 15) != 0)) return TMAN_ERR_SHAPE;
    if (variant == kGemmLoadFull && (N % 32) != 0) return TMAN_ERR_UNSUPPORTED;     // whole 32-channel units only
    if ((reinterpret_cast<uintptr_t>(x) & 15) != 0 || (reinterpret_cast<uintptr_t>(y) & 15) != 0) return TMAN_ERR_SHAPE;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return TMAN_ERR_CUDA;
    const int sms = sm_count();
    if (sms <= 0) return TMAN_ERR_CUDA;
    const int resident = resident_workers(M, bits, sms);
    if (resident < 1) return TMAN_ERR_CUDA;
    const GemmPlan g = plan_gemm(M, K, N, bits, sms, resident);
    const bool pair = g.pair != 0;
    const int rows_cta = BM * g.mh, bn_cta = pair ? BN / 2 : BN;
    const cuuint32_t estr[3] = {1, 1, 1};

    // activations: boxes of one k-block x a CTA's token rows, 128-byte swizzle
    CUtensorMap tmap_x;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
        const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
        const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)rows_cta};
        if (enc(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(x), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TMAN_ERR_CUDA;
    }
    Layout L = make_layout(K, N, bits, group);
    const uint8_t *pk = static_cast<const uint8_t *>(packed);
    // the bit-plane words as a 3-D array of 32-bit elements: (word and column inside a strip's plane
    // row, plane, strip); one box = the two words of a k-block for the strips of a CTA's channels, one plane
    CUtensorMap tmap_w;
    {
        const cuuint64_t wt = (cuuint64_t)(K / 32);
        const cuuint64_t wdims[3] = {wt * 4, (cuuint64_t)bits, (cuuint64_t)(N / 4)};
        const cuuint64_t wstrides[2] = {wt * 16, wt * 16 * (cuuint64_t)bits};
        const cuuint32_t wbox[3] = {(cuuint32_t)(BK / 8), 1, (cuuint32_t)(bn_cta / 4)};
        if (enc(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint8_t *>(pk + L.planes_off), wdims, wstrides,
                wbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TMAN_ERR_CUDA;
    }
    // the output as 32 x 32 tiles in the 64-byte swizzle (the epilogue's stores)
    CUtensorMap tmap_y;
    {
        const cuuint64_t ydims[2] = {(cuuint64_t)N, (cuuint64_t)M};
        const cuuint64_t ystrides[1] = {(cuuint64_t)N * 2};
        const cuuint32_t ybox[2] = {32, 32};
        if (enc(&tmap_y, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, y, ydims, ystrides, ybox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TMAN_ERR_CUDA;
    }

    uint8_t *w8 = static_cast<uint8_t *>(ws);
    GemmParams p;
    p.packed = pk;
    p.planes = reinterpret_cast<const uint32_t *>(pk + L.planes_off);
    p.scales = reinterpret_cast<const __half *>(pk + L.scales_off);
    p.zeros = reinterpret_cast<const uint16_t *>(pk + L.zeros_off);
    p.status = reinterpret_cast<uint32_t *>(w8);
    p.flags = reinterpret_cast<uint32_t *>(w8 + kGemmFlagsOff);
    p.flags2 = reinterpret_cast<uint32_t *>(w8 + kGemmFlags2Off);
    p.partial = reinterpret_cast<float *>(w8 + kGemmPartialOff);
    p.M = M; p.K = K; p.N = N; p.bits = bits; p.group = group;
    p.tiles_m = g.tiles_m;
    p.tiles_n = g.tiles_n;
    p.span_tiles = g.span_tiles;
    p.split_s = g.split_s;
    p.col_fastest = g.col_fastest;
    p.stamps = reinterpret_cast<long long *>(w8 + kGemmPartialOff + (size_t)kMaxGemmCtas * kPartialBytesPerCta);
    // the fp16 weights [N][K]: boxes of one k-block x a CTA's channels, 128-byte swizzle (the layout the
    // dequantization writes); unused maps are copies of the activation map
    CUtensorMap tmap_wf = tmap_x;
    if (variant == kGemmLoadFull) {
        const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
        const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)bn_cta};
        if (enc(&tmap_wf, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(wt_f16), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TMAN_ERR_CUDA;
    }
    if (bits == 2) return launch_bits<2, kGemmProduct>(tmap_x, tmap_w, tmap_y, tmap_wf, p, g, s);
    if (bits == 3) return launch_bits<3, kGemmProduct>(tmap_x, tmap_w, tmap_y, tmap_wf, p, g, s);
    if (variant == kGemmConvertDq) return launch_bits<4, kGemmConvertDq>(tmap_x, tmap_w, tmap_y, tmap_wf, p, g, s);
    if (variant == kGemmLoadFull) return launch_bits<4, kGemmLoadFull>(tmap_x, tmap_w, tmap_y, tmap_wf, p, g, s);
    if (variant == kGemmSequential) return launch_bits<4, kGemmSequential>(tmap_x, tmap_w, tmap_y, tmap_wf, p, g, s);
    return launch_bits<4, kGemmProduct>(tmap_x, tmap_w, tmap_y, tmap_wf, p, g, s);
}

}  // namespace tman
