// Decode path: bit-serial table-lookup mpGEMV (paper Sec. 2.2 "Bit-serial table lookup", Fig. 2;
// Sec. 4.3 "Mapping of LUT-based Decoding"; Sec. 4.1 Eq. 1-4 for the choice of the cut).
//
// Work split.  A cluster of C CTAs (one CTA per SM) owns a range of output columns; inside the
// cluster the reduction dimension is cut into C K-slices, one per CTA.  A CTA builds the
// activation tables of its slice in shared memory once (in several passes if the slice is
// longer than the table area) and reuses them for every column of the cluster's range -- the
// paper's "maximise reuse of cached lookup tables".  The K-slices are summed through distributed
// shared memory: every CTA pushes its partial sums into the shared memory of the CTA that owns
// the column, one cluster barrier, the owner adds them in rank order and writes fp16.  No global
// scratch, no polling, same bits on every run.
//
// Tables.  One table per 8 activations (two of the paper's 4-bit indices fused into an 8-bit index:
// one lookup covers eight weights of one bit-plane), 256 entries, fp16, each entry carrying the
// MT activation rows of the call (MT = 1, 2, 4, 8; 2*MT bytes).  Tables are stored entry-major: the
// 256-byte row of entry p holds entry p of the tables of up to 32 plane words, so a lane that
// works on word w always reads the bank(s) of w, whatever its index is.  Lanes of a warp therefore
// work on different words at any instant (a rotation over the eight words of a lane's k-part) and
// any mix of indices is conflict-free.
//
// Tiles.  The packed bit-plane words reach shared memory through TMA (one 3-D box per tile: TS
// strips of four columns x all planes x TW consecutive words) in a ring of stages guarded by
// mbarriers; lane 0 of warp 0 keeps the ring topped up.  A tile is consumed by eight warps: unit u
// (two of the eight rotation steps) x column half h (two of a strip's four columns; lanes with an odd
// j = lane / 8 take the other half, which keeps the 8-byte reads of the staged words conflict-free).
// Lane (s, jk, js): strip js*8+s of the tile, words jk*8..jk*8+7.  Per step a lane reads its plane word
// of two columns (8 bytes per plane) and does one lookup per index byte: PRMT forms the address
// (index byte << 8 | word slot), LDS fetches the entry, one (mixed-precision) add or fused
// multiply-add shift-accumulates.  After a pair of words (inside one quantization block, or two
// blocks of 32) the zero-point times the activation sum is subtracted and the block scale applied
// in fp32 (paper Sec. 4.3: low precision inside the block, floating point across blocks).  The sums
// of an item (tile, unit, half) are reduced over the k-part lanes and parked in shared memory,
// where later passes add to them.
#include "common.cuh"

#include <cuda.h>
#include <mutex>

namespace tman {

namespace {

constexpr int kGemvWarps = 16;
constexpr int kGemvThreads = 32 * kGemvWarps;
constexpr int kGemvMaxGroup = 4;
constexpr int kGemvMaxCluster = 8;
constexpr int kGemvMaxStages = 28;
constexpr int kGemvMaxTilesPerCluster = 64;
constexpr int kGemvSmemLimit = 232448;                // 227 KB of dynamic shared memory per CTA
constexpr uint32_t kGemvSmemBase = 1024;              // shared-window address of the first dynamic byte
constexpr uint64_t kWaitNs = 1000000000ull;           // a bounded wait gives up after about a second

// Optional phase time stamps (globaltimer, one row of 16 per CTA and call), compiled in only with
// -DTMAN_STAMPS for profiling builds; results are unaffected.
#ifdef TMAN_STAMPS
__device__ unsigned long long *g_gemv_stamps;
#define TMAN_STAMP(i)                                                                                          \
    do {                                                                                                       \
        if (g_gemv_stamps && (threadIdx.x & 31) == 0) {                                                        \
            unsigned long long t_;                                                                             \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                            \
            if ((i) < 6) { if (threadIdx.x == 0) g_gemv_stamps[(size_t)blockIdx.x * 32 + (i)] = t_; }          \
            else atomicMax(&g_gemv_stamps[(size_t)blockIdx.x * 32 + (i)], t_);                                 \
        }                                                                                                      \
    } while (0)
#define TMAN_CLK_DECL long long clk_acc_[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}; long long clk_t_ = clock64()
#define TMAN_CLK(k) do { const long long n_ = clock64(); clk_acc_[k] += n_ - clk_t_; clk_t_ = n_; } while (0)
#define TMAN_CLK_OUT do { if (g_gemv_stamps && threadIdx.x == 96) for (int k_ = 0; k_ < 12; ++k_) g_gemv_stamps[(size_t)blockIdx.x * 32 + 16 + k_] = (unsigned long long)clk_acc_[k_]; } while (0)
#else
#define TMAN_STAMP(i) do { } while (0)
#define TMAN_CLK_DECL do { } while (0)
#define TMAN_CLK(k) do { } while (0)
#define TMAN_CLK_OUT do { } while (0)
#endif

// Compile-time shape of a variant: BITS planes, MT activation rows per table entry.
template <int BITS, int MT>
struct Cfg {
    static constexpr int EB = 2 * MT;                            // bytes of a table entry
    static constexpr int NJK = (MT <= 2) ? 4 : (MT == 4 ? 2 : 1);  // k-parts (8 words each) of a tile
    static constexpr int NJS = 4 / NJK;                          // strip groups (8 strips each) of a tile
    static constexpr int TW = 8 * NJK;                           // plane words of a tile along K
    static constexpr int TS = 8 * NJS;                           // strips of a tile
    static constexpr int TC = 4 * TS;                            // columns of a tile
    static constexpr int TILE_BYTES = TS * BITS * TW * 16;       // 4096 * BITS
    static constexpr int ROW_BYTES = TW * 4 * 256 * EB;          // tables of the TW words of one tile row: 64 KB (MT = 1) or 128 KB
    static constexpr int MAX_ROWS = (MT == 1) ? 2 : 1;           // tile rows whose tables are resident at once
    static constexpr int NV = 2 * MT;                            // sums of an item per lane: 2 columns x MT rows
    static constexpr int HALVINGS = (NJK == 4) ? 1 : 0;          // k-parts jk and jk ^ 2 hold the same columns and are added
    static constexpr int VPL = NV >> HALVINGS;                   // sums a lane still holds after that
    static constexpr int PARK_TILE_BYTES = 8 * 32 * VPL * 4;     // parked sums of a tile's eight items
};

// bit-plane words (3-D), scales (2-D, 32-bit pairs of fp16) and zero-points (2-D, 16-bit) of every matrix
struct TMaps { CUtensorMap m[kGemvMaxGroup]; CUtensorMap sc[kGemvMaxGroup]; CUtensorMap z[kGemvMaxGroup]; };

struct GemvParams {
    const uint8_t  *packed[kGemvMaxGroup];
    const uint32_t *scales[kGemvMaxGroup];   // fp16 pairs: entry (strip * nblk + block) * 2 + half
    const uint16_t *zeros[kGemvMaxGroup];    // four zero-point nibbles of a strip and block
    __half         *y[kGemvMaxGroup];
    int Ng[kGemvMaxGroup];                   // output columns of each matrix
    int tile0[kGemvMaxGroup + 1];            // first tile of each matrix in the concatenated tile space
    int count;                               // matrices in this launch
    const __half   *x;
    uint32_t       *status;
    int M, K, bits, group;
    int wshift;                 // log2(group / 32): plane words per quantization block
    int nblk;                   // K / group
    int words_total;            // K / 32
    int ntiles;                 // tiles over all matrices
    int tpc;                    // tiles per cluster
    int wpc;                    // plane words per CTA (K-slice), a multiple of 8
    int nkt;                    // tile rows of a K-slice
    int rpp;                    // tile rows per pass (tables resident at once)
    int npass;
    int stages;                 // ring depth
    int epc;                    // output elements (column x row) each CTA of a cluster finishes
    uint32_t ring_off, park_off, inbox_off, sums_off, bar_off;   // shared-memory layout (bytes from the dynamic base)
    int sz_tma;                 // 1: a tile's scales and zero-points are copied into its stage (needs nblk % 8 == 0)
    int nbt;                    // quantization blocks of a tile row
    int zw;                     // zero-point entries per strip in a stage (a copy starts at a multiple of 8 entries)
    int stage_bytes;            // bit-plane words, then scales, then zero-points
};

// ---- PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait on an mbarrier phase; also gives up as soon as another thread of the CTA has.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag)
{
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 255u) == 255u) {
            if (abort_flag && *abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitNs) return false;
        }
    }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tmap, int x, int y, int z, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tmap, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_id_x()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t cluster_addr, float v)
{
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}
__device__ __forceinline__ uint2 lds64(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}

// Transposing reduction over the lanes selected by MASK, 2*MASK, ..., below END: every stage
// halves the number of values a lane keeps (or, once one is left, plainly adds).
template <int N_, int MASK, int END>
struct LaneReduce {
    static __device__ __forceinline__ void run(float *vals, int lane)
    {
        if constexpr (MASK < END) {
            if constexpr (N_ >= 2) {
                constexpr int H = N_ / 2;
                const bool up = (lane & MASK) != 0;
#pragma unroll
                for (int j = 0; j < H; ++j) {
                    const float keep = up ? vals[j + H] : vals[j];
                    const float send = up ? vals[j] : vals[j + H];
                    vals[j] = keep + __shfl_xor_sync(0xffffffffu, send, MASK);
                }
                LaneReduce<H, MASK * 2, END>::run(vals, lane);
            } else {
                vals[0] += __shfl_xor_sync(0xffffffffu, vals[0], MASK);
                LaneReduce<1, MASK * 2, END>::run(vals, lane);
            }
        }
    }
};

// Byte offset, inside the table area of one tile row, added to (index byte << 8 | word slot) for the
// index byte c of a plane word.  MT = 1: two tables share a 32-bit bank word (64 KB per 32 words);
// otherwise the byte pairs (0,1) and (2,3) live in two 64 KB halves.
template <int MT>
__host__ __device__ constexpr uint32_t table_imm(int c)
{
    return (MT == 1) ? (uint32_t)((c >> 1) * 128 + (c & 1) * 2) : (uint32_t)((c >> 1) * 65536 + (c & 1) * 128);
}

template <int MT> struct Acc {
    float   a32[2];                        // MT = 1: fp32 sums of the two columns
    __half2 a16[2][MT > 1 ? MT / 2 : 1];   // MT > 1: fp16 sums, two rows per register
    __device__ __forceinline__ void clear()
    {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            a32[c] = 0.f;
#pragma unroll
            for (int q = 0; q < (MT > 1 ? MT / 2 : 1); ++q) a16[c][q] = __floats2half2_rn(0.f, 0.f);
        }
    }
};

// One lookup: the entry of index byte C of plane word w, shift-accumulated with weight 2^PLANE.
// `slot` holds the lane's word slot in byte 0, the tile row in byte 2 and the top byte of the CTA's shared
// window in byte 3; byte 1 is zero.
template <int MT, int C, int PLANE>
__device__ __forceinline__ void lookup(uint32_t w, uint32_t slot, Acc<MT> &acc, int col)
{
    const uint32_t off = __byte_perm(w, slot, 0x7604u | ((uint32_t)C << 4));
    constexpr uint32_t IMM = kGemvSmemBase + table_imm<MT>(C);
    if constexpr (MT == 1) {
        unsigned short t;
        asm volatile("ld.shared.u16 %0, [%1 + %2];" : "=h"(t) : "r"(off), "n"(IMM));
        if constexpr (PLANE == 0) {
            asm("add.f32.f16 %0, %1, %0;" : "+f"(acc.a32[col]) : "h"(t));
        } else {
            constexpr unsigned short kTwoPow = (unsigned short)(0x3C00 + 0x0400 * PLANE);   // 2^PLANE in fp16
            asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc.a32[col]) : "h"(t), "h"(kTwoPow));
        }
    } else {
        uint32_t t[MT / 2];
        if constexpr (MT == 2) {
            asm volatile("ld.shared.b32 %0, [%1 + %2];" : "=r"(t[0]) : "r"(off), "n"(IMM));
        } else if constexpr (MT == 4) {
            asm volatile("ld.shared.v2.b32 {%0, %1}, [%2 + %3];" : "=r"(t[0]), "=r"(t[1]) : "r"(off), "n"(IMM));
        } else {
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4 + %5];"
                         : "=r"(t[0]), "=r"(t[1]), "=r"(t[2]), "=r"(t[3]) : "r"(off), "n"(IMM));
        }
        const __half2 wgt = __float2half2_rn((float)(1 << PLANE));
#pragma unroll
        for (int r = 0; r < MT / 2; ++r) {
            const __half2 e = *reinterpret_cast<const __half2 *>(&t[r]);
            acc.a16[col][r] = (PLANE == 0) ? __hadd2(acc.a16[col][r], e) : __hfma2(e, wgt, acc.a16[col][r]);
        }
    }
}

template <int MT, int PLANE>
__device__ __forceinline__ void lookup_word2(const uint2 &q, uint32_t slot, Acc<MT> &acc)
{
#pragma unroll
    for (int col = 0; col < 2; ++col) {
        const uint32_t w = col ? q.y : q.x;
        lookup<MT, 0, PLANE>(w, slot, acc, col);
        lookup<MT, 1, PLANE>(w, slot, acc, col);
        lookup<MT, 2, PLANE>(w, slot, acc, col);
        lookup<MT, 3, PLANE>(w, slot, acc, col);
    }
}

// all planes of one plane word (two columns): waddr = the lane's 8 bytes of plane 0
template <int BITS, int MT>
__device__ __forceinline__ void lookup_planes(uint32_t waddr, uint32_t plane_stride, uint32_t slot, Acc<MT> &acc)
{
    uint2 q[BITS];
#pragma unroll
    for (int i = 0; i < BITS; ++i) q[i] = lds64(waddr + i * plane_stride);
    lookup_word2<MT, 0>(q[0], slot, acc);
    lookup_word2<MT, 1>(q[1], slot, acc);
    if constexpr (BITS >= 3) lookup_word2<MT, 2>(q[2], slot, acc);
    if constexpr (BITS >= 4) lookup_word2<MT, 3>(q[3], slot, acc);
}

// ---- the kernel --------------------------------------------------------------------------------
template <int BITS, int MT>
__global__ void __launch_bounds__(kGemvThreads, 1)
mpgemv_kernel(const __grid_constant__ TMaps maps, const __grid_constant__ GemvParams p)
{
    using C_ = Cfg<BITS, MT>;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank(), csize = cluster_nctarank();
    const int cluster = (int)cluster_id_x();

    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + p.bar_off);           // full[stages], empty[stages]
    volatile uint32_t *flags = reinterpret_cast<volatile uint32_t *>(bars + 2 * kGemvMaxStages);   // [0] stop, [1] bad header, [2] tiles issued
    // per tile of the cluster: where its scales and zero-points start, its matrix and first strip
    struct TileMeta { const uint32_t *sc; const uint16_t *z; int nleft, m, strip0, pad; };
    TileMeta *meta = reinterpret_cast<TileMeta *>(bars + 2 * kGemvMaxStages + 8);
    // index checks of the accesses whose targets are computed at run time: a violation is recorded in the
    // status word (0x100 + site) and the access is skipped
    auto in_range = [&](bool ok, uint32_t site) {
        if (!ok) atomicCAS(p.status, 0u, 0x100u + site);
        return ok;
    };
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8u * (uint32_t)p.stages;
    float *sums = reinterpret_cast<float *>(smem + p.sums_off);                // activation sums per word and row
    float *inbox = reinterpret_cast<float *>(smem + p.inbox_off);              // [source rank][epc]
    float *park = reinterpret_cast<float *>(smem + p.park_off);                // [item][lane][VPL]

    // Let the next kernel of the stream be scheduled early (programmatic dependent launch) and tell the
    // cluster that this CTA is running (its shared memory may be written by the peers from now on).
    TMAN_STAMP(0);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    cluster_arrive_relaxed();
    if (tid == 0) {
        for (int g = 0; g < p.count; ++g) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&maps.m[g])) : "memory");
            if (p.sz_tma) {
                asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&maps.sc[g])) : "memory");
                asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&maps.z[g])) : "memory");
            }
        }
        for (int i = 0; i < p.stages; ++i) {
            mbar_init(full0 + 8u * i, 1);
            mbar_init(empty0 + 8u * i, 8);
        }
        flags[0] = 0;
        flags[1] = 0;
        flags[2] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // the cut of this CTA
    const int tile_lo = cluster * p.tpc;
    const int ntl = max(0, min(p.tpc, p.ntiles - tile_lo));          // tiles of this cluster
    const int nitems = ntl * 8;
    const int cta_w0 = (int)rank * p.wpc;
    const int cta_w1 = min(cta_w0 + p.wpc, p.words_total);
    // In a cluster the 32-bit shared address of a CTA's own memory carries the CTA's rank in its top byte;
    // the offset inside the CTA's window is what the lookups' immediates were built for.
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t window = smem_base & 0xFF000000u;
    const bool base_ok = (smem_base & 0x00FFFFFFu) == kGemvSmemBase;
    if (tid < ntl) {
        const int T = tile_lo + tid;
        int m = 0;
#pragma unroll
        for (int t = 1; t < kGemvMaxGroup; ++t) m += (t < p.count && T >= p.tile0[t]) ? 1 : 0;
        const int strip0 = (T - p.tile0[m]) * C_::TS;
        TileMeta tm;
        tm.sc = p.scales[m] + (size_t)strip0 * p.nblk * 2;
        tm.z = p.zeros[m] + (size_t)strip0 * p.nblk;
        tm.nleft = (p.Ng[m] >> 2) - strip0;
        tm.m = m;
        tm.strip0 = strip0;
        tm.pad = 0;
        meta[tid] = tm;
    }
    __syncthreads();

    // Nothing of the caller's memory is read into the SM before this point: everything below may depend
    // on the previous kernel of the stream.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    TMAN_STAMP(1);

    // ---- the ring: tile number q is issued by lane 0 of warp q % 16, in the order the warps visit the tiles:
    // pass, pair of tiles (i), tile row (r), tile of the pair (g).  The issuing thread is held while the copy
    // engine's queue is full, so the duty rotates over the warps; the position of a tile in that order is found
    // with exact float divisions (tile numbers stay far below 2^21).
    const uint32_t total_tiles = (uint32_t)ntl * (uint32_t)p.nkt;
    const uint32_t per_pass = (uint32_t)(ntl * p.rpp);
    const float inv_per_pass = 1.0f / (float)(per_pass ? per_pass : 1u), inv_stages = 1.0f / (float)p.stages;
    const uint32_t ahead_tiles = (uint32_t)min(p.stages, 8);    // tiles kept in flight or in use
    uint32_t my_q = (uint32_t)warp;                         // next tile this warp issues
    bool issue_ok = base_ok;
    auto issue_tile = [&](uint32_t q) {                    // lane 0 only
        int pass_q = (int)(((float)q + 0.5f) * inv_per_pass);
        if (pass_q > p.npass - 1) pass_q = p.npass - 1;
        const uint32_t rem = q - (uint32_t)pass_q * per_pass;
        const int row0 = pass_q * p.rpp;
        const int rows_q = min(p.rpp, p.nkt - row0);
        const int iq = (int)(((float)rem + 0.5f) / (float)(2 * rows_q));
        const uint32_t rem2 = rem - (uint32_t)(iq * 2 * rows_q);
        const bool two = ntl - 2 * iq >= 2;
        const int rq = two ? (int)(rem2 >> 1) : (int)rem2, gq = two ? (int)(rem2 & 1u) : 0;
        const TileMeta tm = meta[2 * iq + gq];
        const uint32_t round = (uint32_t)(((float)q + 0.5f) * inv_stages), st = q - round * (uint32_t)p.stages;
        // Tiles are issued strictly in order (tile q after tile q - 1), whichever warp issues them: the
        // wait below is then never more than one phase behind its barrier (a parity wait two phases
        // behind would pass at once).
        bool ok = true;
        {
            uint64_t t0 = 0;
            for (uint32_t it = 0; flags[2] != q; ++it) {
                if ((it & 63u) == 63u) {
                    if (flags[0]) { ok = false; break; }
                    const uint64_t now = global_timer_ns();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > kWaitNs) { ok = false; break; }
                }
            }
        }
        if (ok && round > 0) ok = mbar_wait(empty0 + 8u * st, (round - 1) & 1u, flags);
        if (ok) ok = in_range(st < (uint32_t)p.stages && 2 * iq + gq < ntl && rq < rows_q && tm.m >= 0 && tm.m < p.count &&
                              p.ring_off + (st + 1) * (uint32_t)p.stage_bytes <= p.park_off, 1);
        if (!ok) {
            issue_ok = false;
            if (!flags[1] && !flags[0]) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_TIMEOUT);
            flags[0] = 1;
            return;
        }
        const uint32_t dst = smem_u32(smem + p.ring_off) + st * (uint32_t)p.stage_bytes;
        const int w_tile = cta_w0 + (row0 + rq) * C_::TW;                 // first plane word of the tile
        const uint32_t sc_bytes = (uint32_t)(C_::TS * p.nbt * 8), z_bytes = (uint32_t)(C_::TS * p.zw * 2);
        mbar_expect_tx(full0 + 8u * st, C_::TILE_BYTES + (p.sz_tma ? sc_bytes + z_bytes : 0u));
        tma_load_3d(dst, &maps.m[tm.m], w_tile * 4, 0, tm.strip0, full0 + 8u * st);
        if (p.sz_tma) {
            const int blk = w_tile >> p.wshift;                            // first block of the tile row
            tma_load_2d(dst + C_::TILE_BYTES, &maps.sc[tm.m], blk * 2, tm.strip0, full0 + 8u * st);
            tma_load_2d(dst + C_::TILE_BYTES + sc_bytes, &maps.z[tm.m], blk & ~7, tm.strip0, full0 + 8u * st);
        }
        __threadfence_block();
        flags[2] = q + 1;
    };
    // every warp: issue my next tile once it falls inside the window that starts at tile `first_in_use`
    auto issue_due = [&](uint32_t first_in_use, uint32_t ahead) {
        if (my_q < total_tiles && my_q < first_in_use + ahead && issue_ok) {
            if (lane == 0) issue_tile(my_q);
            my_q += kGemvWarps;
        }
    };
    TMAN_STAMP(2);

    if (warp == 1) {
        // header check (every CTA sees the same headers, so the whole grid takes the same branch)
        bool ok = true;
        for (int g = 0; g < p.count; ++g) {
            const uint32_t *h = reinterpret_cast<const uint32_t *>(p.packed[g]);
            uint32_t want = 4u;
            if (lane == 0) want = 0x4E414D54u;
            if (lane == 1) want = 0x30303242u;
            if (lane == 2) want = kVersion;
            if (lane == 3) want = (uint32_t)p.K;
            if (lane == 4) want = (uint32_t)p.Ng[g];
            if (lane == 5) want = (uint32_t)p.bits;
            if (lane == 6) want = (uint32_t)p.group;
            if (lane < 8) ok = ok && (__ldg(h + lane) == want);
        }
        ok = __all_sync(0xffffffffu, ok);
        if (lane == 0 && (!ok || !base_ok)) {
            flags[1] = 1;
            flags[0] = 1;
            if (blockIdx.x == 0) atomicCAS(p.status, 0u, (uint32_t)(ok ? TMAN_ERR_LAYOUT : TMAN_ERR_BAD_PACKED));
        }
    }

    const int s = lane & 7, j = lane >> 3;
    const int jk = j % C_::NJK, js = j / C_::NJK;
    const int grp = warp >> 3, u = (warp >> 1) & 3, h = warp & 1;
    const int hl = h ^ (j & 1);                     // column half of this lane: columns 2*hl, 2*hl + 1 of its strip
    // word slots of the two steps of this lane's unit inside its k-part, and of the pair they form
    const int pair_in_part = ((s >> 1) + u) & 3;
    const int wk0 = 2 * pair_in_part + (s & 1), wk1 = 2 * pair_in_part + ((s + 1) & 1);
    const bool second_first = (s & 1) != 0;         // this lane visits the pair's second word first
    const uint32_t ring = smem_u32(smem + p.ring_off);
    const uint32_t lane_off = (uint32_t)(js * 8 + s) * (uint32_t)(BITS * C_::TW * 16) + (uint32_t)hl * 8u;
    const bool per_word = p.wshift == 0;            // blocks of 32: one block per word

    uint32_t seq_base = 0;
    bool alive = true;
    for (int pass = 0; pass < p.npass; ++pass) {
        const int row0 = pass * p.rpp, rows = min(p.rpp, p.nkt - row0);
        if (pass > 0) __syncthreads();              // everyone is done with the previous pass's tables

        // Scales and zero-points: with the tile in its stage (see issue_tile), or, where the block count
        // rules that out, fetched by every lane one step ahead of their use.
        struct ScaleZero { uint32_t sc0, sc1, z0, z1; };
        auto fetch_sz = [&](int i, int r) {
            ScaleZero v = {0u, 0u, 0u, 0u};
            const int tl = 2 * i + grp;
            if (!p.sz_tma && tl < ntl && r < rows) {
                const TileMeta tm = meta[tl];
                const int nb = min(js * 8 + s, tm.nleft - 1);
                const uint32_t *psc = tm.sc + (size_t)nb * p.nblk * 2 + hl;
                const uint16_t *pz = tm.z + (size_t)nb * p.nblk;
                const int gw_pair = cta_w0 + (row0 + r) * C_::TW + jk * 8 + 2 * pair_in_part;
                const int b0 = min(gw_pair >> p.wshift, p.nblk - 1);
                v.sc0 = __ldg(psc + 2 * b0);
                v.z0 = __ldg(pz + b0);
                v.sc1 = v.sc0;
                v.z1 = v.z0;
                if (per_word) {
                    const int b1 = min((gw_pair + 1) >> p.wshift, p.nblk - 1);
                    v.sc1 = __ldg(psc + 2 * b1);
                    v.z1 = __ldg(pz + b1);
                }
            }
            return v;
        };
        ScaleZero ahead_sz = fetch_sz(0, 0);
        TMAN_CLK_DECL;

        // ---- phase A: tables of this pass (paper Sec. 2.2; one table per 8 activations, 256 entries,
        // entry = sum of the activations whose index bit is set; fp32 sums rounded once to fp16) -------
        // A thread fills 32 consecutive entries of a pair (MT = 1: the tables of index bytes 2*cb and
        // 2*cb+1; else two activation rows of the table of byte cb); the lanes of a warp write distinct
        // banks (word slot x row pair).  A warp has at most two such units per pass.  All small loads of
        // the pass (activations, scales, zero-points) are issued before the tile copies: requests leave
        // the SM in order, and a burst of tile copies would hold them back.
        constexpr int PAIRS = (MT == 1) ? 1 : MT / 2;
        constexpr int NCB = (MT == 1) ? 2 : 4;
        constexpr int NWU = NCB * 8;                              // warp-level work units of a tile row
        static_assert(32 / PAIRS == C_::TW, "a warp covers the words of a tile row");
        static_assert(NWU * C_::MAX_ROWS <= 2 * kGemvWarps, "two units per warp");
        const int ws = lane / PAIRS, mp = lane % PAIRS;
        uint2 raw[2][4];                 // per unit and ph: the activations of the pair's two tables / rows
#pragma unroll
        for (int v = 0; v < 2; ++v) {
            const int L = warp + kGemvWarps * v;
#pragma unroll
            for (int ph = 0; ph < 4; ++ph) raw[v][ph] = make_uint2(0u, 0u);
            if (L < rows * NWU) {
                const int r = L / NWU, wu = L % NWU, cb = wu >> 3;
                const int gw = cta_w0 + (row0 + r) * C_::TW + ws;
                if (gw < cta_w1) {
                    if constexpr (MT == 1) {
                        // activations 32*gw + 8*ph + 4*cb + {0, 1} belong to byte 2*cb, + {2, 3} to byte 2*cb + 1
#pragma unroll
                        for (int ph = 0; ph < 4; ++ph)
                            raw[v][ph] = __ldg(reinterpret_cast<const uint2 *>(p.x + (size_t)gw * 32 + 8 * ph + 4 * cb));
                    } else {
#pragma unroll
                        for (int ph = 0; ph < 4; ++ph) {
                            const size_t off = (size_t)gw * 32 + 8 * ph + 2 * cb;
                            if (2 * mp < p.M) raw[v][ph].x = __ldg(reinterpret_cast<const uint32_t *>(p.x + (size_t)(2 * mp) * p.K + off));
                            if (2 * mp + 1 < p.M) raw[v][ph].y = __ldg(reinterpret_cast<const uint32_t *>(p.x + (size_t)(2 * mp + 1) * p.K + off));
                        }
                    }
                }
            }
        }
        // activation sums of every word and row (for the zero-point term): one thread per (tile row, word, row)
        uint4 raws[4];
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) raws[c4] = make_uint4(0u, 0u, 0u, 0u);
        const bool sums_thread = tid < rows * C_::TW * MT;
        if (sums_thread) {
            const int wsr = tid / MT, m = tid % MT;                  // wsr = r * TW + word slot
            const int gw2 = cta_w0 + row0 * C_::TW + wsr;
            if (gw2 < cta_w1 && m < p.M) {
                const uint4 *px = reinterpret_cast<const uint4 *>(p.x + (size_t)m * p.K + (size_t)gw2 * 32);
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) raws[c4] = __ldg(px + c4);
            }
        }
        TMAN_CLK(8);
        // the first tiles are asked for while the activations are on their way (a short window: the issuing
        // thread is held while the copy engine's queue is full, and the tables wait for every warp)
        if (pass == 0) issue_due(0u, min(ahead_tiles, 4u));
        TMAN_CLK(9);
#pragma unroll
        for (int v = 0; v < 2; ++v) {
            const int L = warp + kGemvWarps * v;
            if (L >= rows * NWU) continue;
            const int r = L / NWU, wu = L % NWU, q = wu & 7, cb = wu >> 3;
            uint8_t *tab = smem + (size_t)r * C_::ROW_BYTES;
            // xa[t][ph][hi]: index bit 4*hi + ph of table/row t selects activation 32*gw + 8*ph + 2*c + hi
            float xa[2][4][2];
#pragma unroll
            for (int ph = 0; ph < 4; ++ph) {
                const float2 f0 = __half22float2(*reinterpret_cast<const __half2 *>(&raw[v][ph].x));
                const float2 f1 = __half22float2(*reinterpret_cast<const __half2 *>(&raw[v][ph].y));
                xa[0][ph][0] = f0.x; xa[0][ph][1] = f0.y;
                xa[1][ph][0] = f1.x; xa[1][ph][1] = f1.y;
            }
            // entry p = lo16[p & 15] (the hi = 0 activations) + hi16[p >> 4] (the hi = 1 activations)
            float lo[2][16], hi2[2][2];
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                lut16(xa[t][0][0], xa[t][1][0], xa[t][2][0], xa[t][3][0], lo[t]);
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int hn = 2 * q + hh;     // high nibble of the entries 32*q + 16*hh ..
                    float vv = 0.f;
                    if (hn & 1) vv += xa[t][0][1];
                    if (hn & 2) vv += xa[t][1][1];
                    if (hn & 4) vv += xa[t][2][1];
                    if (hn & 8) vv += xa[t][3][1];
                    hi2[t][hh] = vv;
                }
            }
            uint8_t *dst;
            if constexpr (MT == 1) dst = tab + (size_t)(32 * q) * 256 + cb * 128 + ws * 4;
            else dst = tab + table_imm<MT>(cb) + (size_t)(32 * q) * 256 + ws * C_::EB + mp * 4;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                const __half2 hv = __floats2half2_rn(lo[0][e & 15] + hi2[0][e >> 4], lo[1][e & 15] + hi2[1][e >> 4]);
                *reinterpret_cast<__half2 *>(dst + e * 256) = hv;
            }
        }
        if (sums_thread) {
            float sacc = 0.f;
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                const uint32_t wv[4] = {raws[c4].x, raws[c4].y, raws[c4].z, raws[c4].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&wv[e]));
                    sacc += f.x;
                    sacc += f.y;
                }
            }
            sums[tid] = sacc;              // index (r * TW + word slot) * MT + row
        }
        TMAN_CLK(10);
        __syncthreads();
        TMAN_CLK(11);
        TMAN_STAMP(3);
        if (flags[0]) alive = false;              // bad header, or a wait that ran out somewhere in the CTA

        // ---- phase B: lookups, shift-accumulate, scale and zero-point (paper Sec. 4.3) ---------------
        for (int i = 0; 2 * i < ntl && alive; ++i) {
            const int tl = 2 * i + grp;                    // tile of the cluster this warp works on
            const int cnt_i = min(2, ntl - 2 * i);         // tiles of this pair
            const bool have = tl < ntl;                    // uniform over the warp
            float yv[C_::NV];
#pragma unroll
            for (int e = 0; e < C_::NV; ++e) yv[e] = 0.f;
            for (int r = 0; r < rows; ++r) {
                const uint32_t seq_pair = seq_base + (uint32_t)((2 * i) * rows + r * cnt_i);
                issue_due(seq_pair, ahead_tiles);
                if (!have) continue;
                TMAN_CLK(0);
                const ScaleZero now_sz = ahead_sz;
                if (!p.sz_tma) ahead_sz = (r + 1 < rows) ? fetch_sz(i, r + 1) : fetch_sz(i + 1, 0);
                TMAN_CLK(1);
                const uint32_t seq = seq_pair + (uint32_t)grp;
                const uint32_t round = (uint32_t)(((float)seq + 0.5f) * inv_stages), st = seq - round * (uint32_t)p.stages;
                if (!mbar_wait(full0 + 8u * st, round & 1u, flags)) {
                    if (!flags[0]) {
                        flags[0] = 1;
                        atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_TIMEOUT);
                    }
                    alive = false;
                    break;
                }
                TMAN_CLK(2);
                if (i == 0 && r == 0 && pass == 0) TMAN_STAMP(8);          // latest first-tile arrival over the warps
                const uint32_t stage_addr = ring + st * (uint32_t)p.stage_bytes;
                const uint32_t tile_addr = stage_addr + lane_off;
                uint32_t sc0 = now_sz.sc0, sc1 = now_sz.sc1, z0 = now_sz.z0, z1 = now_sz.z1;
                if (p.sz_tma) {
                    // the tile's scales [strip][block] (8 bytes) and zero-points [strip][zw] (2 bytes) behind its words
                    const int w_tile = cta_w0 + (row0 + r) * C_::TW;
                    const int blk_tile = w_tile >> p.wshift;
                    const int b0 = (w_tile + jk * 8 + 2 * pair_in_part) >> p.wshift;
                    const uint32_t sc_a = stage_addr + C_::TILE_BYTES + (uint32_t)(((js * 8 + s) * p.nbt + (b0 - blk_tile)) * 8 + hl * 4);
                    const uint32_t z_a = stage_addr + C_::TILE_BYTES + (uint32_t)(C_::TS * p.nbt * 8) +
                                         (uint32_t)(((js * 8 + s) * p.zw + (b0 - (blk_tile & ~7))) * 2);
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(sc0) : "r"(sc_a));
                    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(z0) : "r"(z_a));
                    sc1 = sc0;
                    z1 = z0;
                    if (per_word) {
                        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(sc1) : "r"(sc_a + 8u));
                        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(z1) : "r"(z_a + 2u));
                    }
                }
                z0 >>= 8 * hl;
                z1 >>= 8 * hl;
                const float *srow = sums + (size_t)(r * C_::TW + jk * 8 + 2 * pair_in_part) * MT;
                float S0[MT], S1[MT];
#pragma unroll
                for (int m = 0; m < MT; ++m) { S0[m] = srow[(s & 1) * MT + m]; S1[m] = srow[((s + 1) & 1) * MT + m]; }

                Acc<MT> acc;
                // y += s * (A - z * S) for the two columns, S = the activation sum(s) the lookups covered
                auto apply = [&](uint32_t sc, uint32_t z, const float *S) {
                    const float2 scf = __half22float2(*reinterpret_cast<const __half2 *>(&sc));
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        const float zf = (float)((z >> (4 * c)) & 0xFu);
                        const float sf = c ? scf.y : scf.x;
                        if constexpr (MT == 1) {
                            yv[c] = fmaf(sf, fmaf(-zf, S[0], acc.a32[c]), yv[c]);
                        } else {
#pragma unroll
                            for (int q2 = 0; q2 < MT / 2; ++q2) {
                                const float2 a = __half22float2(acc.a16[c][q2]);
                                yv[c * MT + 2 * q2] = fmaf(sf, fmaf(-zf, S[2 * q2], a.x), yv[c * MT + 2 * q2]);
                                yv[c * MT + 2 * q2 + 1] = fmaf(sf, fmaf(-zf, S[2 * q2 + 1], a.y), yv[c * MT + 2 * q2 + 1]);
                            }
                        }
                    }
                };
                const uint32_t slot0 = (uint32_t)((jk * 8 + wk0) * (MT == 1 ? 4 : C_::EB)) | ((uint32_t)r << 16) | window;
                const uint32_t slot1 = (uint32_t)((jk * 8 + wk1) * (MT == 1 ? 4 : C_::EB)) | ((uint32_t)r << 16) | window;
                acc.clear();
                TMAN_CLK(3);
                lookup_planes<BITS, MT>(tile_addr + (uint32_t)(jk * 8 + wk0) * 16u, C_::TW * 16, slot0, acc);
                TMAN_CLK(4);
                if (MT > 1 || per_word) {
                    // fp16 sums are handed to fp32 after every word; blocks of 32 end here too
                    apply(second_first ? sc1 : sc0, second_first ? z1 : z0, S0);
                    acc.clear();
                }
                lookup_planes<BITS, MT>(tile_addr + (uint32_t)(jk * 8 + wk1) * 16u, C_::TW * 16, slot1, acc);
                if (MT > 1 || per_word) {
                    apply(second_first ? sc0 : sc1, second_first ? z0 : z1, S1);
                } else {
                    float Sp[MT];
#pragma unroll
                    for (int m = 0; m < MT; ++m) Sp[m] = S0[m] + S1[m];
                    apply(sc0, z0, Sp);
                }
                TMAN_CLK(5);
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8u * st);
                TMAN_CLK(6);
            }
            if (have && alive) {
                // add the k-parts that hold the same columns (jk and jk ^ 2), then park (later passes add)
                LaneReduce<C_::NV, 16, (C_::NJK == 4) ? 32 : 16>::run(yv, lane);
                float *dst = park + ((size_t)(tl * 8 + u * 2 + h) * 32 + lane) * C_::VPL;
#pragma unroll
                for (int e = 0; e < C_::VPL; ++e) dst[e] = (pass == 0) ? yv[e] : dst[e] + yv[e];
            }
        }
        seq_base += (uint32_t)(ntl * rows);
        TMAN_CLK(7);
        TMAN_CLK_OUT;
    }
    TMAN_STAMP(9);                                   // latest end of lookups over the warps
    if (warp == 0) TMAN_STAMP(10);
    if (warp == 15) TMAN_STAMP(11);
    if (lane == 0 && flags[0] && my_q >= (uint32_t)kGemvWarps) {
        // giving up: the copy this warp issued last must have landed before the CTA may leave
        const uint32_t q = my_q - (uint32_t)kGemvWarps;
        mbar_wait(full0 + 8u * (q % (uint32_t)p.stages), (q / (uint32_t)p.stages) & 1u, nullptr);
    }
    __syncthreads();

    // ---- combine the K-slices through distributed shared memory --------------------------------------
    TMAN_STAMP(4);
    cluster_wait_acquire();                     // every CTA of the cluster has started
    const bool bad = flags[0] != 0;
    const int ne = ntl * C_::TC * MT;           // output elements of the cluster: (tile, row, column)
    if (!bad) {
        const uint32_t inbox_addr = smem_u32(inbox);
        for (int e = tid; e < ne; e += kGemvThreads) {
            const int cc = e % C_::TC, m = (e / C_::TC) % MT, tl = e / (C_::TC * MT);
            const int st_ = cc >> 2, c = cc & 3, s_ = st_ & 7, js_ = st_ >> 3;
            const int H = c >> 1;                             // column half
            const int idx = (c & 1) * MT + m;                 // index among a lane's 2*MT sums
            // after the k-parts jk and jk ^ 2 were added (four k-parts only), lane bit 4 tells which half
            // of the sums a lane kept
            const int part = C_::HALVINGS ? idx / C_::VPL : 0, k = C_::HALVINGS ? idx % C_::VPL : idx;
            float v = 0.f;
#pragma unroll
            for (int par = 0; par < (C_::NJK >= 2 ? 2 : 1); ++par) {
                const int jj = js_ * C_::NJK + par + 2 * part;   // lanes of this strip that hold the column
                const int ln = s_ + 8 * jj;
                const int hsel = H ^ (jj & 1);                  // the warp half whose lane jj works on column half H
#pragma unroll
                for (int uu = 0; uu < 4; ++uu) v += park[((size_t)(tl * 8 + uu * 2 + hsel) * 32 + ln) * C_::VPL + k];
            }
            const int owner = e / p.epc, slot = e - owner * p.epc;
            if (in_range(owner >= 0 && owner < (int)csize && slot >= 0 && slot < p.epc &&
                         p.inbox_off + (uint32_t)(((int)csize * p.epc) * 4) <= p.sums_off, 2))
            st_cluster_f32(mapa_u32(inbox_addr + (uint32_t)(((int)rank * p.epc + slot) * 4), (uint32_t)owner), v);
        }
    }
    __syncwarp();
    cluster_arrive_release();
    cluster_wait_acquire();
    TMAN_STAMP(5);
    if (!bad) {
        const int e_lo = (int)rank * p.epc, e_hi = min(ne, e_lo + p.epc);
        for (int e = e_lo + tid; e < e_hi; e += kGemvThreads) {
            float v = 0.f;
            for (uint32_t src = 0; src < csize; ++src) v += inbox[(int)src * p.epc + (e - e_lo)];
            const int cc = e % C_::TC, m = (e / C_::TC) % MT, tl = e / (C_::TC * MT);
            const int T = tile_lo + tl;
            int g = 0;
#pragma unroll
            for (int t = 1; t < kGemvMaxGroup; ++t) g += (t < p.count && T >= p.tile0[t]) ? 1 : 0;
            const int n = (T - p.tile0[g]) * C_::TC + cc;
            if (n < p.Ng[g] && m < p.M) p.y[g][(size_t)m * p.Ng[g] + n] = __float2half_rn(v);
        }
    }
    TMAN_STAMP(12);
}

// ---- host side ---------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
    if (q != cudaDriverEntryPointSuccess) return nullptr;
    return reinterpret_cast<EncodeTiledFn>(fn);
}

inline int mt_of(int M) { return M <= 1 ? 1 : (M <= 2 ? 2 : (M <= 4 ? 4 : 8)); }
inline int mt_index(int mt) { return mt == 1 ? 0 : (mt == 2 ? 1 : (mt == 4 ? 2 : 3)); }

struct VariantInfo {
    int tw, ts, tc, tile_bytes, row_bytes, max_rows, park_tile_bytes;
};
template <int BITS, int MT> VariantInfo variant_info()
{
    using C_ = Cfg<BITS, MT>;
    return {C_::TW, C_::TS, C_::TC, C_::TILE_BYTES, C_::ROW_BYTES, C_::MAX_ROWS, C_::PARK_TILE_BYTES};
}
VariantInfo variant_of(int bits, int mt)
{
    switch (bits * 10 + mt_index(mt)) {
        case 20: return variant_info<2, 1>();
        case 21: return variant_info<2, 2>();
        case 22: return variant_info<2, 4>();
        case 23: return variant_info<2, 8>();
        case 30: return variant_info<3, 1>();
        case 31: return variant_info<3, 2>();
        case 32: return variant_info<3, 4>();
        case 33: return variant_info<3, 8>();
        case 40: return variant_info<4, 1>();
        case 41: return variant_info<4, 2>();
        case 42: return variant_info<4, 4>();
        default: return variant_info<4, 8>();
    }
}

template <int BITS, int MT>
int kernel_capacity(int cluster, int smem_bytes)
{
    auto kern = mpgemv_kernel<BITS, MT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemvSmemLimit) != cudaSuccess) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)cluster * 64);
    cfg.blockDim = dim3(kGemvThreads);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    return n;
}

// Clusters of `cluster` CTAs of the variant that the current device holds at once, looked up once per
// device (the kernel takes one CTA per SM whatever its shared-memory size, so the full size is asked).
std::mutex g_cap_lock;
int g_cap[64][3][4][kGemvMaxCluster + 1];      // [device][bits - 2][mt index][cluster size], 0 = not asked yet, -1 = none
int device_capacity(int bits, int mt, int cluster)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    std::lock_guard<std::mutex> guard(g_cap_lock);
    int &slot = g_cap[dev][bits - 2][mt_index(mt)][cluster];
    if (slot == 0) {
        int n = 0;
        switch (bits * 10 + mt_index(mt)) {
            case 20: n = kernel_capacity<2, 1>(cluster, kGemvSmemLimit); break;
            case 21: n = kernel_capacity<2, 2>(cluster, kGemvSmemLimit); break;
            case 22: n = kernel_capacity<2, 4>(cluster, kGemvSmemLimit); break;
            case 23: n = kernel_capacity<2, 8>(cluster, kGemvSmemLimit); break;
            case 30: n = kernel_capacity<3, 1>(cluster, kGemvSmemLimit); break;
            case 31: n = kernel_capacity<3, 2>(cluster, kGemvSmemLimit); break;
            case 32: n = kernel_capacity<3, 4>(cluster, kGemvSmemLimit); break;
            case 33: n = kernel_capacity<3, 8>(cluster, kGemvSmemLimit); break;
            case 40: n = kernel_capacity<4, 1>(cluster, kGemvSmemLimit); break;
            case 41: n = kernel_capacity<4, 2>(cluster, kGemvSmemLimit); break;
            case 42: n = kernel_capacity<4, 4>(cluster, kGemvSmemLimit); break;
            default: n = kernel_capacity<4, 8>(cluster, kGemvSmemLimit); break;
        }
        slot = n > 0 ? n : -1;
    }
    return slot > 0 ? slot : 0;
}

}  // namespace

// ---- the cut of a call (host): the counterpart of the paper's constraint search, Sec. 4.1 Eq. 1-4 ----
// Candidates: cluster size C (how many K-slices are summed on chip) x column tiles per cluster.
// Constraints (the paper's Eq. 4, "stage buffers fit on-chip memory", restated): the tables resident at
// once (tile rows of 64 KB or 128 KB), a ring of at least two tiles (three where the call has them), the
// parked sums of the cluster's tiles, the inbox and the activation sums must fit 227 KB of shared
// memory; only `capacity(C)` clusters run at once (more clusters than that run as further waves).
// Cost (clocks of one SM, busiest CTA): table builds (bytes / 128 per clock, per pass) + lookups
// (shared-memory wavefronts of the CTA's units over the measured pipe use) + the exchange, per wave.
// The paper's heuristics map onto it: the largest table slice that fits (its "maximise K_lut"), all
// columns of a cluster per table build ("maximise M_iter").
GemvPlan plan_gemv(int M, int K, const int *Ns, int count, int bits, int group, const int *capacity /* [9]: by cluster size */)
{
    GemvPlan best = {};
    best.cluster = 0;
    const int mt = mt_of(M);
    const VariantInfo v = variant_of(bits, mt);
    const int words = K / 32;
    int ntiles = 0;
    for (int g = 0; g < count; ++g) ntiles += (Ns[g] + v.tc - 1) / v.tc;
    double best_cost = 0.0;
    auto up256 = [](int b) { return (b + 255) / 256 * 256; };
    for (int C = 1; C <= kGemvMaxCluster; ++C) {
        if (capacity[C] <= 0) continue;
        int wpc = (words + C - 1) / C;
        wpc = (wpc + 7) / 8 * 8;
        if ((words + wpc - 1) / wpc != C) continue;          // the same cut as a smaller cluster
        const int nkt = (wpc + v.tw - 1) / v.tw;
        const int rpp = nkt < v.max_rows ? nkt : v.max_rows;
        const int npass = (nkt + rpp - 1) / rpp;
        const int tables = rpp * v.row_bytes;
        const int sums = up256(rpp * v.tw * mt * 4);
        const int fixed = tables + sums + 2 * kGemvMaxStages * 8 + 64 + kGemvMaxTilesPerCluster * 32;
        // a stage holds a tile's bit-plane words and, where the copy engine can address them (rows of the
        // zero-point array a multiple of 16 bytes apart), its scales and zero-points
        // (a zero-point copy starts at a multiple of 8 entries = 16 bytes, so its rows are up to 8 entries wider)
        const int nbt = (v.tw * 32) / group, zw = nbt >= 8 ? nbt + 8 : 8;
        const int sz_tma = ((K / group) % 8 == 0) ? 1 : 0;
        const int stage_bytes = (v.tile_bytes + (sz_tma ? v.ts * (nbt * 8 + zw * 2) : 0) + 127) / 128 * 128;
        // the most tiles per cluster whose parked sums and inbox still leave room for the ring
        int even = (ntiles + capacity[C] - 1) / capacity[C];
        if (even > kGemvMaxTilesPerCluster) even = kGemvMaxTilesPerCluster;
        for (int tpc = even; tpc >= 1; tpc = (tpc > even / 2 + 1) ? tpc - 1 : 0) {
            const int ncl = (ntiles + tpc - 1) / tpc;
            const int waves = (ncl + capacity[C] - 1) / capacity[C];
            const int epc = (tpc * v.tc * mt + C - 1) / C;
            const int park = up256(tpc * v.park_tile_bytes);
            const int inbox = up256(C * epc * 4);
            const int tiles_cta = tpc * nkt;                  // tiles a CTA streams
            int stages = (kGemvSmemLimit - fixed - park - inbox) / stage_bytes;
            if (stages > kGemvMaxStages) stages = kGemvMaxStages;
            if (stages > tiles_cta) stages = tiles_cta;
            if (stages < (tiles_cta < 2 ? tiles_cta : 2)) {
                if (tpc == 1) break;
                continue;
            }
            // cost of the busiest CTA, in SM clocks
            const double wf_lookup = mt <= 2 ? 1.0 : (mt == 4 ? 2.0 : 4.0);
            const double pipe_use = 25.0 / 32.0;              // measured: 25 lookups per clock of 32
            const double pairs = (tpc + 1) / 2;               // two tiles are worked on at a time
            const double unit_wf = 2.0 * bits * (2.0 + 8.0 * wf_lookup);     // one warp, one tile row
            const double lookups = pairs * kGemvWarps * nkt * unit_wf / pipe_use;
            const double stream = (double)tiles_cta * stage_bytes / 22.0;    // HBM share of an SM: ~22 bytes per clock
            const double build = (double)npass * (tables / 128.0 + 500.0);
            const double exchange = 700.0 + 90.0 * C;
            const double cost = waves * (build + (lookups > stream ? lookups : stream) + exchange + 1200.0);
            if (best.cluster == 0 || cost < best_cost) {
                best_cost = cost;
                best.mt = mt; best.cluster = C; best.wpc = wpc; best.nkt = nkt; best.rpp = rpp; best.npass = npass;
                best.ntiles = ntiles; best.tpc = tpc; best.clusters = ncl; best.waves = waves; best.stages = stages;
                best.epc = epc; best.tables_bytes = tables; best.park_bytes = park; best.inbox_bytes = inbox;
                best.sums_bytes = sums; best.sz_tma = sz_tma; best.nbt = nbt; best.zw = zw; best.stage_bytes = stage_bytes;
                best.smem_bytes = fixed + park + inbox + stages * stage_bytes;
                best.cost_clocks = (int)cost;
            }
            if (waves == 1) break;                            // fewer tiles per cluster only cost more from here
            if (tpc == 1) break;
        }
    }
    return best;
}

namespace {

template <int BITS, int MT>
tman_status launch_variant(const TMaps &maps, GemvParams &p, const GemvPlan &g, cudaStream_t s)
{
    using C_ = Cfg<BITS, MT>;
    auto kern = mpgemv_kernel<BITS, MT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemvSmemLimit) != cudaSuccess)
        return TMAN_ERR_CUDA;
    p.ring_off = (uint32_t)g.tables_bytes;
    p.park_off = p.ring_off + (uint32_t)(g.stages * g.stage_bytes);
    p.inbox_off = p.park_off + (uint32_t)g.park_bytes;
    p.sums_off = p.inbox_off + (uint32_t)g.inbox_bytes;
    p.bar_off = p.sums_off + (uint32_t)g.sums_bytes;
    p.sz_tma = g.sz_tma;
    p.nbt = g.nbt;
    p.zw = g.zw;
    p.stage_bytes = g.stage_bytes;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(g.clusters * g.cluster));
    cfg.blockDim = dim3(kGemvThreads);
    cfg.dynamicSmemBytes = (size_t)g.smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)g.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, kern, maps, p) != cudaSuccess) return TMAN_ERR_CUDA;
    return TMAN_OK;
}

tman_status capacities(int bits, int mt, int *cap /* [kGemvMaxCluster + 1] */)
{
    int dev = 0, reserved = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&reserved, cudaDevAttrReservedSharedMemoryPerBlock, dev) != cudaSuccess)
        return TMAN_ERR_CUDA;
    if ((uint32_t)reserved != kGemvSmemBase) return TMAN_ERR_UNSUPPORTED;
    cap[0] = 0;
    bool any = false;
    for (int C = 1; C <= kGemvMaxCluster; ++C) {
        cap[C] = device_capacity(bits, mt, C);
        any = any || cap[C] > 0;
    }
    return any ? TMAN_OK : TMAN_ERR_CUDA;
}

}  // namespace

tman_status mpgemv_plan(int M, int K, const int *Ns, int count, int bits, int group, const int *capacity9, GemvPlan *out)
{
    int cap[kGemvMaxCluster + 1];
    if (capacity9) {
        for (int c = 0; c <= kGemvMaxCluster; ++c) cap[c] = capacity9[c];
    } else {
        tman_status st = capacities(bits, mt_of(M), cap);
        if (st != TMAN_OK) return st;
    }
    *out = plan_gemv(M, K, Ns, count, bits, group, cap);
    return out->cluster > 0 ? TMAN_OK : TMAN_ERR_UNSUPPORTED;
}

__global__ void ws_fill_kernel(uint32_t *ws, size_t words)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < words) ws[i] = (i < kWsStatusBytes / 4) ? 0u : 0x7FA5A5A5u;
}

// status word (and its padding) zero, everything after it the "empty" pattern the prefill kernel's flags start from
tman_status launch_workspace_init(void *ws, size_t ws_bytes, cudaStream_t s)
{
    const size_t words = ws_bytes / 4;
    ws_fill_kernel<<<(unsigned)((words + 255) / 256), 256, 0, s>>>(static_cast<uint32_t *>(ws), words);
    return launch_status();
}

size_t mpgemv_workspace_bytes(int M, int K, int N)
{
    (void)M; (void)K; (void)N;
    return kWsStatusBytes;       // the K-slices are summed on chip: only the status word lives in the workspace
}

tman_status launch_mpgemv_grouped(int count, const void *const *packed, const void *x, void *const *y, int M, int K,
                                  const int *Ns, int bits, int group, void *ws, size_t ws_bytes, cudaStream_t s)
{
    (void)ws_bytes;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return TMAN_ERR_CUDA;
    GemvPlan g;
    tman_status st = mpgemv_plan(M, K, Ns, count, bits, group, nullptr, &g);
    if (st != TMAN_OK) return st;
    const VariantInfo v = variant_of(bits, g.mt);

    TMaps maps;
    GemvParams p;
    p.count = count;
    int tiles = 0;
    const cuuint32_t estr[3] = {1, 1, 1};
    for (int m = 0; m < kGemvMaxGroup; ++m) {
        const int mm = m < count ? m : 0;
        Layout L = make_layout(K, Ns[mm], bits, group);
        const uint8_t *pk = static_cast<const uint8_t *>(packed[mm]);
        p.packed[m] = pk;
        p.scales[m] = reinterpret_cast<const uint32_t *>(pk + L.scales_off);
        p.zeros[m] = reinterpret_cast<const uint16_t *>(pk + L.zeros_off);
        p.y[m] = static_cast<__half *>(y[mm]);
        p.Ng[m] = Ns[mm];
        p.tile0[m] = tiles;
        if (m < count) tiles += (Ns[m] + v.tc - 1) / v.tc;
        // the bit-plane words as a 3-D array of 32-bit elements: (word and column inside a strip's plane
        // row, plane, strip); one box = a tile: TW words x all planes x TS strips
        const cuuint64_t wt = (cuuint64_t)(K / 32);
        const cuuint64_t wdims[3] = {wt * 4, (cuuint64_t)bits, (cuuint64_t)(Ns[mm] / 4)};
        const cuuint64_t wstrides[2] = {wt * 16, wt * 16 * (cuuint64_t)bits};
        const cuuint32_t wbox[3] = {(cuuint32_t)(v.tw * 4), (cuuint32_t)bits, (cuuint32_t)v.ts};
        if (enc(&maps.m[m], CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint8_t *>(pk + L.planes_off), wdims, wstrides,
                wbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TMAN_ERR_CUDA;
        if (g.sz_tma) {
            // scales: (pairs of fp16 of a strip's blocks, strip); zero-points: (16-bit entry of a block, strip)
            const cuuint64_t nblk = (cuuint64_t)(K / group);
            const cuuint64_t sdims[2] = {nblk * 2, (cuuint64_t)(Ns[mm] / 4)};
            const cuuint64_t sstrides[1] = {nblk * 8};
            const cuuint32_t sbox[2] = {(cuuint32_t)(g.nbt * 2), (cuuint32_t)v.ts};
            if (enc(&maps.sc[m], CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint8_t *>(pk + L.scales_off), sdims, sstrides,
                    sbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return TMAN_ERR_CUDA;
            const cuuint64_t zdims[2] = {nblk, (cuuint64_t)(Ns[mm] / 4)};
            const cuuint64_t zstrides[1] = {nblk * 2};
            const cuuint32_t zbox[2] = {(cuuint32_t)g.zw, (cuuint32_t)v.ts};
            if (enc(&maps.z[m], CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<uint8_t *>(pk + L.zeros_off), zdims, zstrides,
                    zbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return TMAN_ERR_CUDA;
        } else {
            maps.sc[m] = maps.m[m];
            maps.z[m] = maps.m[m];
        }
    }
    p.tile0[kGemvMaxGroup] = tiles;
    for (int m = count; m < kGemvMaxGroup; ++m) p.tile0[m] = tiles;
    p.x = static_cast<const __half *>(x);
    p.status = static_cast<uint32_t *>(ws);
    p.M = M; p.K = K; p.bits = bits; p.group = group;
    p.wshift = (group == 32) ? 0 : (group == 64) ? 1 : 2;
    p.nblk = K / group;
    p.words_total = K / 32;
    p.ntiles = g.ntiles;
    p.tpc = g.tpc; p.wpc = g.wpc; p.nkt = g.nkt; p.rpp = g.rpp; p.npass = g.npass;
    p.stages = g.stages; p.epc = g.epc;
    p.ring_off = p.park_off = p.inbox_off = p.sums_off = p.bar_off = 0;
    p.sz_tma = p.nbt = p.zw = p.stage_bytes = 0;
    switch (bits * 10 + mt_index(g.mt)) {
        case 20: return launch_variant<2, 1>(maps, p, g, s);
        case 21: return launch_variant<2, 2>(maps, p, g, s);
        case 22: return launch_variant<2, 4>(maps, p, g, s);
        case 23: return launch_variant<2, 8>(maps, p, g, s);
        case 30: return launch_variant<3, 1>(maps, p, g, s);
        case 31: return launch_variant<3, 2>(maps, p, g, s);
        case 32: return launch_variant<3, 4>(maps, p, g, s);
        case 33: return launch_variant<3, 8>(maps, p, g, s);
        case 40: return launch_variant<4, 1>(maps, p, g, s);
        case 41: return launch_variant<4, 2>(maps, p, g, s);
        case 42: return launch_variant<4, 4>(maps, p, g, s);
        default: return launch_variant<4, 8>(maps, p, g, s);
    }
}

tman_status launch_mpgemv(const void *packed, const void *x, void *y, int M, int K, int N, int bits,
                          int group, void *ws, size_t ws_bytes, cudaStream_t s)
{
    return launch_mpgemv_grouped(1, &packed, x, &y, M, K, &N, bits, group, ws, ws_bytes, s);
}

#ifdef TMAN_STAMPS
extern "C" void tman_debug_set_stamps(void *p)
{
    unsigned long long *q = static_cast<unsigned long long *>(p);
    cudaMemcpyToSymbol(g_gemv_stamps, &q, sizeof(q));
}
#endif

}  // namespace tman
