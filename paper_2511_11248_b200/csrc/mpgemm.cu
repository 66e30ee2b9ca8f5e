// Prefill path: two-level lookup dequantization fused into a tcgen05 GEMM
// (paper Sec. 4.1 "Unified Layout through Fused LUT-based Dequantization", Fig. 7;
//  Sec. 4.2 "Pipelining to Hide Dequantization Overhead", Fig. 9).
//
// A CTA computes tiles of 128*MH tokens x up to 128 output channels, one after the other (one CTA per
// SM, each with an equal share of the output).  Four kinds of agents run concurrently on a ring of
// shared-memory stages guarded by mbarriers (the paper's DMA / vector-core / matrix-core stages):
//   * warp 0, one lane : TMA loads of the fp16 activation tile (128-byte swizzle) and of the packed
//                        bit-plane words of the weight tile (one box per plane);
//   * warps 2..17      : (two groups of eight that take turns, two k-blocks each) read the staged
//                        plane words of their column, rebuild the codes
//                        (level 1: bit-serial -> bit-parallel), look every code up in the
//                        per-(block, column) conversion table kept in registers and addressed
//                        with byte-permute instructions (level 2: scale and zero-point baked in),
//                        and write the fp16 weight tile in the K-major swizzled layout the
//                        tensor core reads;
//   * warp 1, one lane : tcgen05.mma (M128 N<=128 K16, fp16 x fp16 -> fp32 in tensor memory), one
//                        per row block; tcgen05.commit hands the stage back;
//   * warps 18..25     : epilogue of the previous tile (tcgen05.ld, round to fp16, store) while the
//                        next tile accumulates into the second set of tensor-memory columns.
// Every wait is bounded: when a bound is hit the kernel records TMAN_ERR_TIMEOUT, stops issuing
// work, and still reaches the common tear-down that frees tensor memory.
#include "common.cuh"

#include <cuda.h>

namespace tman {
namespace {

// A CTA multiplies MH row blocks of 128 tokens by one dequantized weight tile of up to BN columns: every
// weight is rebuilt once per 128*MH tokens (MH = 2 halves the dequantization work per flop).
// Two tile configurations.  WIDE: BN = 256, one MMA covers 256 output channels, so an activation tile
// is read from shared memory once per 256 channels (shared-memory bandwidth is what bounds this
// kernel); three stages of 72 KB fit and tensor memory holds one accumulator set.  Narrow: BN = 128,
// four stages and two accumulator sets (the epilogue of a sub-tile overlaps the next one); used when
// the output is so small that an SM's share is at most 128 columns wide.
constexpr int BM = 128, BK = 64;
template <int WIDE> struct Cfg {
    static constexpr int BN = WIDE ? 256 : 128;
    static constexpr int NSTAGE = WIDE ? 3 : 4;
    static constexpr int NACC = WIDE ? 1 : 2;       // accumulator sets in tensor memory (MH * BN columns each)
    static constexpr int B_STAGE_BYTES = BN * BK * 2;
    static constexpr int P_PLANE_BYTES = (BN / 4) * (BK / 32) * 16;   // one plane of a packed tile
};
constexpr int A_HALF_BYTES = BM * BK * 2;
constexpr int NUM_DEQ_WARPS = 16;               // each fills 16 columns of a weight tile
constexpr int NUM_EPI_WARPS = 8;                // two per quarter of the tensor-memory lanes (alternate 32-column chunks)
constexpr int GEMM_THREADS = 32 * (2 + NUM_DEQ_WARPS + NUM_EPI_WARPS);
template <int WIDE> constexpr int smem_bytes(int mh, int bits)
{
    return Cfg<WIDE>::NSTAGE * (mh * A_HALF_BYTES + Cfg<WIDE>::B_STAGE_BYTES + bits * Cfg<WIDE>::P_PLANE_BYTES) +
           1024 /*align*/ + 256 /*barriers*/;
}

struct GemmParams {
    const uint8_t  *packed;
    const uint32_t *planes;
    const __half   *scales;
    const uint16_t *zeros;
    __half         *y;
    uint32_t       *status;
    int M, K, N, bits, group;
    int tiles_m;
    int sms;
    int R;          // column ranges per row tile
    int wide;       // tile configuration
    int pair;       // CTA-pair kernel
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
// Bounded wait: gives up after about one second.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 1023u) == 1023u) {
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > 1000000000ull) return false;
        }
    }
}
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Arrive on a barrier of another CTA of the cluster.  Only the signal crosses CTAs: the data a
// CTA's tensor core reads is in that CTA's own shared memory, made visible by the writer's
// fence.proxy.async, so no cluster-scope release (a slow memory barrier) is needed here.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t ld_shared_cluster_u32(uint32_t cluster_addr)
{
    uint32_t v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
    return v;
}
__device__ __forceinline__ void tcgen05_alloc2(uint32_t dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tcgen05_relinquish2()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tcgen05_dealloc2(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// commit of the pair's MMAs, arriving on the barrier at the same address in both CTAs
__device__ __forceinline__ void tcgen05_commit2_both(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tcgen05_mma2_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tmap, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tmap, int x, int y, int z, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
// Tile store: shared memory (written by this warp, made visible with fence.proxy.async) -> global.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *tmap, uint32_t src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(src) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// the issuing thread's earlier tile stores have finished reading shared memory / have completed
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_alloc(uint32_t dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tcgen05_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tcgen05_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tcgen05_mma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tcgen05_ld_32x32b_x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tcgen05_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 fp16) and
// which is stored with the 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= (uint64_t)1 << 16;                              // leading byte offset (unused here)
    d |= (uint64_t)(1024 >> 4) << 32;                    // stride byte offset: 8 rows
    d |= (uint64_t)1 << 46;                              // descriptor version for this architecture
    d |= (uint64_t)2 << 61;                              // 128-byte swizzle
    return d;
}

// Byte permute with the full 4-bit selectors (bit 3 of a selector replicates the sign bit of the
// selected byte), which the __byte_perm intrinsic does not expose.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

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

// Work of a CTA.  The output is cut into row tiles of 128*MH tokens and, inside a row tile, into R
// column ranges of (almost) equal width, a multiple of 16 columns.  The tiles_m * R items are dealt
// to the CTAs round-robin; a CTA walks through an item in sub-tiles of at most BN columns, again of
// (almost) equal width.  Every role derives the same list from (blockIdx, gridDim).
struct SubTile { int tile_m, col0, bn; };

struct TileWalk {
    int item, nitems, stride, tiles_m, R, n16, max16, unit;
    int tm, lo, len, nsub, j;
    // unit: column granularity (16; 32 for CTA pairs, whose two CTAs each take half of a sub-tile)
    __device__ TileWalk(const GemmParams &p, int cta, int ncta, int bn_max, int unit_ = 16)
        : item(cta - ncta), nitems(p.tiles_m * p.R), stride(ncta), tiles_m(p.tiles_m), R(p.R),
          n16((p.N + unit_ - 1) / unit_),   // a last unit may reach past N: computed, never stored
          max16(bn_max / unit_), unit(unit_),
          tm(0), lo(0), len(0), nsub(0), j(0) {}
    __device__ bool next(SubTile &t)
    {
        if (j == nsub) {
            item += stride;
            if (item >= nitems) return false;
            tm = item % tiles_m;
            const int r = item / tiles_m;
            lo = (int)(((long long)n16 * r) / R);
            len = (int)(((long long)n16 * (r + 1)) / R) - lo;
            nsub = (len + max16 - 1) / max16;
            j = 0;
        }
        const int u0 = lo + (len * j) / nsub, u1 = lo + (len * (j + 1)) / nsub;
        t.tile_m = tm;
        t.col0 = u0 * unit;
        t.bn = (u1 - u0) * unit;
        ++j;
        return true;
    }
};

template <int BITS, int MH, int WIDE>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
mpgemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w, const GemmParams p)
{
    constexpr int BN = Cfg<WIDE>::BN, NSTAGE = Cfg<WIDE>::NSTAGE, NACC = Cfg<WIDE>::NACC;
    constexpr int B_STAGE_BYTES = Cfg<WIDE>::B_STAGE_BYTES, P_PLANE_BYTES = Cfg<WIDE>::P_PLANE_BYTES;
    constexpr int A_STAGE_BYTES = MH * A_HALF_BYTES;
    constexpr int ACC_COLS = MH * BN;                  // one fp32 accumulator of BN columns per row block
    constexpr int TMEM_COLS = NACC * ACC_COLS;
    constexpr int P_STAGE_BYTES = BITS * P_PLANE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    if (!header_matches(p.packed, p.K, p.N, p.bits, p.group)) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_BAD_PACKED);
        return;
    }
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *a_tiles = smem;
    uint8_t *b_tiles = smem + NSTAGE * A_STAGE_BYTES;
    uint8_t *p_tiles = smem + NSTAGE * (A_STAGE_BYTES + B_STAGE_BYTES);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + NSTAGE * (A_STAGE_BYTES + B_STAGE_BYTES + P_STAGE_BYTES));
    // bars[0..NSTAGE) loaded (TMA), [NSTAGE..2NSTAGE) full (dequantized), [2NSTAGE..3NSTAGE) empty,
    // then accumulator full[2], accumulator empty[2]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * NSTAGE + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = p.K / BK;

    const uint32_t loaded0 = smem_u32(bars), full0 = smem_u32(bars + NSTAGE), empty0 = smem_u32(bars + 2 * NSTAGE),
                   accf0 = smem_u32(bars + 3 * NSTAGE), acce0 = smem_u32(bars + 3 * NSTAGE + 2);

    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(loaded0 + 8 * s, 1);
            mbar_init(full0 + 8 * s, NUM_DEQ_WARPS);
            mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < NACC; ++b) {
            mbar_init(accf0 + 8 * b, 1);
            mbar_init(acce0 + 8 * b, NUM_EPI_WARPS);
        }
        fence_barrier_init();
    }
    if (warp == 1) {
        tcgen05_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tcgen05_relinquish();
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(tmem_slot);

    bool ok = true;
    TileWalk walk(p, (int)blockIdx.x, (int)gridDim.x, BN);
    SubTile t;
    if (warp == 0) {
        // ---- stage 1: activation tiles and packed weight tiles by TMA -------------------------
        if (lane == 0) {
            uint32_t it = 0;
            while (ok && walk.next(t)) {
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = (int)(it % NSTAGE);
                    const uint32_t ph = (it / NSTAGE) & 1u;
                    if (!mbar_wait(empty0 + 8 * s, ph ^ 1u)) { ok = false; break; }
                    mbar_expect_tx(loaded0 + 8 * s, A_STAGE_BYTES + P_STAGE_BYTES);
                    tma_load_2d(smem_u32(a_tiles + s * A_STAGE_BYTES), &tmap_x, kb * BK, t.tile_m * (BM * MH), loaded0 + 8 * s);
#pragma unroll
                    for (int i = 0; i < BITS; ++i)
                        tma_load_3d(smem_u32(p_tiles + s * P_STAGE_BYTES + i * P_PLANE_BYTES), &tmap_w, kb * (BK / 8), i,
                                    t.col0 / 4, loaded0 + 8 * s);
                }
            }
        }
    } else if (warp == 1) {
        // ---- stage 3: tensor-core MMA --------------------------------------------------------
        if (lane == 0) {
            uint32_t it = 0, ti = 0;
            while (ok && walk.next(t)) {
                const uint32_t buf = ti % NACC, aph = (ti / NACC) & 1u;
                if (!mbar_wait(acce0 + 8 * buf, aph ^ 1u)) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t idesc = (1u << 4) | ((uint32_t)(t.bn >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = (int)(it % NSTAGE);
                    const uint32_t ph = (it / NSTAGE) & 1u;
                    if (!mbar_wait(full0 + 8 * s, ph)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint64_t bdesc = make_kmajor_sw128_desc(smem_u32(b_tiles + s * B_STAGE_BYTES));
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j)
#pragma unroll
                        for (int h = 0; h < MH; ++h) {
                            const uint64_t adesc = make_kmajor_sw128_desc(smem_u32(a_tiles + s * A_STAGE_BYTES + h * A_HALF_BYTES));
                            tcgen05_mma_f16(tmem_base + buf * ACC_COLS + (uint32_t)(h * BN), adesc + 2 * j, bdesc + 2 * j, idesc,
                                            (kb > 0 || j > 0) ? 1u : 0u);
                        }
                    tcgen05_commit(empty0 + 8 * s);
                }
                if (ok) tcgen05_commit(accf0 + 8 * buf);
                ++ti;
            }
        }
    } else if (warp < 2 + NUM_DEQ_WARPS) {
        // ---- stage 2: two-level lookup dequantization ----------------------------------------
        // A warp owns 16 columns and both plane words of a k-block: lane = (strip of the warp, word,
        // column of the strip).  With this split the 32 lanes read 32 different banks of the staged
        // plane words and write eight different 16-byte bank groups per quarter-warp.
        // Sub-tiles of at most 128 columns need only half of the warps per k-block: the two halves
        // then take turns, two k-blocks each, so that all sixteen warps still share the work.
        const int wd16 = warp - 2;
        const int sl = lane >> 3, v = (lane >> 2) & 1, c = lane & 3;
        const int nblk = p.K / p.group;
        const int gshift = (p.group == 32) ? 5 : (p.group == 64) ? 6 : 7;
        auto block_of = [&](int kb) { return ((2 * kb + v) * 32) >> gshift; };

        uint32_t it0 = 0;                                  // pipeline position of the sub-tile's first k-block
        while (ok && walk.next(t)) {
            const int ngroups = (t.bn <= 128) ? 2 : 1;   // eight warps cover 128 columns
            const int wd = (ngroups == 2) ? (wd16 & (NUM_DEQ_WARPS / 2 - 1)) : wd16;
            const int grp = (ngroups == 2) ? wd16 / (NUM_DEQ_WARPS / 2) : 0;
            const int n_local = wd * 16 + sl * 4 + c;
            const uint32_t p_off = (uint32_t)(wd * 4 + sl) * 32u + (uint32_t)v * 16u + (uint32_t)c * 4u;
            const uint32_t row_off = (uint32_t)(n_local >> 3) * 1024u + (uint32_t)(n_local & 7) * 128u;
            const uint32_t xr = (uint32_t)(n_local & 7);
            const uint32_t p_base = smem_u32(p_tiles) + p_off, b_base = smem_u32(b_tiles) + row_off;
            // k-blocks this warp works on: all of them, or every other pair (num_kb is even)
            auto mine = [&](int kb) { return ngroups == 1 || ((kb >> 1) & 1) == grp; };
            auto next_mine = [&](int kb) { return (ngroups == 1 || !(kb & 1)) ? kb + 1 : kb + 3; };
            const int n = t.col0 + n_local;
            const bool valid = n_local < t.bn && n < p.N;   // columns past the sub-tile are not used by the MMA
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
            __half sv_next = __float2half(0.f);
            uint32_t zz_next = 0u;

            for (int kb = 0; kb < num_kb; ++kb) {
                const uint32_t it = it0 + (uint32_t)kb;
                const int s = (int)(it % NSTAGE);
                const uint32_t ph = (it / NSTAGE) & 1u;
                const bool work = valid && mine(kb);
                if (work) {
                    const int Bk = block_of(kb);
                    if (Bk != cur_B) {
                        if (next_B != Bk) fetch_sz(Bk, sv_next, zz_next);
                        cur_B = Bk;
                        T.build(sv_next, zz_next);
                    }
                    // scale and zero-point of the block after this one are fetched one k-block ahead
                    const int kn = next_mine(kb);
                    const int Bn = block_of(kn);
                    if (kn < num_kb && Bn != cur_B && Bn != next_B) {
                        next_B = Bn;
                        fetch_sz(Bn, sv_next, zz_next);
                    }
                }
                if (!mbar_wait(loaded0 + 8 * s, ph)) { ok = false; break; }
                if (work) {
                    uint32_t w[BITS];
                    const uint32_t pp = p_base + (uint32_t)s * P_STAGE_BYTES;
#pragma unroll
                    for (int i = 0; i < BITS; ++i)
                        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w[i]) : "r"(pp + i * P_PLANE_BYTES) : "memory");
                    uint32_t out[16];
                    dequant_word<BITS>(w, T, out);
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
                if (lane == 0) mbar_arrive(full0 + 8 * s);
            }
            it0 += (uint32_t)num_kb;
        }
    } else {
        // ---- epilogue: tensor memory -> fp16 -> global, one warp per quarter of the lanes --------
        const int quarter = warp & 3;                      // tensor-memory lanes this warp may read
        const int epart = (warp - 2 - NUM_DEQ_WARPS) >> 2; // which of the quarter's warps
        uint32_t ti = 0;
        while (ok && walk.next(t)) {
            const uint32_t buf = ti % NACC, aph = (ti / NACC) & 1u;
            if (!mbar_wait(accf0 + 8 * buf, aph)) { ok = false; break; }
            tcgen05_fence_after();
#pragma unroll 1
            for (int h = 0; h < MH; ++h) {
                const int m = t.tile_m * (BM * MH) + h * BM + quarter * 32 + lane;
#pragma unroll 1
                for (int col = 32 * epart; col < t.bn; col += 32 * (NUM_EPI_WARPS / 4)) {
                    uint32_t r[32];
                    tcgen05_ld_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * ACC_COLS + (uint32_t)(h * BN + col), r);
                    tcgen05_wait_ld();
                    if (m < p.M) {
                        __half *dst = p.y + (size_t)m * p.N + (size_t)t.col0 + col;
#pragma unroll
                        for (int g8 = 0; g8 < 4; ++g8) {
                            if (col + 8 * g8 < t.bn && t.col0 + col + 8 * g8 < p.N) {
                                uint32_t hv[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const __half2 hh = __floats2half2_rn(__uint_as_float(r[8 * g8 + 2 * e]),
                                                                         __uint_as_float(r[8 * g8 + 2 * e + 1]));
                                    hv[e] = *reinterpret_cast<const uint32_t *>(&hh);
                                }
                                *reinterpret_cast<uint4 *>(dst + 8 * g8) = make_uint4(hv[0], hv[1], hv[2], hv[3]);
                            }
                        }
                    }
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce0 + 8 * buf);
            ++ti;
        }
    }

    if (!ok) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_TIMEOUT);
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        tcgen05_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---- CTA-pair variant ------------------------------------------------------------------------
// Two CTAs of a cluster share one tile of 2*128*MH tokens x up to 256 output channels: each holds its
// own 128*MH token rows, dequantizes half of the tile's channels, and the pair multiplies with
// tcgen05.mma.cta_group::2 (M = 256), issued by the pair's first CTA.  Each SM then reads only half of
// the weight tile per MMA and dequantizes half as much per flop, which is what the single-CTA kernel
// is short of (shared-memory bandwidth, ALU pipe).  Barriers that both CTAs feed (weight tile ready,
// accumulator drained) live in the first CTA and are reached with cluster-scope arrives; the MMA's
// commits arrive in both CTAs.  No TMA multicast is used: each CTA loads its own tiles.
constexpr int PAIR_BN = 256;                     // channels of a pair tile (128 per CTA)
constexpr int PAIR_NSTAGE = 4;
constexpr int PAIR_B_STAGE_BYTES = (PAIR_BN / 2) * BK * 2;
constexpr int PAIR_P_PLANE_BYTES = (PAIR_BN / 8) * (BK / 32) * 16;
constexpr int PAIR_OUT_BYTES = 32 * 32 * 2;      // an epilogue warp's output staging: 32 tokens x 32 channels
constexpr int pair_smem_bytes(int mh, int bits)
{
    // stages, barriers (256 B), staging (1024-aligned as the stages are: bits * 1 KB keeps it so), slack to align
    return PAIR_NSTAGE * (mh * A_HALF_BYTES + PAIR_B_STAGE_BYTES + bits * PAIR_P_PLANE_BYTES) + 1024
           + NUM_EPI_WARPS * PAIR_OUT_BYTES + 256;
}

template <int BITS, int MH>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
mpgemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                   const __grid_constant__ CUtensorMap tmap_y, const GemmParams p)
{
    constexpr int NSTAGE = PAIR_NSTAGE, B_STAGE_BYTES = PAIR_B_STAGE_BYTES, P_PLANE_BYTES = PAIR_P_PLANE_BYTES;
    constexpr int A_STAGE_BYTES = MH * A_HALF_BYTES;
    constexpr int P_STAGE_BYTES = BITS * P_PLANE_BYTES;
    constexpr int TMEM_COLS = MH * PAIR_BN;            // MH accumulators of 256 columns (512 for MH = 2)
    extern __shared__ uint8_t smem_raw[];
    const uint32_t rank = cluster_ctarank();           // 0: issues the MMAs and owns the shared barriers
    const bool hdr_ok = header_matches(p.packed, p.K, p.N, p.bits, p.group);   // same answer in every CTA
    if (!hdr_ok) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_BAD_PACKED);
        return;
    }
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *a_tiles = smem;
    uint8_t *b_tiles = smem + NSTAGE * A_STAGE_BYTES;
    uint8_t *p_tiles = smem + NSTAGE * (A_STAGE_BYTES + B_STAGE_BYTES);
    uint8_t *out_tiles = smem + NSTAGE * (A_STAGE_BYTES + B_STAGE_BYTES + P_STAGE_BYTES);
    uint64_t *bars = reinterpret_cast<uint64_t *>(out_tiles + NUM_EPI_WARPS * PAIR_OUT_BYTES);
    // bars[0..NSTAGE) loaded (own TMA), [NSTAGE..2NSTAGE) full (both CTAs' dequantization warps; used in
    // CTA 0), [2NSTAGE..3NSTAGE) empty (MMA commit, both CTAs), then accumulator full (commit, both CTAs)
    // and accumulator empty (both CTAs' epilogue warps; used in CTA 0)
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * NSTAGE + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = p.K / BK;
    const uint32_t loaded0 = smem_u32(bars), full0 = smem_u32(bars + NSTAGE), empty0 = smem_u32(bars + 2 * NSTAGE),
                   accf = smem_u32(bars + 3 * NSTAGE), acce = smem_u32(bars + 3 * NSTAGE + 1);

    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(loaded0 + 8 * s, 1);
            mbar_init(full0 + 8 * s, 2 * NUM_DEQ_WARPS);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accf, 1);
        mbar_init(acce, 2 * NUM_EPI_WARPS);
        *tmem_slot = 0xFFFFFFFFu;
        fence_barrier_init();
    }
    __syncthreads();
    if (warp == 1) {
        tcgen05_alloc2(smem_u32(tmem_slot), TMEM_COLS);
        tcgen05_relinquish2();
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();                                // both CTAs' barriers and tensor memory are set up
    tcgen05_fence_after();
    uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(tmem_slot);
    if (tmem_base == 0xFFFFFFFFu) tmem_base = ld_shared_cluster_u32(mapa_u32(smem_u32(tmem_slot), rank ^ 1u));

    bool ok = tmem_base != 0xFFFFFFFFu;
    // the pair walks through its items together; a CTA's rows and channels inside a sub-tile:
    TileWalk walk(p, (int)(blockIdx.x >> 1), (int)(gridDim.x >> 1), PAIR_BN, 32);
    SubTile t;
    const uint32_t full_lead = mapa_u32(full0, 0), acce_lead = mapa_u32(acce, 0);
    if (warp == 0) {
        // ---- stage 1: this CTA's activation rows and packed channels by TMA ---------------------
        if (lane == 0) {
            uint32_t it = 0;
            while (ok && walk.next(t)) {
                const int row0 = t.tile_m * (2 * BM * MH) + (int)rank * (BM * MH);
                const int strip0 = (t.col0 + (int)rank * (t.bn / 2)) / 4;
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = (int)(it % NSTAGE);
                    const uint32_t ph = (it / NSTAGE) & 1u;
                    if (!mbar_wait(empty0 + 8 * s, ph ^ 1u)) { ok = false; break; }
                    mbar_expect_tx(loaded0 + 8 * s, A_STAGE_BYTES + P_STAGE_BYTES);
                    tma_load_2d(smem_u32(a_tiles + s * A_STAGE_BYTES), &tmap_x, kb * BK, row0, loaded0 + 8 * s);
#pragma unroll
                    for (int i = 0; i < BITS; ++i)
                        tma_load_3d(smem_u32(p_tiles + s * P_STAGE_BYTES + i * P_PLANE_BYTES), &tmap_w, kb * (BK / 8), i,
                                    strip0, loaded0 + 8 * s);
                }
            }
        }
    } else if (warp == 1) {
        // ---- stage 3: the pair's MMAs, issued by CTA 0 ------------------------------------------
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, ti = 0;
            while (ok && walk.next(t)) {
                if (!mbar_wait(acce, (ti & 1u) ^ 1u)) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t idesc = (1u << 4) | ((uint32_t)(t.bn >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = (int)(it % NSTAGE);
                    const uint32_t ph = (it / NSTAGE) & 1u;
                    if (!mbar_wait(full0 + 8 * s, ph)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint64_t bdesc = make_kmajor_sw128_desc(smem_u32(b_tiles + s * B_STAGE_BYTES));
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j)
#pragma unroll
                        for (int h = 0; h < MH; ++h) {
                            const uint64_t adesc = make_kmajor_sw128_desc(smem_u32(a_tiles + s * A_STAGE_BYTES + h * A_HALF_BYTES));
                            tcgen05_mma2_f16(tmem_base + (uint32_t)(h * PAIR_BN), adesc + 2 * j, bdesc + 2 * j, idesc,
                                             (kb > 0 || j > 0) ? 1u : 0u);
                        }
                    tcgen05_commit2_both(empty0 + 8 * s);
                }
                if (ok) tcgen05_commit2_both(accf);
                ++ti;
            }
        }
    } else if (warp < 2 + NUM_DEQ_WARPS) {
        // ---- stage 2: two-level lookup dequantization of this CTA's half of the channels --------
        // at most 128 channels per CTA: the two halves of the sixteen warps take turns, two k-blocks each
        const int wd16 = warp - 2;
        const int wd = wd16 & (NUM_DEQ_WARPS / 2 - 1), grp = wd16 / (NUM_DEQ_WARPS / 2);
        const int sl = lane >> 3, v = (lane >> 2) & 1, c = lane & 3;
        const int nblk = p.K / p.group;
        const int gshift = (p.group == 32) ? 5 : (p.group == 64) ? 6 : 7;
        auto block_of = [&](int kb) { return ((2 * kb + v) * 32) >> gshift; };
        const int n_local = wd * 16 + sl * 4 + c;
        const uint32_t p_off = (uint32_t)(wd * 4 + sl) * 32u + (uint32_t)v * 16u + (uint32_t)c * 4u;
        const uint32_t row_off = (uint32_t)(n_local >> 3) * 1024u + (uint32_t)(n_local & 7) * 128u;
        const uint32_t xr = (uint32_t)(n_local & 7);
        const uint32_t p_base = smem_u32(p_tiles) + p_off, b_base = smem_u32(b_tiles) + row_off;
        auto mine = [&](int kb) { return ((kb >> 1) & 1) == grp; };
        auto next_mine = [&](int kb) { return !(kb & 1) ? kb + 1 : kb + 3; };

        uint32_t it0 = 0;
        while (ok && walk.next(t)) {
            const int half = t.bn / 2;
            const int n = t.col0 + (int)rank * half + n_local;
            const bool valid = n_local < half && n < p.N;
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
            __half sv_next = __float2half(0.f);
            uint32_t zz_next = 0u;
            for (int kb = 0; kb < num_kb; ++kb) {
                const uint32_t it = it0 + (uint32_t)kb;
                const int s = (int)(it % NSTAGE);
                const uint32_t ph = (it / NSTAGE) & 1u;
                const bool work = valid && mine(kb);
                if (work) {
                    const int Bk = block_of(kb);
                    if (Bk != cur_B) {
                        if (next_B != Bk) fetch_sz(Bk, sv_next, zz_next);
                        cur_B = Bk;
                        T.build(sv_next, zz_next);
                    }
                    const int kn = next_mine(kb);
                    const int Bn = block_of(kn);
                    if (kn < num_kb && Bn != cur_B && Bn != next_B) {
                        next_B = Bn;
                        fetch_sz(Bn, sv_next, zz_next);
                    }
                }
                if (!mbar_wait(loaded0 + 8 * s, ph)) { ok = false; break; }
                if (work) {
                    uint32_t w[BITS];
                    const uint32_t pp = p_base + (uint32_t)s * P_STAGE_BYTES;
#pragma unroll
                    for (int i = 0; i < BITS; ++i)
                        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w[i]) : "r"(pp + i * P_PLANE_BYTES) : "memory");
                    uint32_t out[16];
                    dequant_word<BITS>(w, T, out);
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
                if (lane == 0) mbar_arrive_cluster(full_lead + 8 * s);
            }
            it0 += (uint32_t)num_kb;
        }
    } else {
        // ---- epilogue: this CTA's rows, tensor memory -> fp16 -> shared memory -> global (tile stores) --
        // A warp reads 32 tokens x 32 channels (one token per lane), writes them as 64-byte rows into its
        // staging tile in the 64-byte swizzle (16-byte chunk index ^ bits 1..2 of the row: no bank
        // conflicts) and one lane stores the tile; tokens >= M and channels >= N are clipped by the store.
        const int quarter = warp & 3;
        const int ew = warp - 2 - NUM_DEQ_WARPS, epart = ew >> 2;
        const uint32_t stage = smem_u32(out_tiles + ew * PAIR_OUT_BYTES);
        const uint32_t my_row = stage + (uint32_t)lane * 64u, xr = ((uint32_t)lane >> 1) & 3u;
        uint32_t ti = 0;
        while (ok && walk.next(t)) {
            if (!mbar_wait(accf, ti & 1u)) { ok = false; break; }
            tcgen05_fence_after();
            bool released = false;
#pragma unroll 1
            for (int h = 0; h < MH; ++h) {
                const int m0 = t.tile_m * (2 * BM * MH) + (int)rank * (BM * MH) + h * BM + quarter * 32;
#pragma unroll 1
                for (int col = 32 * epart; col < t.bn; col += 32 * (NUM_EPI_WARPS / 4)) {
                    const bool last = (h == MH - 1) && (col + 32 * (NUM_EPI_WARPS / 4) >= t.bn);
                    uint32_t r[32];
                    if (m0 < p.M) {
                        tcgen05_ld_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(h * PAIR_BN + col), r);
                        tcgen05_wait_ld();
                    }
                    if (last) {                        // the accumulators are read: the next tile's MMAs may start
                        tcgen05_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(acce_lead);
                        released = true;
                    }
                    if (m0 < p.M) {
                        uint32_t hv[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const __half2 hh = __floats2half2_rn(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1]));
                            hv[e] = *reinterpret_cast<const uint32_t *>(&hh);
                        }
                        if (lane == 0) tma_store_wait_read();      // the staging tile is free again
                        __syncwarp();
#pragma unroll
                        for (uint32_t cj = 0; cj < 4; ++cj)
                            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(my_row + ((cj ^ xr) << 4)), "r"(hv[4 * cj]),
                                         "r"(hv[4 * cj + 1]), "r"(hv[4 * cj + 2]), "r"(hv[4 * cj + 3]) : "memory");
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) tma_store_2d(&tmap_y, stage, t.col0 + col, m0);
                    }
                }
            }
            if (!released) {                           // a warp without a chunk in this sub-tile
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(acce_lead);
            }
            ++ti;
        }
        if (lane == 0) tma_store_wait_all();
    }

    if (!ok) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_TIMEOUT);
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();                                // nobody touches the peer's memory after this
    if (warp == 1 && tmem_base != 0xFFFFFFFFu) {
        tcgen05_fence_after();
        tcgen05_dealloc2(tmem_base, TMEM_COLS);
    }
}

// ---- host side ---------------------------------------------------------------------------
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

template <int BITS, int MH, int WIDE>
tman_status launch_tile(const CUtensorMap &tmap_x, const CUtensorMap &tmap_w, const GemmParams &p, cudaStream_t s)
{
    auto kern = mpgemm_kernel<BITS, MH, WIDE>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<WIDE>(MH, BITS)) != cudaSuccess)
        return TMAN_ERR_CUDA;
    // one CTA per SM (fewer when there are fewer items than that): every CTA walks through its items
    long long grid = p.sms;
    if (grid > (long long)p.tiles_m * p.R) grid = (long long)p.tiles_m * p.R;
    kern<<<(unsigned)grid, GEMM_THREADS, smem_bytes<WIDE>(MH, BITS), s>>>(tmap_x, tmap_w, p);
    return launch_status();
}

template <int BITS, int MH>
tman_status launch_pair_tile(const CUtensorMap &tmap_x, const CUtensorMap &tmap_w, const CUtensorMap &tmap_y,
                             const GemmParams &p, cudaStream_t s)
{
    auto kern = mpgemm_pair_kernel<BITS, MH>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, pair_smem_bytes(MH, BITS)) != cudaSuccess)
        return TMAN_ERR_CUDA;
    long long pairs = p.sms / 2;
    if (pairs > (long long)p.tiles_m * p.R) pairs = (long long)p.tiles_m * p.R;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(GEMM_THREADS);
    cfg.dynamicSmemBytes = pair_smem_bytes(MH, BITS);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, tmap_x, tmap_w, tmap_y, p) != cudaSuccess) return TMAN_ERR_CUDA;
    return TMAN_OK;
}

template <int BITS>
tman_status launch_bits(const CUtensorMap &tmap_x, const CUtensorMap &tmap_w, const CUtensorMap &tmap_y,
                        const GemmParams &p, int mh, cudaStream_t s)
{
    if (p.pair) return launch_pair_tile<BITS, 2>(tmap_x, tmap_w, tmap_y, p, s);   // pairs run on more than 256 tokens
    if (p.wide) return mh == 2 ? launch_tile<BITS, 2, 1>(tmap_x, tmap_w, p, s) : launch_tile<BITS, 1, 1>(tmap_x, tmap_w, p, s);
    return mh == 2 ? launch_tile<BITS, 2, 0>(tmap_x, tmap_w, p, s) : launch_tile<BITS, 1, 0>(tmap_x, tmap_w, p, s);
}

}  // namespace

size_t mpgemm_workspace_bytes(int, int, int) { return kWsStatusBytes; }

tman_status launch_mpgemm(const void *packed, const void *x, void *y, int M, int K, int N, int bits,
                          int group, void *ws, size_t, cudaStream_t s)
{
    if ((reinterpret_cast<uintptr_t>(x) & 15) != 0 || (reinterpret_cast<uintptr_t>(y) & 15) != 0) return TMAN_ERR_SHAPE;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return TMAN_ERR_CUDA;
    CUtensorMap tmap;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    // CTA pairs (each CTA 256 token rows of a 512-row tile, half of the tile's channels) when there
    // are enough tokens and a pair of SMs gets a share of the output at least 192 channels wide;
    // otherwise single CTAs, which waste less on narrow shares.
    const int sms_q = sm_count();
    if (sms_q <= 0) return TMAN_ERR_CUDA;
    const long long share = (long long)N * ((M + 4 * BM - 1) / (4 * BM)) / (sms_q / 2 > 0 ? sms_q / 2 : 1);
    const bool pair = M > 2 * BM && share >= 192;
    const int mh = (M > BM) ? 2 : 1;                   // row blocks per CTA
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)(BM * mh)};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return TMAN_ERR_CUDA;

    Layout L = make_layout(K, N, bits, group);
    const uint8_t *pk = static_cast<const uint8_t *>(packed);
    GemmParams p;
    p.packed = pk;
    p.planes = reinterpret_cast<const uint32_t *>(pk + L.planes_off);
    p.scales = reinterpret_cast<const __half *>(pk + L.scales_off);
    p.zeros = reinterpret_cast<const uint16_t *>(pk + L.zeros_off);
    p.y = static_cast<__half *>(y);
    p.status = static_cast<uint32_t *>(ws);
    p.M = M; p.K = K; p.N = N; p.bits = bits; p.group = group;
    p.pair = pair ? 1 : 0;
    p.tiles_m = pair ? (M + 2 * BM * mh - 1) / (2 * BM * mh) : (M + BM * mh - 1) / (BM * mh);
    p.sms = sm_count();
    if (p.sms <= 0) return TMAN_ERR_CUDA;
    // Tile configuration and column ranges per row tile: the pair that minimises (waves of items over
    // the SMs) x (cost of an item).  A sub-tile of w 16-column units costs about w + 10 units of
    // shared-memory traffic per k-block (the activation tile is written once and read once per MMA
    // whatever the width), and a wide sub-tile holds twice as many units as a narrow one.
    if (pair) {
        // pairs: units of 32 columns, sub-tiles of up to 8 units, one item at a time per pair of SMs
        const int n32 = (N + 31) / 32, npairs = p.sms / 2;
        double best = 1e300;
        p.R = 1;
        p.wide = 0;
        for (int R = 1; R <= n32 && R <= 4096; ++R) {
            const long long items = (long long)p.tiles_m * R;
            const long long waves = (items + npairs - 1) / npairs;
            const int w = (n32 + R - 1) / R;
            const int nsub = (w + 7) / 8;
            const double cost = (double)waves * (w + 3.0 * nsub);
            if (cost < best - 1e-9) { best = cost; p.R = R; }
        }
    } else {
        const int n16 = (N + 15) / 16;
        double best = 1e300;
        p.R = 1;
        p.wide = 0;
        for (int wide = 0; wide < 2; ++wide) {
            const int maxw = (wide ? Cfg<1>::BN : Cfg<0>::BN) / 16;
            for (int R = 1; R <= n16 && R <= 4096; ++R) {
                const long long items = (long long)p.tiles_m * R;
                const long long waves = (items + p.sms - 1) / p.sms;
                const int w16 = (n16 + R - 1) / R;
                const int nsub = (w16 + maxw - 1) / maxw;
                const double cost = (double)waves * (w16 + 10.0 * nsub);
                if (cost < best - 1e-9) { best = cost; p.R = R; p.wide = wide; }
            }
        }
    }
    // the bit-plane words as a 3-D array of 32-bit elements: (word and column inside a strip's plane
    // row, plane, strip); one box = the two words of a k-block for the strips of a tile, one plane
    CUtensorMap tmap_w;
    {
        const cuuint64_t wt = (cuuint64_t)(K / 32);
        const cuuint64_t wdims[3] = {wt * 4, (cuuint64_t)bits, (cuuint64_t)(N / 4)};
        const cuuint64_t wstrides[2] = {wt * 16, wt * 16 * (cuuint64_t)bits};
        const cuuint32_t wbox[3] = {(cuuint32_t)(BK / 8), 1, (cuuint32_t)((pair ? PAIR_BN / 2 : (p.wide ? Cfg<1>::BN : Cfg<0>::BN)) / 4)};
        const cuuint32_t westr[3] = {1, 1, 1};
        if (enc(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint8_t *>(pk + L.planes_off), wdims, wstrides,
                wbox, westr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TMAN_ERR_CUDA;
    }
    // the output as 32 x 32 tiles in the 64-byte swizzle (the pair kernel's epilogue stores)
    CUtensorMap tmap_y;
    {
        const cuuint64_t ydims[2] = {(cuuint64_t)N, (cuuint64_t)M};
        const cuuint64_t ystrides[1] = {(cuuint64_t)N * 2};
        const cuuint32_t ybox[2] = {32, 32};
        if (enc(&tmap_y, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, y, ydims, ystrides, ybox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TMAN_ERR_CUDA;
    }
    if (bits == 2) return launch_bits<2>(tmap, tmap_w, tmap_y, p, mh, s);
    if (bits == 3) return launch_bits<3>(tmap, tmap_w, tmap_y, p, mh, s);
    return launch_bits<4>(tmap, tmap_w, tmap_y, p, mh, s);
}

}  // namespace tman
