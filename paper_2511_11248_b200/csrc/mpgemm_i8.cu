// Prefill of the integer path: per-tensor ternary weights dequantized to INT8 by two table lookups and
// multiplied with 8-bit integer activations on the tensor cores (paper Sec. 6.2 "mpGEMM": per-tensor
// weights are dequantized to INT8 for the matrix unit; Sec. 4.1 / Fig. 7: bit repacking + conversion table;
// Sec. 4.2 / Fig. 9: load, dequantize and multiply as three pipelined agents).
//
//   acc[m][n] = sum_k a8[m][k] * (q[k][n] - 1)        (exact, int32 accumulators in tensor memory)
//   y[m][n]   = fp16( row_scale[m] * w_scale * acc[m][n] )
//
// One CTA per SM walks over tiles of 128 tokens x BN channels (BN = 256 when the output still has two
// tiles or more per SM, else 128).  Per k-block of 128 (one 128-byte row of INT8):
//   warp 0      TMA: the activation tile (2-D map, 128-byte swizzle) and the two plane tiles of the
//               CTA's channels (3-D map over (word/column, plane, strip)) into a ring of 6 (BN = 128) or 4 stages
//   next BN/32 warps   dequantization: a thread takes the plane words of one strip (four channels) and 32 k:
//               level 1 interleaves the two planes into 2-bit codes, one per nibble, in k order; level 2
//               looks four codes at a time up in a four-entry byte table {-1, 0, +1, 0} with one byte
//               permute; 32 INT8 per channel are stored into the K-major, 128-byte-swizzled weight tile
//   warp 1      tcgen05.mma kind::i8 (128 x BN x 32 per instruction), commit releases the stage
//               (two accumulator sets in tensor memory: a tile's epilogue overlaps the next tile's MMAs)
//   last 4 warps   epilogue: tcgen05.ld of 32 tokens x 32 channels, integer -> float, the row's and the
//               tensor's scale, fp16, 64-byte row stores
// Every wait is bounded (about a second) and reports TMAN_ERR_TIMEOUT; tensor memory is always freed.
#include "common.cuh"

#include <cuda.h>

#include "sm100_ptx.cuh"

namespace tman {
namespace {

constexpr int I8_BM = 128, I8_BK = 128;
constexpr int I8_A_BYTES = I8_BM * I8_BK;                               // 16 KB
constexpr int I8_EPI_WARPS = 4;
// Tile width BN = 128 or 256 channels (256 when the output still has enough tiles for every SM): one
// dequantization warp per 32 channels, as many stages as fit the shared memory.
template <int BN> struct I8Cfg {
    static constexpr int B_BYTES = BN * I8_BK;                              // 16 / 32 KB
    static constexpr int P_PLANE_BYTES = (BN / 4) * (I8_BK / 32) * 16;      // strips x 4 words x 4 columns x 4 B
    static constexpr int P_BYTES = 2 * P_PLANE_BYTES;
    static constexpr int STAGES = BN == 128 ? 6 : 4;                        // 36 / 56 KB each
    static constexpr int DEQ_WARPS = BN / 32;
    static constexpr int THREADS = 32 * (2 + DEQ_WARPS + I8_EPI_WARPS);
    static constexpr int SMEM_BYTES = STAGES * (I8_A_BYTES + B_BYTES + P_BYTES) + 256;
};

struct GemmI8Params {
    const uint8_t *packed;
    const float   *row_scale;
    float          w_scale;
    __half        *y;
    uint32_t      *status;
    int M, K, N, group;
    int tiles_m, tiles_n;
};

template <int I8_BN>
__global__ void __launch_bounds__(I8Cfg<I8_BN>::THREADS, 1)
mpgemm_i8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w, const GemmI8Params p)
{
    using C = I8Cfg<I8_BN>;
    constexpr int I8_STAGES = C::STAGES, I8_B_BYTES = C::B_BYTES, I8_P_PLANE_BYTES = C::P_PLANE_BYTES, I8_P_BYTES = C::P_BYTES;
    constexpr int I8_DEQ_WARPS = C::DEQ_WARPS, I8_TMEM_COLS = 2 * I8_BN;     // two accumulator sets: the epilogue of a tile
                                                                             // overlaps the multiplications of the next
    extern __shared__ __align__(1024) uint8_t smem[];
    if (!header_matches(p.packed, p.K, p.N, 2, p.group)) {          // same answer in every CTA
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_BAD_PACKED);
        return;
    }
    if ((smem_u32(smem) & 1023u) != 0u) {                           // the swizzled tiles need 1 KB alignment
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_LAYOUT);
        return;
    }
    uint8_t *a_tiles = smem;
    uint8_t *b_tiles = smem + I8_STAGES * I8_A_BYTES;
    uint8_t *p_tiles = smem + I8_STAGES * (I8_A_BYTES + I8_B_BYTES);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + I8_STAGES * (I8_A_BYTES + I8_B_BYTES + I8_P_BYTES));
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * I8_STAGES + 4);
    const uint32_t loaded0 = smem_u32(bars), full0 = smem_u32(bars + I8_STAGES), empty0 = smem_u32(bars + 2 * I8_STAGES),
                   accf = smem_u32(bars + 3 * I8_STAGES), acce = smem_u32(bars + 3 * I8_STAGES + 2);   // two of each
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = p.K / I8_BK;
    const int tiles = p.tiles_m * p.tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < I8_STAGES; ++s) {
            mbar_init(loaded0 + 8 * s, 1);
            mbar_init(full0 + 8 * s, I8_DEQ_WARPS);
            mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(accf + 8 * b, 1);
            mbar_init(acce + 8 * b, I8_EPI_WARPS);
        }
        *tmem_slot = 0xFFFFFFFFu;
        fence_barrier_init();
    }
    __syncthreads();
    if (warp == 1) {
        tcgen05_alloc(smem_u32(tmem_slot), I8_TMEM_COLS);
        tcgen05_relinquish();
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(tmem_slot);
    bool ok = tmem_base != 0xFFFFFFFFu;

    // tile t: row tile fastest, so that CTAs running at the same time share the weight columns in L2
    auto tile_m0 = [&](int t) { return (t % p.tiles_m) * I8_BM; };
    auto tile_n0 = [&](int t) { return (t / p.tiles_m) * I8_BN; };

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            for (int t = blockIdx.x; ok && t < tiles; t += gridDim.x) {
                const int m0 = tile_m0(t), strip0 = tile_n0(t) / 4;
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = (int)(it % I8_STAGES);
                    const uint32_t ph = (it / I8_STAGES) & 1u;
                    if (!mbar_wait(empty0 + 8 * s, ph ^ 1u)) { ok = false; break; }
                    mbar_expect_tx(loaded0 + 8 * s, I8_A_BYTES + I8_P_BYTES);
                    tma_load_2d(smem_u32(a_tiles + s * I8_A_BYTES), &tmap_a, kb * I8_BK, m0, loaded0 + 8 * s);
#pragma unroll
                    for (int i = 0; i < 2; ++i)
                        tma_load_3d(smem_u32(p_tiles + s * I8_P_BYTES + i * I8_P_PLANE_BYTES), &tmap_w, kb * (I8_BK / 8), i,
                                    strip0, loaded0 + 8 * s);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // instruction descriptor: D = s32, A = B = s8, both K-major, N = tile width, M = 128
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(I8_BN >> 3) << 17) | ((uint32_t)(I8_BM >> 4) << 24);
            uint32_t it = 0, ti = 0;
            for (int t = blockIdx.x; ok && t < tiles; t += gridDim.x, ++ti) {
                const uint32_t buf = ti & 1u, acc_tmem = tmem_base + buf * (uint32_t)I8_BN;
                if (!mbar_wait(acce + 8 * buf, ((ti >> 1) & 1u) ^ 1u)) { ok = false; break; }
                tcgen05_fence_after();
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = (int)(it % I8_STAGES);
                    const uint32_t ph = (it / I8_STAGES) & 1u;
                    if (!mbar_wait(full0 + 8 * s, ph)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint64_t adesc = make_kmajor_sw128_desc(smem_u32(a_tiles + s * I8_A_BYTES));
                    const uint64_t bdesc = make_kmajor_sw128_desc(smem_u32(b_tiles + s * I8_B_BYTES));
#pragma unroll
                    for (int j = 0; j < I8_BK / 32; ++j)          // 32 k = 32 bytes = two 16-byte units per instruction
                        tcgen05_mma_i8(acc_tmem, adesc + 2 * j, bdesc + 2 * j, idesc, (kb > 0 || j > 0) ? 1u : 0u);
                    tcgen05_commit(empty0 + 8 * s);
                }
                if (ok) tcgen05_commit(accf + 8 * buf);
            }
        }
    } else if (warp < 2 + I8_DEQ_WARPS) {
        // thread d: strip d / 4 of the tile (four channels), plane word d % 4 of the k-block (32 k)
        const int d = threadIdx.x - 64, strip = d >> 2, v = d & 3;
        const uint32_t p_off = (uint32_t)strip * 64u + (uint32_t)v * 16u;
        const uint32_t table = 0x000100FFu;                      // byte c = value of code c: -1, 0, +1, (3 does not occur) 0
        uint32_t it = 0;
        for (int t = blockIdx.x; ok && t < tiles; t += gridDim.x) {
            for (int kb = 0; kb < num_kb; ++kb, ++it) {
                const int s = (int)(it % I8_STAGES);
                const uint32_t ph = (it / I8_STAGES) & 1u;
                if (!mbar_wait(loaded0 + 8 * s, ph)) { ok = false; break; }
                const uint32_t pp = smem_u32(p_tiles + s * I8_P_BYTES) + p_off;
                uint4 w0, w1;
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w0.x), "=r"(w0.y), "=r"(w0.z), "=r"(w0.w) : "r"(pp) : "memory");
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w1.x), "=r"(w1.y), "=r"(w1.z), "=r"(w1.w)
                             : "r"(pp + I8_P_PLANE_BYTES) : "memory");
                const uint32_t btile = smem_u32(b_tiles + s * I8_B_BYTES);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t p0 = c == 0 ? w0.x : c == 1 ? w0.y : c == 2 ? w0.z : w0.w;
                    const uint32_t p1 = c == 0 ? w1.x : c == 1 ? w1.y : c == 2 ? w1.z : w1.w;
                    // level 1: word bit 4j + ph belongs to weight 8ph + j; X[ph] nibble j = its 2-bit code
                    const uint32_t a0 = (p0 & 0x55555555u) | ((p1 << 1) & 0xAAAAAAAAu);
                    const uint32_t a1 = ((p0 >> 1) & 0x55555555u) | (p1 & 0xAAAAAAAAu);
                    const uint32_t X0 = a0 & 0x33333333u, X2 = (a0 >> 2) & 0x33333333u;
                    const uint32_t X1 = a1 & 0x33333333u, X3 = (a1 >> 2) & 0x33333333u;
                    // Threads of odd strips write their two 16-byte chunks in the other order: a quarter-warp
                    // (two strips x four words) then covers all eight chunk positions of the swizzle in
                    // each store instruction instead of four of them twice (no bank conflicts).
                    const bool odd = (strip & 1) != 0;
                    const uint32_t Xa0 = odd ? X2 : X0, Xa1 = odd ? X3 : X1, Xb0 = odd ? X0 : X2, Xb1 = odd ? X1 : X3;
                    const uint32_t ca = (uint32_t)(2 * v) + (odd ? 1u : 0u), cb = ca ^ 1u;
                    // level 2: four codes per byte permute
                    const uint32_t o0 = __byte_perm(table, 0u, Xa0), o1 = __byte_perm(table, 0u, Xa0 >> 16);
                    const uint32_t o2 = __byte_perm(table, 0u, Xa1), o3 = __byte_perm(table, 0u, Xa1 >> 16);
                    const uint32_t o4 = __byte_perm(table, 0u, Xb0), o5 = __byte_perm(table, 0u, Xb0 >> 16);
                    const uint32_t o6 = __byte_perm(table, 0u, Xb1), o7 = __byte_perm(table, 0u, Xb1 >> 16);
                    // channel row of the tile, 128 bytes per row, 16-byte chunk index XOR (row & 7)
                    const uint32_t row = (uint32_t)(4 * strip + c), xr = row & 7u;
                    const uint32_t rbase = btile + (row >> 3) * 1024u + xr * 128u;
                    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(rbase + (ca ^ xr) * 16u),
                                 "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(rbase + (cb ^ xr) * 16u),
                                 "r"(o4), "r"(o5), "r"(o6), "r"(o7) : "memory");
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(full0 + 8 * s);
            }
        }
    } else {
        // epilogue warp: its quarter of the tensor-memory lanes = 32 tokens, one per lane
        const int quarter = warp & 3;
        uint32_t ti = 0;
        for (int t = blockIdx.x; ok && t < tiles; t += gridDim.x, ++ti) {
            const int m = tile_m0(t) + quarter * 32 + lane, n0 = tile_n0(t);
            const uint32_t buf = ti & 1u;
            if (!mbar_wait(accf + 8 * buf, (ti >> 1) & 1u)) { ok = false; break; }
            tcgen05_fence_after();
            const float sc = (m < p.M) ? __ldg(p.row_scale + m) * p.w_scale : 0.f;
#pragma unroll 1
            for (int cc = 0; cc < I8_BN / 32; ++cc) {
                uint32_t r[32];
                tcgen05_ld_32x32b_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * (uint32_t)I8_BN + (uint32_t)(32 * cc), r);
                tcgen05_wait_ld();
                if (m < p.M) {
#pragma unroll
                    for (int g8 = 0; g8 < 4; ++g8) {                 // eight channels = 16 bytes at a time (N % 8 == 0)
                        const int n = n0 + 32 * cc + 8 * g8;
                        if (n < p.N) {
                            uint32_t h[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __half2 hh = __floats2half2_rn((float)(int)r[8 * g8 + 2 * e] * sc, (float)(int)r[8 * g8 + 2 * e + 1] * sc);
                                h[e] = *reinterpret_cast<const uint32_t *>(&hh);
                            }
                            *reinterpret_cast<uint4 *>(p.y + (size_t)m * p.N + n) = make_uint4(h[0], h[1], h[2], h[3]);
                        }
                    }
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce + 8 * buf);
        }
    }
    if (!ok && lane == 0) atomicCAS(p.status, 0u, (uint32_t)TMAN_ERR_TIMEOUT);
    __syncthreads();
    if (warp == 1 && tmem_base != 0xFFFFFFFFu) {
        tcgen05_fence_after();
        tcgen05_dealloc(tmem_base, I8_TMEM_COLS);
    }
}

}  // namespace

namespace {
template <int BN>
tman_status launch_i8(const CUtensorMap &tmap_a, const CUtensorMap &tmap_w, GemmI8Params p, int sms, cudaStream_t s)
{
    using C = I8Cfg<BN>;
    p.tiles_n = (p.N + BN - 1) / BN;
    const int tiles = p.tiles_m * p.tiles_n;
    auto kern = mpgemm_i8_kernel<BN>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess) return TMAN_ERR_CUDA;
    const int grid = tiles < sms ? tiles : sms;
    kern<<<(unsigned)grid, C::THREADS, C::SMEM_BYTES, s>>>(tmap_a, tmap_w, p);
    return launch_status();
}
}  // namespace

tman_status launch_mpgemm_ternary_i8(const void *packed, const int8_t *a8, const float *row_scale, float w_scale, void *y,
                                     int M, int K, int N, int group, void *ws, cudaStream_t s)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return TMAN_ERR_CUDA;
    const int sms = sm_count();
    if (sms <= 0) return TMAN_ERR_CUDA;
    const cuuint32_t estr[3] = {1, 1, 1};
    // 256-channel tiles when they still give every SM two tiles or more, else 128-channel tiles
    const long long tiles256 = (long long)((M + I8_BM - 1) / I8_BM) * ((N + 255) / 256);
    const bool wide = tiles256 >= 2LL * sms;
    const int bn = wide ? 256 : 128;
    CUtensorMap tmap_a;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
        const cuuint64_t strides[1] = {(cuuint64_t)K};
        const cuuint32_t box[2] = {(cuuint32_t)I8_BK, (cuuint32_t)I8_BM};
        if (enc(&tmap_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(a8), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TMAN_ERR_CUDA;
    }
    Layout L = make_layout(K, N, 2, group);
    const uint8_t *pk = static_cast<const uint8_t *>(packed);
    CUtensorMap tmap_w;
    {
        const cuuint64_t wt = (cuuint64_t)(K / 32);
        const cuuint64_t wdims[3] = {wt * 4, 2, (cuuint64_t)(N / 4)};
        const cuuint64_t wstrides[2] = {wt * 16, wt * 16 * 2};
        const cuuint32_t wbox[3] = {(cuuint32_t)(I8_BK / 8), 1, (cuuint32_t)(bn / 4)};
        if (enc(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint8_t *>(pk + L.planes_off), wdims, wstrides,
                wbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TMAN_ERR_CUDA;
    }
    GemmI8Params p;
    p.packed = pk;
    p.row_scale = row_scale;
    p.w_scale = w_scale;
    p.y = static_cast<__half *>(y);
    p.status = static_cast<uint32_t *>(ws);
    p.M = M; p.K = K; p.N = N; p.group = group;
    p.tiles_m = (M + I8_BM - 1) / I8_BM;
    return wide ? launch_i8<256>(tmap_a, tmap_w, p, sms, s) : launch_i8<128>(tmap_a, tmap_w, p, sms, s);
}

}  // namespace tman
