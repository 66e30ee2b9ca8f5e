// Microbenchmarks behind the decode kernel's design: what one SM can look up per clock with the
// candidate table shapes, what a load path streams, and what the building blocks of a split-K
// combine cost.  The paper settles the same questions for its vector unit with an instruction
// study (Sec. 5 "Implementation", Table 1: 16-entry against 32-entry lookup instructions, counted as
// lookups x log2(entries) "equivalent multiply-adds") and a load-path study (Table 2: DMA against
// prefetch against vector loads).  Nothing here is on the product path.
#include "common.cuh"

namespace tman {
namespace {

constexpr int kMbThreads = 512;
constexpr int kMbPoolBytes = 16 * 1024;          // index words, read the way a staged weight tile is
constexpr int kMbTableBytes = 128 * 1024;
constexpr int kMbRounds = 64;                    // passes over the index pool per thread

__device__ __forceinline__ uint32_t hash32(uint32_t v)
{
    v ^= v >> 16; v *= 0x7feb352du; v ^= v >> 15; v *= 0x846ca68bu; v ^= v >> 16;
    return v;
}

// One lookup per index byte (8 weights of one bit-plane), fp32 entries, bank = lane.
struct LutF32x256 {
    static constexpr int kWeightsPerLookup = 8;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    uint32_t lane_off;
    __device__ void init(int lane) { lane_off = (uint32_t)lane * 4u; }
    template <int C> __device__ __forceinline__ void look(uint32_t w, int col, uint32_t base)
    {
        const uint32_t off = __byte_perm(w, lane_off, 0x7604u | ((uint32_t)C << 4));
        float t;
        asm volatile("ld.shared.f32 %0, [%1 + %2];" : "=f"(t) : "r"(off + base), "n"((C >> 1) * 65536 + (C & 1) * 128));
        acc[col] += t;
    }
    __device__ float result() const { return acc[0] + acc[1] + acc[2] + acc[3]; }
};

// The same with fp16 entries (two tables share a bank word) and a mixed-precision add.
struct LutF16x256 {
    static constexpr int kWeightsPerLookup = 8;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    uint32_t lane_off;
    __device__ void init(int lane) { lane_off = (uint32_t)lane * 4u; }
    template <int C> __device__ __forceinline__ void look(uint32_t w, int col, uint32_t base)
    {
        const uint32_t off = __byte_perm(w, lane_off, 0x7604u | ((uint32_t)C << 4));
        unsigned short t;
        asm volatile("ld.shared.u16 %0, [%1 + %2];" : "=h"(t) : "r"(off + base), "n"((C >> 1) * 128 + (C & 1) * 2));
        asm volatile("add.f32.f16 %0, %1, %0;" : "+f"(acc[col]) : "h"(t));
    }
    __device__ float result() const { return acc[0] + acc[1] + acc[2] + acc[3]; }
};

// 16-entry fp32 tables indexed by a nibble (4 weights of one bit-plane): the paper's table shape.
struct LutF32x16 {
    static constexpr int kWeightsPerLookup = 4;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    uint32_t lane_off;
    __device__ void init(int lane) { lane_off = (uint32_t)lane * 4u; }
    template <int NIB> __device__ __forceinline__ void look_nibble(uint32_t w, int col, uint32_t base)
    {
        const uint32_t off = ((w >> (4 * NIB)) & 15u) * 128u + lane_off;
        float t;
        asm volatile("ld.shared.f32 %0, [%1 + %2];" : "=f"(t) : "r"(off + base), "n"(NIB * 2048));
        acc[col] += t;
    }
    template <int C> __device__ __forceinline__ void look(uint32_t w, int col, uint32_t base)
    {
        look_nibble<2 * C>(w, col, base);
        look_nibble<2 * C + 1>(w, col, base);
    }
    __device__ float result() const { return acc[0] + acc[1] + acc[2] + acc[3]; }
};

// 16-entry tables spread over the lanes of a half-warp and read with a shuffle (lanes = output
// channels, as on the paper's vector unit).
struct LutShfl16 {
    static constexpr int kWeightsPerLookup = 4;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    float tab[8];
    __device__ void init(int lane)
    {
#pragma unroll
        for (int n = 0; n < 8; ++n) tab[n] = (float)((lane * 7 + n * 3) & 15) * 0.125f;
    }
    template <int C> __device__ __forceinline__ void look(uint32_t w, int col, uint32_t)
    {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int nib = 2 * C + h;
            acc[col] += __shfl_sync(0xffffffffu, tab[nib], (int)(w >> (4 * nib)), 16);
        }
    }
    __device__ float result() const { return acc[0] + acc[1] + acc[2] + acc[3]; }
};

// 256-entry tables whose entries carry ROWS activation rows in fp16 (a 4-, 8- or 16-byte load),
// accumulated with packed half-precision adds.
template <int ROWS>
struct LutF16Rows {
    static constexpr int kWeightsPerLookup = 8;
    static constexpr int kSlots = 64 / ROWS;     // entries of one table that fit 128 bytes (half a 256-byte row)
    __half2 acc[4][ROWS / 2];
    uint32_t lane_off;
    __device__ void init(int lane)
    {
        lane_off = (uint32_t)(lane % kSlots) * (uint32_t)(2 * ROWS);
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int r = 0; r < ROWS / 2; ++r) acc[c][r] = __floats2half2_rn(0.f, 0.f);
    }
    template <int C> __device__ __forceinline__ void look(uint32_t w, int col, uint32_t base)
    {
        const uint32_t off = __byte_perm(w, lane_off, 0x7604u | ((uint32_t)C << 4)) + base;
        uint32_t t[ROWS / 2];
        if constexpr (ROWS == 2) {
            asm volatile("ld.shared.b32 %0, [%1 + %2];" : "=r"(t[0]) : "r"(off), "n"((C >> 1) * 65536 + (C & 1) * 128));
        } else if constexpr (ROWS == 4) {
            asm volatile("ld.shared.v2.b32 {%0, %1}, [%2 + %3];" : "=r"(t[0]), "=r"(t[1]) : "r"(off), "n"((C >> 1) * 65536 + (C & 1) * 128));
        } else {
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4 + %5];"
                         : "=r"(t[0]), "=r"(t[1]), "=r"(t[2]), "=r"(t[3]) : "r"(off), "n"((C >> 1) * 65536 + (C & 1) * 128));
        }
#pragma unroll
        for (int r = 0; r < ROWS / 2; ++r) acc[col][r] = __hadd2(acc[col][r], *reinterpret_cast<const __half2 *>(&t[r]));
    }
    __device__ float result() const
    {
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int r = 0; r < ROWS / 2; ++r) s += __low2float(acc[c][r]) + __high2float(acc[c][r]);
        return s;
    }
};

// Every thread reads 16-byte groups of index words from a shared-memory pool (conflict-free: eight
// adjacent lanes read eight adjacent groups) and does one lookup per index byte, four columns per
// group.  Reports the clocks the CTA took.
template <class LUT>
__global__ void __launch_bounds__(kMbThreads, 1) lookup_bench_kernel(unsigned long long *clocks, float *sink)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    uint32_t *pool = reinterpret_cast<uint32_t *>(smem + kMbTableBytes);
    const int tid = threadIdx.x, lane = tid & 31;
    for (int i = tid; i < kMbTableBytes / 4; i += blockDim.x)
        reinterpret_cast<uint32_t *>(smem)[i] = 0x3c003c00u ^ ((hash32((uint32_t)i) & 0x03ff03ffu) >> 1);
    for (int i = tid; i < kMbPoolBytes / 4; i += blockDim.x) pool[i] = hash32(0x9e3779b9u * (uint32_t)(i + 1) + blockIdx.x);
    __syncthreads();
    LUT lut;
    lut.init(lane);
    const uint32_t base = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t pool_addr = (uint32_t)__cvta_generic_to_shared(pool);
    const int groups = kMbPoolBytes / 16;
    const long long t0 = clock64();
    for (int r = 0; r < kMbRounds; ++r) {
#pragma unroll 2
        for (int g = tid; g < groups; g += (int)blockDim.x) {
            uint32_t w[4];
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(pool_addr + (uint32_t)((g + r) % groups) * 16u));
#pragma unroll
            for (int col = 0; col < 4; ++col) {
                lut.template look<0>(w[col], col, base);
                lut.template look<1>(w[col], col, base);
                lut.template look<2>(w[col], col, base);
                lut.template look<3>(w[col], col, base);
            }
        }
    }
    const long long t1 = clock64();
    __syncthreads();
    const float res = lut.result();
    if (res == 123.456f) sink[0] = res;
    if (tid == 0) clocks[blockIdx.x] = (unsigned long long)(t1 - t0);
}

template <class LUT>
tman_status launch_lookup_bench(int threads, unsigned long long *clocks, float *sink, int sms, cudaStream_t s)
{
    auto kern = lookup_bench_kernel<LUT>;
    const int smem = kMbTableBytes + kMbPoolBytes;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return TMAN_ERR_CUDA;
    kern<<<sms, threads, smem, s>>>(clocks, sink);
    return launch_status();
}

// ---- load paths ------------------------------------------------------------------------------
// Coalesced 16-byte loads, every CTA streaming its contiguous share once.
__global__ void __launch_bounds__(kMbThreads, 1) stream_ldg_kernel(const uint4 *buf, size_t n16, float *sink)
{
    const size_t per = n16 / gridDim.x;
    const uint4 *p = buf + per * blockIdx.x;
    uint32_t a = 0;
    for (size_t i = threadIdx.x; i + 3 * kMbThreads < per; i += 4 * kMbThreads) {
        const uint4 v0 = __ldcs(p + i), v1 = __ldcs(p + i + kMbThreads), v2 = __ldcs(p + i + 2 * kMbThreads),
                    v3 = __ldcs(p + i + 3 * kMbThreads);
        a ^= v0.x ^ v1.y ^ v2.z ^ v3.w;
    }
    if (a == 0x12345678u) sink[0] = 1.f;
}

__device__ __forceinline__ bool mb_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Bulk asynchronous copies (cp.async.bulk) of `chunk` bytes into a ring of shared-memory stages; the
// warps only wait for a stage and read one word of it.  Waits are bounded.
__global__ void __launch_bounds__(128, 1) stream_bulk_kernel(const uint8_t *buf, size_t bytes, int chunk, int stages,
                                                             float *sink, uint32_t *status)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)stages * chunk);
    const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
    const uint32_t dst0 = (uint32_t)__cvta_generic_to_shared(smem);
    const size_t per = (bytes / gridDim.x) / chunk * chunk;
    const uint8_t *src = buf + per * blockIdx.x;
    const int nchunks = (int)(per / chunk);
    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0 + 8 * i) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    auto issue = [&](int c) {
        const int st = c % stages;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar0 + 8 * st), "r"(chunk) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(dst0 + (uint32_t)st * chunk), "l"(src + (size_t)c * chunk), "r"(chunk), "r"(bar0 + 8 * st) : "memory");
    };
    if (threadIdx.x == 0)
        for (int c = 0; c < stages && c < nchunks; ++c) issue(c);
    uint32_t a = 0;
    bool bad = false;
    for (int c = 0; c < nchunks && !bad; ++c) {
        const int st = c % stages;
        const uint32_t parity = (uint32_t)(c / stages) & 1u;
        uint32_t tries = 0;
        while (!mb_try(bar0 + 8 * st, parity)) {
            if (++tries > (1u << 22)) { bad = true; break; }
        }
        a ^= reinterpret_cast<const uint32_t *>(smem + (size_t)st * chunk)[threadIdx.x];
        __syncthreads();                       // everyone has read the stage: refill it
        if (threadIdx.x == 0 && c + stages < nchunks) issue(c + stages);
    }
    if (bad) atomicCAS(status, 0u, (uint32_t)TMAN_ERR_TIMEOUT);
    if (a == 0x12345678u) sink[0] = 1.f;
}

// ---- building blocks of a split-K combine ------------------------------------------------------
// Clocks of (a) a cluster barrier alone and (b) a store to every peer's shared memory followed by a
// release/acquire cluster barrier and a read of what the peers stored; averaged over `reps` rounds.
__global__ void __launch_bounds__(256, 1) cluster_exchange_kernel(unsigned long long *out, int reps)
{
    __shared__ float inbox[16][256];
    uint32_t rank, size;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(size));
    const uint32_t my = (uint32_t)__cvta_generic_to_shared(&inbox[rank][threadIdx.x]);
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    long long t0 = clock64();
    for (int r = 0; r < reps; ++r)
        asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    long long t1 = clock64();
    float acc = 0.f;
    for (int r = 0; r < reps; ++r) {
        for (uint32_t peer = 0; peer < size; ++peer) {
            uint32_t remote;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(my), "r"(peer));
            asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"((float)(r + rank)) : "memory");
        }
        asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        for (uint32_t peer = 0; peer < size; ++peer) acc += inbox[peer][threadIdx.x];
        asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
    long long t2 = clock64();
    if (threadIdx.x == 0) {
        out[2 * blockIdx.x] = (unsigned long long)(t1 - t0) / (unsigned)reps;
        out[2 * blockIdx.x + 1] = (unsigned long long)(t2 - t1) / (unsigned)reps;
    }
    if (acc == 123.456f) out[0] = 0;
}

// Dependent loads through a chain that fits L2 (one thread): clocks per load.
__global__ void chase_kernel(const uint32_t *chain, int steps, unsigned long long *out)
{
    uint32_t i = 0;
    for (int s = 0; s < 64; ++s) i = __ldcg(chain + i);
    const long long t0 = clock64();
    for (int s = 0; s < steps; ++s) i = __ldcg(chain + i);
    const long long t1 = clock64();
    out[0] = (unsigned long long)(t1 - t0) / (unsigned)steps;
    out[1] = i;
}
__global__ void chase_init_kernel(uint32_t *chain, uint32_t n, uint32_t stride)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) chain[i] = (i + stride) % n;
}

__global__ void noop_cluster_kernel(int) {}

}  // namespace

tman_status launch_microbench(int kind, int arg, void *results, size_t results_bytes, void *buffer, size_t buffer_bytes,
                              cudaStream_t s)
{
    const int sms = sm_count();
    if (sms <= 0) return TMAN_ERR_CUDA;
    auto *res64 = static_cast<unsigned long long *>(results);
    auto *sink = reinterpret_cast<float *>(static_cast<uint8_t *>(results) + results_bytes - 256);
    if (kind >= 0 && kind <= 6) {
        const int threads = (arg >= 32 && arg <= kMbThreads && arg % 32 == 0) ? arg : kMbThreads;
        if (results_bytes < (size_t)sms * 8 + 256) return TMAN_ERR_BUFFER_TOO_SMALL;
        switch (kind) {
            case 0: return launch_lookup_bench<LutF32x256>(threads, res64, sink, sms, s);
            case 1: return launch_lookup_bench<LutF16x256>(threads, res64, sink, sms, s);
            case 2: return launch_lookup_bench<LutF32x16>(threads, res64, sink, sms, s);
            case 3: return launch_lookup_bench<LutShfl16>(threads, res64, sink, sms, s);
            case 4: return launch_lookup_bench<LutF16Rows<2>>(threads, res64, sink, sms, s);
            case 5: return launch_lookup_bench<LutF16Rows<4>>(threads, res64, sink, sms, s);
            default: return launch_lookup_bench<LutF16Rows<8>>(threads, res64, sink, sms, s);
        }
    }
    if (kind == 10) {
        if (!buffer || buffer_bytes < (size_t)sms * kMbThreads * 64) return TMAN_ERR_BUFFER_TOO_SMALL;
        stream_ldg_kernel<<<sms, kMbThreads, 0, s>>>(static_cast<const uint4 *>(buffer), buffer_bytes / 16, sink);
        return launch_status();
    }
    if (kind == 11) {
        // arg = chunk bytes (a multiple of 1 KB); as many stages as fit 192 KB, at most 16
        const int chunk = (arg >= 1024 && arg <= 65536 && arg % 1024 == 0) ? arg : 8192;
        int stages = (192 * 1024) / chunk;
        if (stages > 16) stages = 16;
        if (!buffer || buffer_bytes < (size_t)sms * chunk * stages) return TMAN_ERR_BUFFER_TOO_SMALL;
        const int smem = stages * chunk + 256;
        if (cudaFuncSetAttribute(stream_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return TMAN_ERR_CUDA;
        stream_bulk_kernel<<<sms, 128, smem, s>>>(static_cast<const uint8_t *>(buffer), buffer_bytes, chunk, stages, sink,
                                                   reinterpret_cast<uint32_t *>(results));
        return launch_status();
    }
    if (kind == 20) {
        // arg = cluster size (1, 2, 4, 8); one cluster per 16 SMs is plenty for a latency figure
        const int cs = (arg == 1 || arg == 2 || arg == 4 || arg == 8) ? arg : 4;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(cs * 8));
        cfg.blockDim = dim3(256);
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cs;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (results_bytes < (size_t)cs * 8 * 16 + 256) return TMAN_ERR_BUFFER_TOO_SMALL;
        if (cudaLaunchKernelEx(&cfg, cluster_exchange_kernel, res64, 64) != cudaSuccess) return TMAN_ERR_CUDA;
        return TMAN_OK;
    }
    if (kind == 21) {
        // arg = chain bytes (kept in L2 when it is a few MB); stride of 4 KB + one line between links
        const uint32_t n = (uint32_t)((arg > 0 ? (size_t)arg : (size_t)(8 << 20)) / 4);
        if (!buffer || buffer_bytes < (size_t)n * 4) return TMAN_ERR_BUFFER_TOO_SMALL;
        chase_init_kernel<<<(n + 255) / 256, 256, 0, s>>>(static_cast<uint32_t *>(buffer), n, 1024 + 32);
        chase_kernel<<<1, 1, 0, s>>>(static_cast<const uint32_t *>(buffer), 2048, res64);
        return launch_status();
    }
    return TMAN_ERR_UNSUPPORTED;
}

// How many clusters of `cluster` CTAs (threads, dynamic shared memory each) the current device can
// hold at once (0 on error).
int cluster_capacity(int threads, int smem_bytes, int cluster)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)cluster * 64);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(noop_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess) return 0;
    if (cluster > 8 &&
        cudaFuncSetAttribute(noop_cluster_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) return 0;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, noop_cluster_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    return n;
}

}  // namespace tman
