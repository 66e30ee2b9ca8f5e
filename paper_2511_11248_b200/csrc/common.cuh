// Shared declarations of the CUDA side: packed-buffer layout, workspace layout, argument checks.
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>

#include "tman.h"

namespace tman {

// ---- packed buffer -----------------------------------------------------------------------
// 256-byte header, then bit-plane words, scales, zero-points (each section 256-byte padded).
struct PackedHeader {
    char     magic[8];      // "TMANB200"
    uint32_t version;       // kVersion
    uint32_t K, N, bits, group, lut_g;
    uint64_t planes_off, scales_off, zeros_off, total_bytes;
};
static_assert(sizeof(PackedHeader) == 64, "header fields occupy the first 64 bytes");

constexpr size_t   kHeaderBytes = 256;
constexpr uint32_t kVersion = 2;

// Bit of a plane word that holds the weight with k % 32 == r: weight 8*ph + j sits at bit 4*j + ph
// (an offline permutation, paper Sec. 4.1, that makes the prefill repacking come out in k order).
__host__ __device__ constexpr int plane_bit(int r) { return 4 * (r & 7) + (r >> 3); }

__host__ __device__ inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

struct Layout {
    size_t planes_off, scales_off, zeros_off, total;
    size_t planes_bytes, scales_bytes, zeros_bytes;
};

__host__ __device__ inline Layout make_layout(int K, int N, int bits, int group)
{
    Layout L;
    L.planes_bytes = (size_t)K * N * bits / 8;
    L.scales_bytes = (size_t)(K / group) * N * 2;
    L.zeros_bytes = (size_t)(K / group) * (N / 4) * 2;
    L.planes_off = kHeaderBytes;
    L.scales_off = L.planes_off + up256(L.planes_bytes);
    L.zeros_off = L.scales_off + up256(L.scales_bytes);
    L.total = L.zeros_off + up256(L.zeros_bytes);
    return L;
}

// device-side header check: every kernel that reads a packed buffer calls it first
__device__ inline bool header_matches(const void *packed, int K, int N, int bits, int group)
{
    const uint32_t *h = reinterpret_cast<const uint32_t *>(packed);
    // "TMAN" = 0x4E414D54, "B200" = 0x30303242 (little endian)
    bool ok = (h[0] == 0x4E414D54u) && (h[1] == 0x30303242u) && (h[2] == kVersion) &&
              (h[3] == (uint32_t)K) && (h[4] == (uint32_t)N) && (h[5] == (uint32_t)bits) &&
              (h[6] == (uint32_t)group) && (h[7] == 4u);
    return ok;
}

// ---- workspace ---------------------------------------------------------------------------
// [0, 256)      status word (u32) + padding
// [256, ...)     fp32 split-K partial sums; "no sum pending" sentinel between calls
constexpr size_t kWsStatusBytes = 256;

// ---- argument checks (host) --------------------------------------------------------------
inline tman_status check_format(int K, int N, int bits, int group)
{
    if (K <= 0 || N <= 0) return TMAN_ERR_SHAPE;
    if (bits < 1 || bits > 4) return TMAN_ERR_SHAPE;
    if (group != 32 && group != 64 && group != 128) return TMAN_ERR_SHAPE;
    if (K % 128 != 0 || N % 8 != 0) return TMAN_ERR_SHAPE;
    return TMAN_OK;
}

inline tman_status launch_status()
{
    return cudaGetLastError() == cudaSuccess ? TMAN_OK : TMAN_ERR_CUDA;
}

// number of SMs of the current device (queried per call; cheap attribute read)
inline int sm_count()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return n;
}

// ---- table building block (device) -------------------------------------------------------
// The 16 partial sums of four activations: out[p] = sum_{j<4} x_j * bit_j(p), accumulated in
// increasing j (paper Sec. 2.2: each bit pattern indexes a precomputed sum).
__device__ __forceinline__ void lut16(float x0, float x1, float x2, float x3, float (&out)[16])
{
    out[0] = 0.f;
    out[1] = x0;
    out[2] = x1;
    out[3] = x0 + x1;
    out[4] = x2;
    out[5] = x0 + x2;
    out[6] = x1 + x2;
    out[7] = out[3] + x2;
#pragma unroll
    for (int p = 0; p < 8; ++p) out[8 + p] = (p == 0) ? x3 : out[p] + x3;
}

// entry points implemented per file
tman_status launch_pack(const uint8_t *codes, const void *scales, const uint8_t *zeros, int K, int N,
                        int bits, int group, void *packed, cudaStream_t s);
// A packing on stream s is followed by one decode launch in plain stream order (no programmatic
// dependent launch): note_packed_write records the stream, packed_write_pending asks and clears.
void note_packed_write(cudaStream_t s);
bool packed_write_pending(cudaStream_t s, bool clear);
tman_status launch_dequant_ternary_int8(const void *packed, int K, int N, int group, int8_t *w8, uint32_t *status,
                                        cudaStream_t s);
tman_status launch_unpack(const void *packed, int K, int N, int bits, int group, uint8_t *codes,
                          void *scales, uint8_t *zeros, uint32_t *status, cudaStream_t s);
tman_status launch_debug_indices(const void *packed, int K, int N, int bits, int group, uint8_t *idx,
                                 uint32_t *status, cudaStream_t s);
tman_status launch_debug_luts(const void *x, int M, int K, float *lut, cudaStream_t s);
size_t      mpgemv_workspace_bytes(int M, int K, int N, int bits);
// The decode call's plan: passes over the weights, each with one kernel variant (see mpgemv.cu).
constexpr int kGemvMaxRows = 8;
constexpr int kGemvVariantCount = 4;
constexpr int kGemvSmemLimit = 227 * 1024;
constexpr int kGemvPlanSms = 148;
struct GemvPass { int variant, rows, variant_rows, words, nkappa, ctas_per_slice, smem_bytes; };
struct GemvPlan { int npass; GemvPass pass[kGemvMaxRows]; size_t ws_bytes; double cost_us; };
tman_status launch_quantize_rows(const void *x, int M, int K, int qmax, int16_t *a, float *s_a, cudaStream_t s);
tman_status launch_mpgemv_ternary(const void *packed, const int16_t *a, const float *s_a, float s_w, void *y,
                                  int32_t *acc_out, int M, int K, int N, int group, void *ws, size_t ws_bytes, cudaStream_t s);
size_t      mpgemv_ternary_workspace_bytes(int M, int K, int N);
tman_status launch_wait_timeout(void *ws, size_t ws_bytes, uint32_t limit, cudaStream_t s);
GemvPlan    plan_gemv(int M, int K, int N, int bits, int sms, size_t ws_limit);
tman_status launch_workspace_init(void *ws, size_t ws_bytes, cudaStream_t s);
tman_status launch_mpgemv(const void *packed, const void *x, void *y, int M, int K, int N, int bits,
                          int group, void *ws, size_t ws_bytes, cudaStream_t s);
tman_status launch_mpgemv_grouped(int count, const void *const *packed, const void *x, void *const *y, int M, int K,
                                  const int *Ns, int bits, int group, void *ws, size_t ws_bytes, cudaStream_t s);
size_t      mpgemm_workspace_bytes(int M, int K, int N);
tman_status mpgemm_plan(int M, int K, int N, int bits, int *out8);
tman_status mpgemm_plan_for(int M, int K, int N, int bits, int sms, int resident, int *out8);
tman_status launch_quantize_rows_i8(const void *x, int M, int K, int8_t *a, float *s_a, cudaStream_t s);
tman_status launch_mpgemm_ternary_i8(const void *packed, const int8_t *a8, const float *row_scale, float w_scale, void *y,
                                     int M, int K, int N, int group, void *ws, cudaStream_t s);
tman_status mpgemm_read_stamps(const void *ws, int ctas, long long *out_host, cudaStream_t s);
tman_status launch_mpgemm_variant(int variant, const void *packed, const void *x, void *y, int M, int K, int N, int bits,
                                  int group, const void *wt_f16, void *ws, size_t ws_bytes, cudaStream_t s);
tman_status launch_mpgemm(const void *packed, const void *x, void *y, int M, int K, int N, int bits,
                          int group, void *ws, size_t ws_bytes, cudaStream_t s);
tman_status launch_microbench(int kind, int arg, void *results, size_t results_bytes, void *buffer, size_t buffer_bytes,
                              cudaStream_t s);
int         cluster_capacity(int threads, int smem_bytes, int cluster);

}  // namespace tman
