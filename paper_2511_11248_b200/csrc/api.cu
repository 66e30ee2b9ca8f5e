// C ABI: argument validation and dispatch.  No allocation, no global state, no device sync
// (except tman_read_status, whose job is to wait).
#include "common.cuh"

using namespace tman;

// Alignment rules of the header, in one place: packed buffers and workspaces start on a 256-byte
// boundary, activation and output matrices on a 16-byte boundary.  Checked on the host before anything
// touches the GPU; a violation is TMAN_ERR_SHAPE.
static bool aligned_to(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
static bool buffers_aligned(const void *packed, const void *workspace) { return aligned_to(packed, 256) && aligned_to(workspace, 256); }
static bool matrices_aligned(const void *x, const void *y) { return aligned_to(x, 16) && aligned_to(y, 16); }

extern "C" {

const char *tman_status_string(int status)
{
    switch (status) {
        case TMAN_OK: return "TMAN_OK";
        case TMAN_ERR_NULL: return "TMAN_ERR_NULL";
        case TMAN_ERR_SHAPE: return "TMAN_ERR_SHAPE";
        case TMAN_ERR_UNSUPPORTED: return "TMAN_ERR_UNSUPPORTED";
        case TMAN_ERR_BUFFER_TOO_SMALL: return "TMAN_ERR_BUFFER_TOO_SMALL";
        case TMAN_ERR_BAD_PACKED: return "TMAN_ERR_BAD_PACKED";
        case TMAN_ERR_CUDA: return "TMAN_ERR_CUDA";
        case TMAN_ERR_TIMEOUT: return "TMAN_ERR_TIMEOUT";
        case TMAN_ERR_LAYOUT: return "TMAN_ERR_LAYOUT";
        default: return "TMAN_ERR_UNKNOWN";
    }
}

int tman_version(void) { return 1000 * 0 + 1; }

tman_status tman_packed_bytes(int K, int N, int bits, int group, size_t *out_bytes)
{
    if (!out_bytes) return TMAN_ERR_NULL;
    tman_status st = check_format(K, N, bits, group);
    if (st != TMAN_OK) return st;
    *out_bytes = make_layout(K, N, bits, group).total;
    return TMAN_OK;
}

tman_status tman_workspace_bytes(int op, int M, int K, int N, int bits, int group, size_t *out_bytes)
{
    if (!out_bytes) return TMAN_ERR_NULL;
    tman_status st = check_format(K, N, bits, group);
    if (st != TMAN_OK) return st;
    if (M < 1) return TMAN_ERR_SHAPE;
    if (op == 0) {
        if (M > 8) return TMAN_ERR_SHAPE;
        *out_bytes = mpgemv_workspace_bytes(M, K, N, bits);
    } else if (op == 1) {
        *out_bytes = mpgemm_workspace_bytes(M, K, N);
    } else if (op == 2) {
        *out_bytes = kWsStatusBytes;
    } else if (op == 3) {
        if (M > 8) return TMAN_ERR_SHAPE;
        *out_bytes = mpgemv_ternary_workspace_bytes(M, K, N);
    } else {
        return TMAN_ERR_UNSUPPORTED;
    }
    return TMAN_OK;
}

tman_status tman_workspace_init(void *workspace, size_t ws_bytes, tman_stream_t stream)
{
    if (!workspace) return TMAN_ERR_NULL;
    if (ws_bytes < kWsStatusBytes) return TMAN_ERR_BUFFER_TOO_SMALL;
    if (!aligned_to(workspace, 256)) return TMAN_ERR_SHAPE;
    return launch_workspace_init(workspace, ws_bytes, reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_read_status(const void *workspace, int *out_status, tman_stream_t stream)
{
    if (!workspace || !out_status) return TMAN_ERR_NULL;
    if (!aligned_to(workspace, 256)) return TMAN_ERR_SHAPE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    uint32_t v = 0;
    if (cudaMemcpyAsync(&v, workspace, sizeof(v), cudaMemcpyDeviceToHost, s) != cudaSuccess) return TMAN_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return TMAN_ERR_CUDA;
    *out_status = (int)v;
    return TMAN_OK;
}

tman_status tman_pack_weights(const uint8_t *codes, const void *scales_f16, const uint8_t *zeros,
                              int K, int N, int bits, int group,
                              void *packed, size_t packed_bytes, tman_stream_t stream)
{
    if (!codes || !scales_f16 || !zeros || !packed) return TMAN_ERR_NULL;
    tman_status st = check_format(K, N, bits, group);
    if (st != TMAN_OK) return st;
    if (packed_bytes < make_layout(K, N, bits, group).total) return TMAN_ERR_BUFFER_TOO_SMALL;
    if (!aligned_to(packed, 256)) return TMAN_ERR_SHAPE;
    return launch_pack(codes, scales_f16, zeros, K, N, bits, group, packed, reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_unpack_weights(const void *packed, size_t packed_bytes,
                                int K, int N, int bits, int group,
                                uint8_t *codes, void *scales_f16, uint8_t *zeros,
                                void *workspace, size_t ws_bytes, tman_stream_t stream)
{
    if (!codes || !scales_f16 || !zeros || !packed || !workspace) return TMAN_ERR_NULL;
    tman_status st = check_format(K, N, bits, group);
    if (st != TMAN_OK) return st;
    if (packed_bytes < make_layout(K, N, bits, group).total) return TMAN_ERR_BUFFER_TOO_SMALL;
    if (ws_bytes < kWsStatusBytes) return TMAN_ERR_BUFFER_TOO_SMALL;
    if (!buffers_aligned(packed, workspace)) return TMAN_ERR_SHAPE;
    return launch_unpack(packed, K, N, bits, group, codes, scales_f16, zeros,
                         static_cast<uint32_t *>(workspace), reinterpret_cast<cudaStream_t>(stream));
}

static tman_status check_matmul(const void *packed, size_t packed_bytes, const void *x, void *y, int M, int K,
                                int N, int bits, int group, void *ws)
{
    if (!packed || !x || !y || !ws) return TMAN_ERR_NULL;
    tman_status st = check_format(K, N, bits, group);
    if (st != TMAN_OK) return st;
    if (packed_bytes < make_layout(K, N, bits, group).total) return TMAN_ERR_BUFFER_TOO_SMALL;
    if (bits < 2) return TMAN_ERR_UNSUPPORTED;
    if (M < 1) return TMAN_ERR_SHAPE;
    if (!buffers_aligned(packed, ws) || !matrices_aligned(x, y)) return TMAN_ERR_SHAPE;
    return TMAN_OK;
}

tman_status tman_mpgemv(const void *packed, size_t packed_bytes, const void *x_f16, void *y_f16,
                        int M, int K, int N, int bits, int group,
                        void *workspace, size_t ws_bytes, tman_stream_t stream)
{
    tman_status st = check_matmul(packed, packed_bytes, x_f16, y_f16, M, K, N, bits, group, workspace);
    if (st != TMAN_OK) return st;
    if (M > 8) return TMAN_ERR_SHAPE;
    if (ws_bytes < mpgemv_workspace_bytes(1, K, N, bits)) return TMAN_ERR_BUFFER_TOO_SMALL;
    return launch_mpgemv(packed, x_f16, y_f16, M, K, N, bits, group, workspace, ws_bytes,
                         reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_mpgemv_grouped(int count, const void *const *packed, const size_t *packed_bytes,
                                const void *x_f16, void *const *y_f16, int M, int K, const int *N,
                                int bits, int group, void *workspace, size_t ws_bytes, tman_stream_t stream)
{
    if (!packed || !packed_bytes || !y_f16 || !N) return TMAN_ERR_NULL;
    if (count < 1 || count > 4) return TMAN_ERR_SHAPE;
    long long ntot = 0;
    for (int g = 0; g < count; ++g) {
        tman_status st = check_matmul(packed[g], packed_bytes[g], x_f16, y_f16[g], M, K, N[g], bits, group, workspace);
        if (st != TMAN_OK) return st;
        ntot += N[g];
    }
    if (M > 8 || ntot > (1 << 30)) return TMAN_ERR_SHAPE;
    if (ws_bytes < mpgemv_workspace_bytes(1, K, (int)ntot, bits)) return TMAN_ERR_BUFFER_TOO_SMALL;
    return launch_mpgemv_grouped(count, packed, x_f16, y_f16, M, K, N, bits, group, workspace, ws_bytes,
                                 reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_quantize_rows(const void *x_f16, int M, int K, int qmax, int16_t *a_i16, float *row_scale,
                               tman_stream_t stream)
{
    if (!x_f16 || !a_i16 || !row_scale) return TMAN_ERR_NULL;
    if (M < 1 || K < 1 || (qmax != 32767 && qmax != 127)) return TMAN_ERR_SHAPE;
    if (!matrices_aligned(x_f16, a_i16)) return TMAN_ERR_SHAPE;
    return launch_quantize_rows(x_f16, M, K, qmax, a_i16, row_scale, reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_mpgemv_ternary(const void *packed, size_t packed_bytes, const int16_t *a_i16, const float *row_scale,
                                float w_scale, void *y_f16, int32_t *acc_i32, int M, int K, int N, int group,
                                void *workspace, size_t ws_bytes, tman_stream_t stream)
{
    tman_status st = check_matmul(packed, packed_bytes, a_i16, y_f16, M, K, N, 2, group, workspace);
    if (st != TMAN_OK) return st;
    if (!row_scale) return TMAN_ERR_NULL;
    if (M > 8) return TMAN_ERR_SHAPE;
    if (K > 16384) return TMAN_ERR_UNSUPPORTED;            // 3 * K * 32767 must stay below the "no sum pending" pattern
    if (acc_i32 && !aligned_to(acc_i32, 16)) return TMAN_ERR_SHAPE;
    if (ws_bytes < mpgemv_ternary_workspace_bytes(M, K, N)) return TMAN_ERR_BUFFER_TOO_SMALL;
    return launch_mpgemv_ternary(packed, a_i16, row_scale, w_scale, y_f16, acc_i32, M, K, N, group, workspace, ws_bytes,
                                 reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_quantize_rows_i8(const void *x_f16, int M, int K, int8_t *a_i8, float *row_scale, tman_stream_t stream)
{
    if (!x_f16 || !a_i8 || !row_scale) return TMAN_ERR_NULL;
    if (M < 1 || K < 1) return TMAN_ERR_SHAPE;
    if (!matrices_aligned(x_f16, a_i8)) return TMAN_ERR_SHAPE;
    return launch_quantize_rows_i8(x_f16, M, K, a_i8, row_scale, reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_mpgemm_ternary_i8(const void *packed, size_t packed_bytes, const int8_t *a_i8, const float *row_scale,
                                   float w_scale, void *y_f16, int M, int K, int N, int group,
                                   void *workspace, size_t ws_bytes, tman_stream_t stream)
{
    tman_status st = check_matmul(packed, packed_bytes, a_i8, y_f16, M, K, N, 2, group, workspace);
    if (st != TMAN_OK) return st;
    if (!row_scale) return TMAN_ERR_NULL;
    if (K > (1 << 24)) return TMAN_ERR_UNSUPPORTED;             // K * 127 must fit the 32-bit accumulators
    if (ws_bytes < kWsStatusBytes) return TMAN_ERR_BUFFER_TOO_SMALL;
    return launch_mpgemm_ternary_i8(packed, a_i8, row_scale, w_scale, y_f16, M, K, N, group, workspace,
                                    reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_dequant_ternary_int8(const void *packed, size_t packed_bytes, int K, int N, int group, int8_t *w8_nk,
                                      void *workspace, size_t ws_bytes, tman_stream_t stream)
{
    if (!packed || !w8_nk || !workspace) return TMAN_ERR_NULL;
    tman_status st = check_format(K, N, 2, group);
    if (st != TMAN_OK) return st;
    if (packed_bytes < make_layout(K, N, 2, group).total) return TMAN_ERR_BUFFER_TOO_SMALL;
    if (ws_bytes < kWsStatusBytes) return TMAN_ERR_BUFFER_TOO_SMALL;
    if (!buffers_aligned(packed, workspace) || !aligned_to(w8_nk, 16)) return TMAN_ERR_SHAPE;
    return launch_dequant_ternary_int8(packed, K, N, group, w8_nk, static_cast<uint32_t *>(workspace),
                                       reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_mpgemm(const void *packed, size_t packed_bytes, const void *x_f16, void *y_f16,
                        int M, int K, int N, int bits, int group,
                        void *workspace, size_t ws_bytes, tman_stream_t stream)
{
    tman_status st = check_matmul(packed, packed_bytes, x_f16, y_f16, M, K, N, bits, group, workspace);
    if (st != TMAN_OK) return st;
    if (ws_bytes < mpgemm_workspace_bytes(M, K, N)) return TMAN_ERR_BUFFER_TOO_SMALL;
    return launch_mpgemm(packed, x_f16, y_f16, M, K, N, bits, group, workspace, ws_bytes,
                         reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_debug_mpgemm_variant(int variant, const void *packed, size_t packed_bytes, const void *x_f16, void *y_f16,
                                      int M, int K, int N, int bits, int group, const void *wt_f16,
                                      void *workspace, size_t ws_bytes, tman_stream_t stream)
{
    tman_status st = check_matmul(packed, packed_bytes, x_f16, y_f16, M, K, N, bits, group, workspace);
    if (st != TMAN_OK) return st;
    if (ws_bytes < mpgemm_workspace_bytes(M, K, N)) return TMAN_ERR_BUFFER_TOO_SMALL;
    return launch_mpgemm_variant(variant, packed, x_f16, y_f16, M, K, N, bits, group, wt_f16, workspace, ws_bytes,
                                 reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_debug_role_stamps(const void *workspace, size_t ws_bytes, int ctas, long long *out_host, tman_stream_t stream)
{
    if (!workspace || !out_host) return TMAN_ERR_NULL;
    if (!aligned_to(workspace, 256)) return TMAN_ERR_SHAPE;
    if (ws_bytes < mpgemm_workspace_bytes(1, 128, 8)) return TMAN_ERR_BUFFER_TOO_SMALL;
    return mpgemm_read_stamps(workspace, ctas, out_host, reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_debug_indices(const void *packed, int K, int N, int bits, int group,
                               uint8_t *idx, void *workspace, size_t ws_bytes, tman_stream_t stream)
{
    if (!packed || !idx || !workspace) return TMAN_ERR_NULL;
    tman_status st = check_format(K, N, bits, group);
    if (st != TMAN_OK) return st;
    if (ws_bytes < kWsStatusBytes) return TMAN_ERR_BUFFER_TOO_SMALL;
    if (!buffers_aligned(packed, workspace)) return TMAN_ERR_SHAPE;
    return launch_debug_indices(packed, K, N, bits, group, idx, static_cast<uint32_t *>(workspace),
                                reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_debug_luts(const void *x_f16, int M, int K, float *lut, tman_stream_t stream)
{
    if (!x_f16 || !lut) return TMAN_ERR_NULL;
    if (M < 1 || K < 4 || K % 4 != 0) return TMAN_ERR_SHAPE;
    return launch_debug_luts(x_f16, M, K, lut, reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_debug_gemm_plan(int M, int K, int N, int bits, int group, int *out8)
{
    if (!out8) return TMAN_ERR_NULL;
    tman_status st = check_format(K, N, bits, group);
    if (st != TMAN_OK) return st;
    if (M < 1) return TMAN_ERR_SHAPE;
    if (bits < 2) return TMAN_ERR_UNSUPPORTED;
    return mpgemm_plan(M, K, N, bits, out8);
}

tman_status tman_debug_gemm_plan_for(int M, int K, int N, int bits, int group, int sms, int resident, int *out8)
{
    if (!out8) return TMAN_ERR_NULL;
    tman_status st = check_format(K, N, bits, group);
    if (st != TMAN_OK) return st;
    if (M < 1 || sms < 1 || resident < 1) return TMAN_ERR_SHAPE;
    if (bits < 2) return TMAN_ERR_UNSUPPORTED;
    return mpgemm_plan_for(M, K, N, bits, sms, resident, out8);
}

tman_status tman_debug_gemv_plan(int M, int K, int N, int bits, int group, int sms, size_t ws_limit, int *out)
{
    if (!out) return TMAN_ERR_NULL;
    tman_status st = check_format(K, N, bits, group);
    if (st != TMAN_OK) return st;
    if (M < 1 || M > kGemvMaxRows || sms < 1) return TMAN_ERR_SHAPE;
    if (bits < 2) return TMAN_ERR_UNSUPPORTED;
    const GemvPlan g = plan_gemv(M, K, N, bits, sms, ws_limit ? ws_limit : (size_t)-1);
    for (int i = 0; i < 4 + 6 * kGemvMaxRows; ++i) out[i] = 0;
    out[0] = g.npass;
    out[1] = (int)((g.ws_bytes + 1023) / 1024);
    out[2] = (int)(g.cost_us * 1000.0 + 0.5);
    for (int i = 0; i < g.npass; ++i) {
        int *o = out + 4 + 6 * i;
        o[0] = g.pass[i].rows; o[1] = g.pass[i].variant_rows; o[2] = g.pass[i].words;
        o[3] = g.pass[i].nkappa; o[4] = g.pass[i].nkappa * g.pass[i].ctas_per_slice; o[5] = g.pass[i].smem_bytes;
    }
    return g.npass ? TMAN_OK : TMAN_ERR_UNSUPPORTED;
}

tman_status tman_debug_wait_timeout(void *workspace, size_t ws_bytes, unsigned int polls, tman_stream_t stream)
{
    if (!workspace) return TMAN_ERR_NULL;
    if (!aligned_to(workspace, 256)) return TMAN_ERR_SHAPE;
    if (polls < 1 || polls > (1u << 20)) return TMAN_ERR_SHAPE;
    return launch_wait_timeout(workspace, ws_bytes, polls, reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_debug_microbench(int kind, int arg, void *results, size_t results_bytes, void *buffer,
                                  size_t buffer_bytes, tman_stream_t stream)
{
    if (!results) return TMAN_ERR_NULL;
    if (results_bytes < 4096 || !buffers_aligned(results, buffer)) return TMAN_ERR_SHAPE;
    return launch_microbench(kind, arg, results, results_bytes, buffer, buffer_bytes, reinterpret_cast<cudaStream_t>(stream));
}

tman_status tman_debug_cluster_capacity(int threads, int smem_bytes, int cluster, int *out_clusters)
{
    if (!out_clusters) return TMAN_ERR_NULL;
    if (threads < 32 || threads > 1024 || smem_bytes < 0 || cluster < 1 || cluster > 16) return TMAN_ERR_SHAPE;
    *out_clusters = cluster_capacity(threads, smem_bytes, cluster);
    return TMAN_OK;
}

}  // extern "C"
