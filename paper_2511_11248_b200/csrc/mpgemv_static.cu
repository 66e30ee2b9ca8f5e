// tman_mpgemv_static: the decode matmul for callers that cannot hand the library a workspace.
//
// Some hosts of this library may not allocate device memory at the point where they call a
// matmul: an inference runtime that sizes one arena at start-up and forbids cudaMalloc afterwards
// (an allocation can synchronise the device and breaks a latency budget), a plug-in that runs inside
// another framework's stream callback, code between "begin" and "end" of a region where the
// allocator is locked.  tman_mpgemv needs scratch memory (a status word and the fp32
// partial sums of the K-slices) that such a caller has nowhere to put.  Here that
// scratch is a fixed array that is part of the library image: every GPU that loads the library
// holds kStaticWsBytes of it from load until the process exits, and nothing is allocated at
// call time.
#include "common.cuh"

#include <mutex>

namespace tman {
namespace {

constexpr size_t kStaticWsBytes = 4u << 20;          // 4 MiB per GPU
constexpr int    kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress: it is
// not a device address and must never be passed to a kernel.
static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

std::mutex g_lock;
void      *g_ws_addr[kMaxDevices];                   // device address of g_static_ws, per device
bool       g_ws_ready[kMaxDevices];

// Device address of the array on the current device, looked up once per device.
tman_status static_ws(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TMAN_ERR_CUDA;
    std::lock_guard<std::mutex> guard(g_lock);
    if (!g_ws_ready[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_ws) != cudaSuccess || ptr == nullptr) return TMAN_ERR_CUDA;
        g_ws_addr[dev] = ptr;
        g_ws_ready[dev] = true;
    }
    *out = g_ws_addr[dev];
    return TMAN_OK;
}

}  // namespace
}  // namespace tman

using namespace tman;

extern "C" tman_status tman_mpgemv_static(const void *packed, size_t packed_bytes, const void *x_f16,
                                          void *y_f16, int M, int K, int N, int bits, int group,
                                          unsigned int *status_dev, tman_stream_t stream)
{
    if (!packed || !x_f16 || !y_f16) return TMAN_ERR_NULL;
    tman_status st = check_format(K, N, bits, group);
    if (st != TMAN_OK) return st;
    if (packed_bytes < make_layout(K, N, bits, group).total) return TMAN_ERR_BUFFER_TOO_SMALL;
    if (bits < 2) return TMAN_ERR_UNSUPPORTED;
    if (M < 1 || M > 8) return TMAN_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(packed) & 255) || (reinterpret_cast<uintptr_t>(x_f16) & 15) ||
        (reinterpret_cast<uintptr_t>(y_f16) & 15))
        return TMAN_ERR_SHAPE;
    // the fixed array is the whole budget: a shape whose scratch does not fit is refused
    const size_t need = mpgemv_workspace_bytes(M, K, N, bits);
    if (need > kStaticWsBytes) return TMAN_ERR_BUFFER_TOO_SMALL;

    void *ws = nullptr;
    st = static_ws(&ws);
    if (st != TMAN_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // The array keeps whatever the last call left.  The status word must start at zero and the
    // partial-sum area must say "no sum pending" everywhere this call will look.
    st = launch_workspace_init(ws, need, s);
    if (st != TMAN_OK) return st;
    st = launch_mpgemv(packed, x_f16, y_f16, M, K, N, bits, group, ws, kStaticWsBytes, s);
    if (st != TMAN_OK) return st;
    if (status_dev &&
        cudaMemcpyAsync(status_dev, ws, sizeof(unsigned int), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return TMAN_ERR_CUDA;
    return TMAN_OK;
}
