// int8_linear_fused_static: the fused W8A8 linear for callers that must not allocate device memory.
//
// Some callers cannot hand this library a workspace because they cannot get one: an inference server that
// gave all of HBM to its own arena at start-up (a later cudaMalloc fails or fragments it), a real-time loop
// where an allocation's implicit device synchronisation is not acceptable, or a plug-in that is only ever
// given its input and output tensors. For them the scratch the from-bf16 path needs (status word, per-token
// scales, int8 activations) lives in a fixed array inside the library's own device image. The price: every GPU that loads the library holds kStaticWorkspaceBytes until the process exits,
// problems whose scratch does not fit are refused, and all calls share the one array.
#include "../../include/w8a8_linear.h"

#include <cuda_runtime.h>

#include <mutex>

namespace {

constexpr size_t kStaticWorkspaceBytes = W8A8_STATIC_WORKSPACE_BYTES;
constexpr int kMaxDevices = 64;

// The scratch itself. In host code this name is only a handle for the runtime, not a device address:
// the address a kernel can use comes from cudaGetSymbolAddress, per device.
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

std::mutex g_mutex;
void* g_device_ptr[kMaxDevices] = {};      // resolved address of g_static_workspace on each device

// Looks up (once per device, with that device current) where the array lives on the current device.
int static_workspace(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return W8A8_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return W8A8_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_device_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || p == nullptr) return W8A8_ERR_CUDA;
        g_device_ptr[dev] = p;
    }
    *out = g_device_ptr[dev];
    return W8A8_OK;
}

} // namespace

extern "C" int int8_linear_fused_static(const void* A_bf16, int64_t lda,
                                        const int8_t* qw, const float* s_ch, const float* bias,
                                        void* out_bf16, int64_t ldo, int64_t M, int64_t N, int64_t K,
                                        int sync_and_check, void* stream) {
    // size check first: it needs no device and gives the caller a clear answer
    const size_t need = int8_linear_workspace_min_bytes(M, N, K, W8A8_ACT_BF16);
    if (need == 0) return W8A8_ERR_INVALID_ARG;
    if (need > kStaticWorkspaceBytes) return W8A8_ERR_WORKSPACE;

    void* ws = nullptr;
    if (int e = static_workspace(&ws)) return e;
    // Same kernels as int8_linear_fused, with the built-in array as their scratch. Nothing in it has to be
    // zero on entry: the call clears the status word itself and writes every scale and code before reading
    // it, so whatever the previous call left behind is harmless.
    int e = int8_linear_fused(A_bf16, W8A8_ACT_BF16, lda, nullptr, qw, s_ch, bias, out_bf16, ldo, M, N, K,
                              ws, kStaticWorkspaceBytes, stream);
    if (e != W8A8_OK || !sync_and_check) return e;
    return int8_check_status(ws, stream);
}
