// dirotq_linear for callers that cannot allocate device memory.
//
// Some callers hold no allocator at the point where they need a layer evaluated: a plug-in that
// is handed input and output buffers by a serving runtime which owns all device memory, code
// that runs on a stream whose owner forbids cudaMalloc/cudaFree (they synchronise the device and
// fail inside a stream capture), or a fixed-memory real-time loop.  dirotq_linear needs a
// workspace (activation codes, scales and the bf16 rank-r coefficients travel through it from
// the first kernel to the second); here that workspace is a fixed array that lives in the
// library's own device image, so nothing is ever allocated.  The price: the array is resident on
// every GPU that loads the library until the process exits, its size caps the problem, and all
// calls share it.
#include "common.h"

#include <atomic>
#include <stdio.h>

namespace dirotq {
namespace {

// 16 MiB + 1 KiB of slack so that a 1024-byte aligned window of 16 MiB always fits.
constexpr size_t kStaticWorkspaceBytes = 16u << 20;
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes + 1024];

struct PerDevice {
    std::atomic<bool> ready;   // set (release) after `base` is written, read (acquire) before it is used
    std::atomic<char*> base;   // DEVICE address of the aligned window
};
PerDevice g_dev[64];

// In host code `g_static_workspace` names a host-side shadow of the symbol, not device memory: the
// device address has to be asked for, once per device, with that device current.
dirotq_status_t static_workspace(int device, char** out) {
    if (device < 0 || device >= 64) return DIROTQ_ERR_INVALID_ARG;
    if (!g_dev[device].ready.load(std::memory_order_acquire)) {
        // two threads racing here both ask and both get the same address
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_static_workspace);
        if (e != cudaSuccess || p == nullptr) return DIROTQ_ERR_CUDA;
        const uintptr_t a = (reinterpret_cast<uintptr_t>(p) + 1023u) & ~static_cast<uintptr_t>(1023u);
        g_dev[device].base.store(reinterpret_cast<char*>(a), std::memory_order_relaxed);
        g_dev[device].ready.store(true, std::memory_order_release);
    }
    *out = g_dev[device].base.load(std::memory_order_relaxed);
    return DIROTQ_OK;
}

}  // namespace
}  // namespace dirotq

using namespace dirotq;

extern "C" dirotq_status_t dirotq_linear_noalloc(const void* x, int M, const dirotq_layer_t* layer, void* y,
                                                 int* device_status, dirotq_stream_t stream) {
    if (layer == nullptr || layer->magic != kLayerMagic || x == nullptr || y == nullptr || M < 1 || layer->geo.no_rot)
        return DIROTQ_ERR_INVALID_ARG;
    size_t need = 0;
    dirotq_status_t st = dirotq_workspace_bytes(layer, M, &need);
    if (st != DIROTQ_OK) return st;
    if (need > kStaticWorkspaceBytes) {
        fprintf(stderr,
                "dirotq_linear_noalloc: this call needs a %zu-byte workspace but the built-in one holds %zu bytes "
                "(M = %d, K = %d); use dirotq_linear with a caller-allocated workspace\n",
                need, kStaticWorkspaceBytes, M, layer->geo.K);
        return DIROTQ_ERR_BUFFER_TOO_SMALL;
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DIROTQ_ERR_CUDA;
    if (dev != layer->device) return DIROTQ_ERR_INVALID_ARG;
    char* ws = nullptr;
    st = static_workspace(dev, &ws);
    if (st != DIROTQ_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the array keeps what the previous call left: the status word must start at zero
    if (cudaMemsetAsync(ws, 0, 256, s) != cudaSuccess) return DIROTQ_ERR_CUDA;
    st = dirotq_linear(x, M, layer, y, ws, need, stream);
    if (st != DIROTQ_OK) return st;
    if (device_status != nullptr &&
        cudaMemcpyAsync(device_status, ws, sizeof(int), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return DIROTQ_ERR_CUDA;
    return DIROTQ_OK;
}
