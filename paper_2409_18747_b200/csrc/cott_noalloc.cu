// Forward pass for callers that cannot hand the library a workspace.
//
// Some users of this library have no way to obtain device scratch at call time: a serving
// process whose own memory pool already owns all of HBM, or a latency-critical loop that must
// not take the device-wide synchronisation that cudaMalloc / cudaFree imply.  For them the
// scratch of the forward pass (status word + per-group partial states) lives in a fixed array
// inside the library image itself.  Nothing is allocated or freed here or below this call.
#include <mutex>
#include "cott_internal.h"

namespace {

constexpr size_t kScratchBytes = 8u << 20;   // 8 MiB, resident on every GPU that loads the library

// Device memory that is part of the loaded module.  In host code this name is only a handle
// for the runtime (not a device address); kernels get the address cudaGetSymbolAddress returns.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_setup_mutex;

// Device address of the scratch array on the current device; resolved once per device, with
// that device current.
cudaError_t scratch_address(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" {

size_t cott_fwd_noalloc_max_bytes(void) { return kScratchBytes; }

cott_status cott_fwd_noalloc(const void* q, const void* k, const void* v, void* o, int B, int H,
                             int N, int d, int causal, cott_dtype dt, const cott_scale_params* sp,
                             void* stream) {
    const size_t need = cott_workspace_bytes(COTT_OP_FWD, dt, B, H, N, d, causal);
    if (need == (size_t)-1) return COTT_ERR_UNSUPPORTED;
    if (need > kScratchBytes) return COTT_ERR_WORKSPACE;   // problem too large for the built-in scratch
    void* ws = nullptr;
    if (scratch_address(&ws) != cudaSuccess) return COTT_ERR_CUDA;
    // Same kernels as cott_fwd; the status word is cleared on the stream at the start of the
    // call and every partial state is written before it is read, so what an earlier call left
    // in the array does not matter.
    return cott_fwd(q, k, v, o, nullptr, B, H, N, d, causal, dt, sp, ws, kScratchBytes, stream);
}

cott_status cott_fwd_noalloc_status(void* stream) {
    void* ws = nullptr;
    if (scratch_address(&ws) != cudaSuccess) return COTT_ERR_CUDA;
    return cott_last_async_status(ws, stream);
}

}  // extern "C"
