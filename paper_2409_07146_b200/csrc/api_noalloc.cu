// gsa_fwd_noalloc: the forward pass for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc (or any allocator) around the layer:
// code that runs inside an inference server's pre-sized memory plan, a real-time loop that
// must not take the allocator's lock or its implicit device synchronisation, a plug-in that
// only receives the framework's input and output buffers.  gsa_fwd needs scratch memory
// from its caller; this entry point brings its own: a fixed array that lives in the library
// image on every GPU that loads it.
#include <atomic>
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kScratchBytes = GSA_NOALLOC_MAX_WORKSPACE_BYTES;   // 32 MiB, held by every device that loads the library

// File-scope device array.  In host code this name is only a handle for the runtime, not a
// device address: the address is asked for once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_fwd_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
std::atomic<void*> g_scratch_ptr[kMaxDevices] = {};

// Address of the scratch array on the CURRENT device (looked up on the first call per device).
cudaError_t scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    void* p = g_scratch_ptr[dev].load(std::memory_order_acquire);      // steady state: no lock
    if (p == nullptr) {
        std::lock_guard<std::mutex> lock(g_mutex);
        p = g_scratch_ptr[dev].load(std::memory_order_relaxed);
        if (p == nullptr) {
            e = cudaGetSymbolAddress(&p, g_fwd_scratch);
            if (e != cudaSuccess) return e;
            g_scratch_ptr[dev].store(p, std::memory_order_release);
        }
    }
    *out = p;
    return cudaSuccess;
}

}  // namespace

extern "C" GSA_API gsa_status_t gsa_fwd_noalloc(const gsa_params_t* params, const void* q, const void* k,
                                                const void* v, const float* gate, const float* K0,
                                                const float* V0, void* o, float* ok_save, float* KT,
                                                float* VT, void* stream, int32_t* dev_status) {
    const size_t need = gsa_workspace_bytes(params, GSA_WS_FWD);
    if (need == 0) {
        // invalid or unsupported params: let the regular entry point name the error
        return gsa_fwd(params, q, k, v, gate, K0, V0, o, ok_save, KT, VT, nullptr, 0, stream, dev_status);
    }
    if (need > kScratchBytes) return GSA_ERR_WORKSPACE;    // shape too large for the built-in scratch
    void* scratch = nullptr;
    if (scratch_address(&scratch) != cudaSuccess) return GSA_ERR_CUDA;
    // Nothing in the scratch has to start at zero: the forward writes every scratch tensor
    // (G, 1-a, partial logits, logits, p) in full before it reads it.
    return gsa_fwd(params, q, k, v, gate, K0, V0, o, ok_save, KT, VT, scratch, kScratchBytes, stream, dev_status);
}
