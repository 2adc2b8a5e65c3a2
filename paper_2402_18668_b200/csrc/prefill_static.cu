// based_prefill_static_scratch: based_prefill for callers that cannot hand the library
// any scratch memory.  The segment-state scratch that based_prefill takes as `workspace`
// lives here in a fixed array in device memory that is part of the library image.
#include <cstdio>
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kScratchBytes = BASED_STATIC_SCRATCH_BYTES;

// One instance per GPU that loads the library, resident until the process exits.
// In host code this name is only a handle for cudaGetSymbolAddress, not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the array on the current device, resolved once per device.
based_status scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BASED_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_addr[dev] == nullptr) {
        void* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || ptr == nullptr) {
            std::fprintf(stderr, "libbased: cudaGetSymbolAddress(static scratch) failed: %s\n", cudaGetErrorString(e));
            return BASED_ERR_CUDA;
        }
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return BASED_OK;
}

}  // namespace

extern "C" size_t based_static_scratch_bytes(void) { return kScratchBytes; }

extern "C" based_status based_prefill_static_scratch(const void* q, const void* k, const void* v, void* out,
                                                     float* kv_state, float* z_state, int B, int H, int L,
                                                     int d_feat, int d_v, based_dtype io, int flags,
                                                     void* cuda_stream) {
    // What the fastest plan would need; with less, the call takes the fastest plan that fits the array (fewer segments
    // per head, in the end the plain chunk loop or the recompute mode, which need no scratch).
    const size_t need = based_prefill_workspace_bytes(B, H, L, d_feat, d_v, io);
    void* scratch = nullptr;
    if (need > 0) {
        const based_status st = scratch_address(&scratch);
        if (st != BASED_OK) return st;
    }
    // Every scratch slot the main pass reads is first written by the segment-state pass of the
    // same call, so nothing has to be cleared between calls.
    return based::prefill_fit_workspace(q, k, v, out, kv_state, z_state, B, H, L, d_feat, d_v, io, flags, scratch,
                                        kScratchBytes, cuda_stream);
}
