// rlcs_gae_no_alloc: GAE for callers that cannot allocate device memory.
//
// The inter-block carry of the scan kernels needs a small scratch area (tile records plus a
// 256-byte header).  The regular entry points take it from a caller-provided workspace; this one
// keeps it in a fixed device array that is part of the library image, so the caller passes inputs
// and outputs only and nothing -- no cudaMalloc, cudaFree or allocating library routine -- is
// called on the way.
#include <cstdint>

#include "../../include/rlcs.h"

namespace {

// Scratch shared by every rlcs_gae_no_alloc call of the process on a device (each GPU that loads
// the library holds its own copy until exit).  1 MiB: 256 bytes of header + 65520 tile records.
constexpr size_t kScratchBytes = size_t(1) << 20;
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};     // device address of g_scratch, per device, once known

// In host code `g_scratch` is only a handle for the runtime, not a device address: handing it to a
// kernel would make the kernel fault or scribble over unrelated memory.  The device address comes
// from cudaGetSymbolAddress, asked once per device with that device current.
int scratch_for_current_device(void** out, void* stream) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RLCS_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return RLCS_ERR_CUDA;
    if (g_scratch_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_scratch) != cudaSuccess || ptr == nullptr) return RLCS_ERR_CUDA;
        // first use on this device: bring the array into the state rlcs_workspace_init gives a workspace
        const int st = rlcs_workspace_init(ptr, kScratchBytes, stream);
        if (st != RLCS_OK) return st;
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return RLCS_OK;
}

}  // namespace

extern "C" {

size_t rlcs_no_alloc_scratch_bytes(void) { return kScratchBytes; }

int rlcs_gae_no_alloc(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                      const float* trunc_bootstrap, const float* bootstrap, float* advantages, float* returns,
                      int64_t N, int64_t T, float gamma, float lambda, void* cuda_stream) {
    // Reject what the fixed array cannot serve before touching the device.
    if (rlcs_workspace_bytes(N, T) > kScratchBytes) return RLCS_ERR_LIMIT;
    void* scratch = nullptr;
    int st = scratch_for_current_device(&scratch, cuda_stream);
    if (st != RLCS_OK) return st;
    // The array keeps whatever the previous call left.  The tile records need no clearing (each
    // call tags its records with a fresh call number), but the finished-block counter and the
    // status word must start at zero even if an earlier call was cut short.
    if (cudaMemsetAsync(static_cast<unsigned char*>(scratch) + 4, 0, 8, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return RLCS_ERR_CUDA;
    return rlcs_gae(rewards, values, dones, truncs, trunc_bootstrap, bootstrap, advantages, returns, N, T, gamma,
                    lambda, scratch, kScratchBytes, cuda_stream);
}

}  // extern "C"
