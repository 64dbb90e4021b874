// rlcs_gae_no_alloc: GAE for callers that cannot allocate device memory.
//
// The inter-block carry of the scan kernels needs a small scratch area (tile records plus a
// 256-byte header).  The regular entry points take it from a caller-provided workspace; this one
// keeps it in a fixed device array that is part of the library image, so the caller passes inputs
// and outputs only and nothing -- no cudaMalloc, cudaFree or allocating library routine -- is
// called on the way.
#include <cstdint>
#include <mutex>

#include "../../include/rlcs.h"

namespace {

// Scratch shared by every rlcs_gae_no_alloc call of the process on a device (each GPU that loads
// the library holds its own copy until exit).  1 MiB: 256 bytes of header + 65520 tile records.
constexpr size_t kScratchBytes = size_t(1) << 20;
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};     // device address of g_scratch, per device, once known
std::mutex g_setup_lock;                   // two host threads making a device's first call: one sets up

// In host code `g_scratch` is only a handle for the runtime, not a device address: handing it to a
// kernel would make the kernel fault or scribble over unrelated memory.  The device address comes
// from cudaGetSymbolAddress, asked once per device with that device current.
// `set_up`: bring the array into the state rlcs_workspace_init gives a workspace on first use.
// That set-up is two memsets that must really run: during a stream capture they would only be
// recorded, so a device's first call is refused while `stream` is capturing.
int scratch_for_current_device(void** out, void* stream, bool set_up) {
    int dev = 0;
    *out = nullptr;
    if (cudaGetDevice(&dev) != cudaSuccess) return RLCS_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return RLCS_ERR_CUDA;
    std::lock_guard<std::mutex> hold(g_setup_lock);
    if (g_scratch_ptr[dev] == nullptr) {
        if (!set_up) return RLCS_OK;           // never used on this device: nothing to report
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(static_cast<cudaStream_t>(stream), &cap) != cudaSuccess) return RLCS_ERR_CUDA;
        if (cap != cudaStreamCaptureStatusNone) return RLCS_ERR_CAPTURE;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_scratch) != cudaSuccess || ptr == nullptr) return RLCS_ERR_CUDA;
        const int st = rlcs_workspace_init(ptr, kScratchBytes, stream);
        if (st != RLCS_OK) return st;
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return RLCS_OK;
}

bool aligned_to(const void* p, uintptr_t a) { return p == nullptr || (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace

extern "C" {

size_t rlcs_no_alloc_scratch_bytes(void) { return kScratchBytes; }

int rlcs_gae_no_alloc(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                      const float* trunc_bootstrap, const float* bootstrap, float* advantages, float* returns,
                      int64_t N, int64_t T, float gamma, float lambda, void* cuda_stream) {
    // Reject what the fixed array cannot serve before touching the device: the bytes of carry
    // scratch this very call would use (none when no row straddles a tile, or when the rows'
    // tiles form thread-block clusters).
    const bool vec = aligned_to(rewards, 32) && aligned_to(values, 32) && aligned_to(advantages, 32) && aligned_to(returns, 32) &&
                     aligned_to(trunc_bootstrap, 32) && aligned_to(bootstrap, 32) && aligned_to(dones, 16) && aligned_to(truncs, 16);
    if (rlcs_gae_carry_bytes(N, T, truncs != nullptr, vec) > kScratchBytes) return RLCS_ERR_LIMIT;
    void* scratch = nullptr;
    int st = scratch_for_current_device(&scratch, cuda_stream, true);
    if (st != RLCS_OK) return st;
    // The array keeps whatever the previous call left.  Tile records need no clearing: a call tags
    // its records with the call counter, which the last block of every completed call advances.
    // The finished-block counter (second header word) must start at zero even if an earlier launch
    // was refused half way.  The status word after it is left alone: it holds RLCS_ERR_TIMEOUT from
    // an earlier call until rlcs_no_alloc_last_device_status reads and clears it.
    if (cudaMemsetAsync(static_cast<unsigned char*>(scratch) + 4, 0, 4, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return RLCS_ERR_CUDA;
    st = rlcs_gae(rewards, values, dones, truncs, trunc_bootstrap, bootstrap, advantages, returns, N, T, gamma,
                  lambda, scratch, kScratchBytes, cuda_stream);
    return st == RLCS_ERR_WORKSPACE ? RLCS_ERR_LIMIT : st;
}

int rlcs_no_alloc_last_device_status(void* cuda_stream) {
    void* scratch = nullptr;
    const int st = scratch_for_current_device(&scratch, cuda_stream, false);
    if (st != RLCS_OK || scratch == nullptr) return st;
    return rlcs_last_device_status(scratch, cuda_stream);
}

}  // extern "C"
