// Limits of the current device that the host-side planners size their grids and shared-memory
// rings by: number of SMs, and shared memory one thread block may use (each resident block also
// costs 1 KB of the SM's total).  Queried once per device; without a device (size queries made on a
// machine that has none) the figures of the B200 this library targets are returned.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>

namespace rlcs_device {

struct Limits {
    long long sms;           // multiprocessors
    size_t smem_per_sm;      // bytes of shared memory usable by the thread blocks of one SM
};

inline Limits limits() {
    constexpr Limits kB200 = {148, 227 * 1024};
    constexpr int kMaxDevices = 64;
    static Limits cache[kMaxDevices];
    static bool known[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();        // no device: not an error for a size query
        return kB200;
    }
    if (!known[dev]) {
        int sms = 0, smem = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess || sms < 1 || smem < 48 * 1024) {
            (void)cudaGetLastError();
            return kB200;
        }
        cache[dev] = Limits{sms, (size_t)smem};
        known[dev] = true;
    }
    return cache[dev];
}

}  // namespace rlcs_device
