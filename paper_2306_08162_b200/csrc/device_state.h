// What the host side remembers between calls, all of it keyed by the ordinal of the CURRENT device: a process may drive
// several GPUs, and both the per-function shared-memory limit and the SM count belong to a device, not to the process.
#pragma once
#include <cuda_runtime.h>

#include <mutex>

namespace qlora {

constexpr int kMaxDevices = 64;

inline int device_ordinal() {
    int dev = 0;
    return (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) ? dev : -1;
}

// One per kernel instantiation (a function-local static): on which devices the kernel's dynamic shared-memory limit has
// been raised, and to how much.  cudaFuncSetAttribute applies to the current device only.
struct SmemLimit {
    std::mutex mu;
    size_t done[kMaxDevices] = {};
    template <typename Kern>
    bool raise(Kern kern, size_t bytes) {
        const int dev = device_ordinal();
        std::lock_guard<std::mutex> lock(mu);
        if (dev >= 0 && done[dev] >= bytes) return true;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return false;
        if (dev >= 0) done[dev] = bytes;
        return true;
    }
};

// Streaming multiprocessors of the current device.
inline int sm_count() {
    static std::mutex mu;
    static int cached[kMaxDevices] = {};
    const int dev = device_ordinal();
    std::lock_guard<std::mutex> lock(mu);
    if (dev >= 0 && cached[dev] > 0) return cached[dev];
    int v = 0;
    if (dev < 0 || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
    cached[dev] = v;
    return v;
}

}  // namespace qlora
