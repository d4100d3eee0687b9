// Per-device facts the launch code caches: the SM count, and "this kernel's attribute has been set on
// this device" flags.  All of it is safe to use from several host threads on several devices: the
// cached values are idempotent and held in atomics indexed by device.
#pragma once
#include <cuda_runtime.h>

#include <atomic>

namespace gf {

constexpr int MAX_DEVICES = 64;

// Index of the current device, or -1 if it cannot be had or is beyond MAX_DEVICES.
inline int current_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return -1;
    return dev;
}

// Number of SMs of the current device (0 on failure).
inline int sm_count()
{
    static std::atomic<int> cached[MAX_DEVICES];          // zero-initialised: 0 = not asked yet
    const int dev = current_device();
    if (dev < 0) return 0;
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

// One flag per device, for work that has to happen once per device and may harmlessly happen twice
// (cudaFuncSetAttribute of a kernel).
struct PerDeviceFlag {
    std::atomic<bool> done[MAX_DEVICES];
    bool is_set(int dev) const { return done[dev].load(std::memory_order_acquire); }
    void set(int dev) { done[dev].store(true, std::memory_order_release); }
};

}  // namespace gf
