// Per-device set-up state of the launchers: the SM count of each device and "this kernel's
// shared-memory limit has been raised on this device" flags.  One mutex guards all of it, so the
// entry points may be called from several host threads and for several devices of one process.
// Internal to the library.
#pragma once

#include <cuda_runtime.h>

#include <mutex>

namespace bt {

constexpr int kMaxDevices = 64;

inline std::mutex& setup_mutex()
{
    static std::mutex m;
    return m;
}

// The current device and its SM count (looked up once per device).
inline cudaError_t current_device(int* dev_out, int* sm_count_out)
{
    static int sm_count[kMaxDevices];  // 0 = not looked up yet
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(setup_mutex());
    if (!sm_count[dev]) {
        int n = 0;
        e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        sm_count[dev] = n > 0 ? n : 1;
    }
    *dev_out = dev;
    *sm_count_out = sm_count[dev];
    return cudaSuccess;
}

// One flag per device; `once(dev, f)` runs f() (a cudaError_t-returning set-up step) the first time
// it is called for a device and remembers a success.
struct PerDeviceOnce {
    bool done[kMaxDevices] = {};
    template <class F>
    cudaError_t once(int dev, F&& f)
    {
        std::lock_guard<std::mutex> lock(setup_mutex());
        if (done[dev]) return cudaSuccess;
        cudaError_t e = f();
        if (e == cudaSuccess) done[dev] = true;
        return e;
    }
};

// Raises a kernel's dynamic shared-memory limit once per device.
template <class Kernel>
inline cudaError_t raise_smem_limit_once(PerDeviceOnce& flag, int dev, Kernel kernel, int bytes)
{
    return flag.once(dev, [&]() { return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes); });
}

}  // namespace bt
