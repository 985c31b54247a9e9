// "Done once per device" bookkeeping for settings that CUDA keeps per device, such as a kernel's
// opt-in to more than 48 KB of dynamic shared memory (cudaFuncSetAttribute acts on the current
// device only).  Plain C++, no CUDA types, so that it can be exercised without a GPU.
#pragma once

#include <atomic>

namespace kge {

constexpr int kMaxDevices = 64;

// One flag per device ordinal.  run(dev, f) calls f() unless an earlier call for the same ordinal
// succeeded (f returns 0 on success, as cudaError_t does), and returns f's code.  Ordinals outside
// the table are never remembered: f runs every time.  f must be idempotent: two threads that race
// on a device's first use may both run it.
struct DeviceOnce {
    std::atomic<bool> done[kMaxDevices];
    DeviceOnce() { for (auto& d : done) d.store(false, std::memory_order_relaxed); }
    template <class F>
    int run(int dev, F&& f) {
        const bool tracked = dev >= 0 && dev < kMaxDevices;
        if (tracked && done[dev].load(std::memory_order_acquire)) return 0;
        const int rc = (int)f();
        if (rc == 0 && tracked) done[dev].store(true, std::memory_order_release);
        return rc;
    }
};

}  // namespace kge
