// "Done once per device" flags for state the CUDA runtime keeps per device (a kernel's opt-in to
// large dynamic shared memory, the address of a __device__ symbol).  Plain C++, no CUDA types,
// so that host-only tests can include it.
#pragma once
#include <atomic>

namespace moe {

constexpr int MAX_DEVICE_ORDINALS = 64;

struct DeviceOnce {
    std::atomic<bool> flag[MAX_DEVICE_ORDINALS];
    DeviceOnce()
    {
        for (auto &f : flag)
            f.store(false);
    }
    // ordinals outside the table are never "done": their set-up simply repeats
    bool done(int device) const
    {
        return device >= 0 && device < MAX_DEVICE_ORDINALS && flag[device].load(std::memory_order_acquire);
    }
    void mark(int device)
    {
        if (device >= 0 && device < MAX_DEVICE_ORDINALS)
            flag[device].store(true, std::memory_order_release);
    }
};

}  // namespace moe
