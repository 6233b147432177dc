// Host-side state that exists once per CUDA device rather than once per process: the multiprocessor count and
// the "already configured on this device" marks of kernels that need an attribute (opt-in shared memory) or an
// occupancy query before their first launch.  cudaFuncSetAttribute applies to the current device only, so a
// process that creates caches on two devices has to configure every kernel on each of them.
#pragma once
#include <atomic>

constexpr int XSV_MAX_DEVICES = 64;

// One slot per device; a slot holds an int that is 0 until set.  Devices beyond the table share the last slot's
// index space by never being cached (get() returns 0 for them, so the caller configures every time).
class XsvPerDeviceInt {
public:
    int get(int device) const { return in_range(device) ? v_[device].load(std::memory_order_acquire) : 0; }
    void set(int device, int value) {
        if (in_range(device)) v_[device].store(value, std::memory_order_release);
    }
    static bool in_range(int device) { return device >= 0 && device < XSV_MAX_DEVICES; }

private:
    std::atomic<int> v_[XSV_MAX_DEVICES] = {};
};

// The device the calling thread has current (-1 if the runtime cannot tell).
int xsv_current_device();
