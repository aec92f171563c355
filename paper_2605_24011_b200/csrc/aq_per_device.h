// Per-device bookkeeping for set-up that CUDA keeps per device, not per process:
// a kernel's dynamic-shared-memory attribute, a device's SM count, the address of
// a __device__ symbol.  Plain host C++ (no CUDA headers), so it can be unit-tested
// without a GPU.
#pragma once
#include <mutex>

namespace aq {

constexpr int AQ_MAX_DEVICES = 64;

// Runs a set-up function once for every device index it is asked about.
// A set-up that fails is not recorded: the next call on that device tries again.
class PerDeviceOnce {
public:
    // fn() returns 0 on success.  Returns fn's code, 0 when the device is already set up,
    // or -1 when dev is outside [0, AQ_MAX_DEVICES).
    template <typename Fn>
    int run(int dev, Fn fn) {
        if (dev < 0 || dev >= AQ_MAX_DEVICES) return -1;
        std::lock_guard<std::mutex> lock(mu_);
        if (done_[dev]) return 0;
        const int rc = fn();
        if (rc == 0) done_[dev] = true;
        return rc;
    }
    bool is_done(int dev) const { return dev >= 0 && dev < AQ_MAX_DEVICES && done_[dev]; }

private:
    std::mutex mu_;
    bool done_[AQ_MAX_DEVICES] = {};
};

// One cached value per device, filled on first use by fn(dev, &value) (0 = success).
template <typename T>
class PerDeviceValue {
public:
    template <typename Fn>
    int get(int dev, T* out, Fn fn) {
        if (dev < 0 || dev >= AQ_MAX_DEVICES) return -1;
        std::lock_guard<std::mutex> lock(mu_);
        if (!have_[dev]) {
            T v{};
            const int rc = fn(dev, &v);
            if (rc != 0) return rc;
            val_[dev] = v;
            have_[dev] = true;
        }
        *out = val_[dev];
        return 0;
    }

private:
    std::mutex mu_;
    bool have_[AQ_MAX_DEVICES] = {};
    T val_[AQ_MAX_DEVICES] = {};
};

}  // namespace aq
