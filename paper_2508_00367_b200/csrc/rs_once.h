// Once-per-device set-up guard.  A kernel attribute set with cudaFuncSetAttribute belongs to the
// device that is current at the call, so "done" has to be remembered per device, not per process,
// and launches may come from several host threads.  No CUDA dependency: `setup` is any callable
// returning 0 on success; a failed set-up is not remembered and is tried again by the next call.
#pragma once
#include <mutex>

namespace rs {

class PerDeviceOnce {
public:
    static constexpr int kMaxDevices = 64;
    // Runs setup() if it has not yet succeeded for `device`; returns its code (0 when already done).
    // A device index outside [0, kMaxDevices) is never cached: setup runs on every call.
    template <typename F> int run(int device, F&& setup) {
        std::lock_guard<std::mutex> lock(mu_);
        const bool cached = device >= 0 && device < kMaxDevices;
        if (cached && done_[device]) return 0;
        const int rc = setup();
        if (rc == 0 && cached) done_[device] = true;
        return rc;
    }
    bool done(int device) {
        std::lock_guard<std::mutex> lock(mu_);
        return device >= 0 && device < kMaxDevices && done_[device];
    }

private:
    std::mutex mu_;
    bool done_[kMaxDevices] = {};
};

}  // namespace rs
