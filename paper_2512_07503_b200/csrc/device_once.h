// Per-device, thread-safe "done once" bookkeeping for settings that belong to a (device, kernel) pair,
// such as cudaFuncAttributeMaxDynamicSharedMemorySize, and for values cached per device (SM count).
// Plain C++: no CUDA types, so that the logic can be unit-tested on a machine without a GPU.
#pragma once

#include <mutex>

namespace sjd {

constexpr int kMaxDevices = 64;

// One flag per device ordinal.  run_once(dev, fn) calls fn() the first time it is asked for `dev` and
// remembers success only; a failure is retried on the next call.  Ordinals outside [0, kMaxDevices) are
// never remembered (fn runs every time).  fn returns 0 for success, anything else is passed through.
class DeviceOnce {
 public:
  template <typename Fn>
  int run_once(int dev, Fn&& fn) {
    if (dev < 0 || dev >= kMaxDevices) return fn();
    std::lock_guard<std::mutex> lock(mutex_);
    if (done_[dev]) return 0;
    const int rc = fn();
    if (rc == 0) done_[dev] = true;
    return rc;
  }
  bool done(int dev) {
    if (dev < 0 || dev >= kMaxDevices) return false;
    std::lock_guard<std::mutex> lock(mutex_);
    return done_[dev];
  }

 private:
  std::mutex mutex_;
  bool done_[kMaxDevices] = {};
};

// One cached integer per device ordinal (0 = not asked yet).  get(dev, fn) returns the cached value or
// asks fn() for it; values <= 0 are returned but not cached.
class DeviceValue {
 public:
  template <typename Fn>
  int get(int dev, Fn&& fn) {
    if (dev < 0 || dev >= kMaxDevices) return fn();
    std::lock_guard<std::mutex> lock(mutex_);
    if (value_[dev] > 0) return value_[dev];
    const int v = fn();
    if (v > 0) value_[dev] = v;
    return v;
  }

 private:
  std::mutex mutex_;
  int value_[kMaxDevices] = {};
};

}  // namespace sjd
