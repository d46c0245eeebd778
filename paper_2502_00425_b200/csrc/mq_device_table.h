// Host-side state that CUDA keeps per DEVICE (a kernel's opt-in shared-memory limit, the SM count
// that sizes a launch) must be cached per device too: a process may drive several GPUs through
// this library, and a value set up or read on the first one says nothing about the second.
// This header is plain C++ (no CUDA types) so that the table logic can be unit-tested on a CPU.
#pragma once

#include <mutex>

namespace mq {

// One lazily initialised slot of type T per device index.  `get(dev, make, out)` returns the cached
// value of device `dev`, calling `make(dev, &value)` (which returns true on success) the first time
// only.  A failed `make` is not cached, so a later call tries again.  A device index outside
// [0, kMax) is served without caching: `make` runs on every call, which is slower but never wrong.
template <typename T, int kMax = 64>
class PerDeviceTable {
 public:
  template <typename Make>
  bool get(int dev, Make make, T* out) {
    if (dev < 0 || dev >= kMax) return make(dev, out);
    std::lock_guard<std::mutex> lock(mu_);
    if (!ready_[dev]) {
      T v{};
      if (!make(dev, &v)) return false;
      value_[dev] = v;
      ready_[dev] = true;
    }
    *out = value_[dev];
    return true;
  }

 private:
  std::mutex mu_;
  T value_[kMax] = {};
  bool ready_[kMax] = {};
};

}  // namespace mq
