// Bookkeeping for things the CUDA runtime keeps per device, not per process: function
// attributes (cudaFuncSetAttribute applies to the current device only), the SM count and
// occupancy results.  A process may drive several GPUs through this library, so every
// "done once" flag and every cached value is indexed by the device ordinal.
// Plain C++ (no CUDA headers) so that the bookkeeping can be exercised on a machine without a GPU.
#pragma once
#include <atomic>
#include <cstdint>

namespace prac {

constexpr int kMaxDevices = 64;

// One flag per device: has a once-per-device set-up step been done there?
class DeviceOnce {
 public:
  bool done(int dev) const {
    return dev >= 0 && dev < kMaxDevices && ((bits_.load(std::memory_order_acquire) >> dev) & 1u) != 0;
  }
  void mark(int dev) {
    if (dev >= 0 && dev < kMaxDevices) bits_.fetch_or(uint64_t{1} << dev, std::memory_order_release);
  }

 private:
  std::atomic<uint64_t> bits_{0};
};

// One cached positive integer per device (0 = not known yet).  Devices beyond the table are
// never cached: get() returns 0 and the caller recomputes.
class DeviceValue {
 public:
  int get(int dev) const {
    return (dev >= 0 && dev < kMaxDevices) ? v_[dev].load(std::memory_order_acquire) : 0;
  }
  void set(int dev, int value) {
    if (dev >= 0 && dev < kMaxDevices) v_[dev].store(value, std::memory_order_release);
  }

 private:
  std::atomic<int> v_[kMaxDevices] = {};
};

}  // namespace prac
