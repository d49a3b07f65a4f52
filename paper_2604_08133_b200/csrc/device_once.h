// Host-side bookkeeping that is kept per CUDA device.  No CUDA headers: plain C++ so that it can be
// unit-tested without a GPU.
//
// A kernel's opt-in to more than 48 KB of dynamic shared memory (cudaFuncSetAttribute) and the SM
// count are properties of a device, not of the process: a process that drives several GPUs must set
// the attribute once on each of them and size its persistent grids for the GPU it launches on.
#pragma once

#include <atomic>

namespace allocmoe {

constexpr int kMaxDevices = 64;

// One flag per device ordinal: "the one-time set-up has been done on this device".  Ordinals outside
// [0, kMaxDevices) are never recorded, so their set-up is simply repeated on every call.
class PerDeviceOnce {
 public:
  bool done(int dev) const {
    return dev >= 0 && dev < kMaxDevices && flag_[dev].load(std::memory_order_acquire) != 0;
  }
  void mark(int dev) {
    if (dev >= 0 && dev < kMaxDevices) flag_[dev].store(1, std::memory_order_release);
  }

 private:
  std::atomic<unsigned char> flag_[kMaxDevices] = {};
};

// One cached int per device ordinal (0 = not known yet).
class PerDeviceInt {
 public:
  int get(int dev) const { return dev >= 0 && dev < kMaxDevices ? v_[dev].load(std::memory_order_acquire) : 0; }
  void set(int dev, int value) {
    if (dev >= 0 && dev < kMaxDevices) v_[dev].store(value, std::memory_order_release);
  }

 private:
  std::atomic<int> v_[kMaxDevices] = {};
};

}  // namespace allocmoe
