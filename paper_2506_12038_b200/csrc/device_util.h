// Per-device bookkeeping of the kernel launchers: a kernel's attributes (the opt-in to large dynamic shared memory)
// belong to the device that is current when they are set, and a process may use several devices from several threads.
#ifndef LCD_DEVICE_UTIL_H_
#define LCD_DEVICE_UTIL_H_

#include <cuda_runtime.h>

#include <atomic>

namespace lcd {

// One flag per device (up to 64) for one kernel instance: first() is true until done() was called for the current
// device.  Two threads that race both set the attribute, which is harmless.
struct PerDeviceFlag {
  std::atomic<unsigned long long> mask{0ull};
  bool first(int* dev) const {
    *dev = 0;
    if (cudaGetDevice(dev) != cudaSuccess || *dev < 0 || *dev >= 64) return true;   // unknown device: always set
    return ((mask.load(std::memory_order_acquire) >> *dev) & 1ull) == 0;
  }
  void done(int dev) {
    if (dev >= 0 && dev < 64) mask.fetch_or(1ull << dev, std::memory_order_release);
  }
};

// Multiprocessors of the current device (148 if it cannot be asked).
inline int current_sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
    n = 148;
  return n;
}

}  // namespace lcd
#endif
