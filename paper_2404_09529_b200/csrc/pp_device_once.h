// A "done once per device" record for set-up that CUDA keeps per device (a kernel's shared-memory
// opt-in, for one). Lock-free and safe from several host threads: two threads may both find a device
// not done and both run the set-up, which is harmless for idempotent set-up; none can see "done"
// before some thread has finished it. Devices beyond the table are never recorded, so their set-up
// simply runs on every call.
#ifndef PREPACK_B200_PP_DEVICE_ONCE_H_
#define PREPACK_B200_PP_DEVICE_ONCE_H_

#include <atomic>
#include <cstdint>

namespace pp {

class DeviceOnce {
 public:
  static constexpr int kMaxDevices = 128;
  bool done(int device) const {
    if (device < 0 || device >= kMaxDevices) return false;
    return (bits_[device >> 6].load(std::memory_order_acquire) >> (device & 63)) & 1u;
  }
  void mark(int device) {
    if (device < 0 || device >= kMaxDevices) return;
    bits_[device >> 6].fetch_or(uint64_t(1) << (device & 63), std::memory_order_release);
  }

 private:
  std::atomic<uint64_t> bits_[kMaxDevices / 64] = {};
};

}  // namespace pp

#endif  // PREPACK_B200_PP_DEVICE_ONCE_H_
