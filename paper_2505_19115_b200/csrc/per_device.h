// Host-side state that belongs to a device, not to the process: the "maximum dynamic shared
// memory" attribute of a kernel and the multiprocessor count are properties of (function, device)
// and (device), so a process that uses the library on several GPUs must set or query them once per
// device.  Plain C++ (no CUDA types): the device ordinal is passed in, so the logic can be
// exercised on a machine without a GPU.
#pragma once

#include <atomic>

namespace nvfp4 {

constexpr int kMaxCachedDevices = 64;

// One flag per device ordinal.  A static instance per kernel instantiation records on which
// devices the one-time set-up of that kernel has succeeded.
struct DeviceFlags {
  std::atomic<unsigned char> done[kMaxCachedDevices];
};

// Runs `setup` (returns true on success) unless it already succeeded for `device`.  A failed set-up
// is not recorded, so the next call tries again.  Ordinals outside the table are never cached: the
// set-up then runs on every call, which is correct, only slower.  Two host threads may both run the
// set-up for the same device the first time; it is idempotent.
template <class Setup>
inline bool once_per_device(DeviceFlags& flags, int device, Setup&& setup) {
  const bool cached = device >= 0 && device < kMaxCachedDevices;
  if (cached && flags.done[device].load(std::memory_order_acquire)) return true;
  if (!setup()) return false;
  if (cached) flags.done[device].store(1, std::memory_order_release);
  return true;
}

// One integer per device ordinal (0 = not queried yet).
struct DeviceInts {
  std::atomic<int> value[kMaxCachedDevices];
};

// Returns the cached value for `device`, or calls `query` (returns a positive value, or <= 0 on
// failure, in which case `fallback` is returned and nothing is cached).
template <class Query>
inline int cached_per_device(DeviceInts& table, int device, int fallback, Query&& query) {
  const bool cached = device >= 0 && device < kMaxCachedDevices;
  if (cached) {
    const int v = table.value[device].load(std::memory_order_acquire);
    if (v > 0) return v;
  }
  const int q = query();
  if (q <= 0) return fallback;
  if (cached) table.value[device].store(q, std::memory_order_release);
  return q;
}

}  // namespace nvfp4
