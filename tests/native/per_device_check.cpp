// Host-only check of the per-device launch-state cache (paper_2505_19115_b200/csrc/per_device.h)
// behind fake device ordinals: no CUDA involved.  Prints "ok" and exits 0 when every check holds.
#include <cstdio>
#include <cstdlib>

#include "per_device.h"

#define CHECK(cond)                                                         \
  do {                                                                      \
    if (!(cond)) { std::printf("FAILED line %d: %s\n", __LINE__, #cond); return 1; } \
  } while (0)

int main() {
  using namespace nvfp4;
  static DeviceFlags flags;                 // zero-initialised like the statics in the launch functions
  int calls[kMaxCachedDevices + 2] = {};
  auto setup_for = [&](int dev, bool succeed) {
    return [&calls, dev, succeed] { ++calls[dev < 0 ? kMaxCachedDevices + 1 : (dev >= kMaxCachedDevices ? kMaxCachedDevices : dev)]; return succeed; };
  };
  // first use on device 0 runs the set-up, the second does not
  CHECK(once_per_device(flags, 0, setup_for(0, true)) && calls[0] == 1);
  CHECK(once_per_device(flags, 0, setup_for(0, true)) && calls[0] == 1);
  // a second device gets its own set-up even though device 0 is done (the bug a process-wide flag has)
  CHECK(once_per_device(flags, 1, setup_for(1, true)) && calls[1] == 1);
  CHECK(once_per_device(flags, 1, setup_for(1, true)) && calls[1] == 1);
  // switching back does not repeat it
  CHECK(once_per_device(flags, 0, setup_for(0, true)) && calls[0] == 1);
  // a failed set-up is reported and not cached: the next call tries again
  CHECK(!once_per_device(flags, 2, setup_for(2, false)) && calls[2] == 1);
  CHECK(once_per_device(flags, 2, setup_for(2, true)) && calls[2] == 2);
  CHECK(once_per_device(flags, 2, setup_for(2, true)) && calls[2] == 2);
  // ordinals outside the table (or an unknown device, -1) are never cached
  CHECK(once_per_device(flags, kMaxCachedDevices, setup_for(kMaxCachedDevices, true)));
  CHECK(once_per_device(flags, kMaxCachedDevices, setup_for(kMaxCachedDevices, true)) && calls[kMaxCachedDevices] == 2);
  CHECK(once_per_device(flags, -1, setup_for(-1, true)));
  CHECK(once_per_device(flags, -1, setup_for(-1, true)) && calls[kMaxCachedDevices + 1] == 2);
  // the last slot of the table is cached
  CHECK(once_per_device(flags, kMaxCachedDevices - 1, setup_for(kMaxCachedDevices - 1, true)));
  CHECK(once_per_device(flags, kMaxCachedDevices - 1, setup_for(kMaxCachedDevices - 1, true)) && calls[kMaxCachedDevices - 1] == 1);

  // per-device integers (the multiprocessor count): each device keeps its own value
  static DeviceInts sms;
  int queries = 0;
  CHECK(cached_per_device(sms, 0, 148, [&] { ++queries; return 148; }) == 148 && queries == 1);
  CHECK(cached_per_device(sms, 1, 148, [&] { ++queries; return 132; }) == 132 && queries == 2);
  CHECK(cached_per_device(sms, 0, 148, [&] { ++queries; return 7; }) == 148 && queries == 2);
  CHECK(cached_per_device(sms, 1, 148, [&] { ++queries; return 7; }) == 132 && queries == 2);
  // a failed query returns the fallback and is asked again next time
  CHECK(cached_per_device(sms, 3, 148, [&] { ++queries; return 0; }) == 148 && queries == 3);
  CHECK(cached_per_device(sms, 3, 148, [&] { ++queries; return 160; }) == 160 && queries == 4);
  CHECK(cached_per_device(sms, -1, 148, [&] { ++queries; return 99; }) == 99 && queries == 5);
  CHECK(cached_per_device(sms, -1, 148, [&] { ++queries; return 98; }) == 98 && queries == 6);
  std::printf("ok\n");
  return 0;
}
