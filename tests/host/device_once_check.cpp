// Host-only check of the per-device set-up bookkeeping used by the kernel launchers: a second device must get its
// own set-up, a device that was set up must not get it again, and out-of-range ordinals are refused.
#include <cstdio>

#include "device_once.h"

int main() {
    uoe::DeviceOnce once;
    int setups = 0;
    const int order[] = {0, 0, 1, 0, 1, 63, 63};
    for (int dev : order)
        if (once.needs(dev)) { ++setups; once.mark(dev); }
    if (setups != 3) { std::printf("setups=%d\n", setups); return 1; }
    if (once.needs(-1) || once.needs(uoe::kMaxDevices) || once.valid(-1) || once.valid(uoe::kMaxDevices)) return 2;
    once.mark(-1);
    once.mark(uoe::kMaxDevices);           // ignored, no out-of-bounds write
    if (!once.needs(2)) return 3;

    uoe::DeviceValue v;
    if (v.has(0) || v.get(0) != 0) return 4;
    v.set(0, 148);
    v.set(1, 132);
    if (!v.has(0) || v.get(0) != 148 || v.get(1) != 132 || v.has(2)) return 5;
    v.set(uoe::kMaxDevices, 7);
    if (v.has(uoe::kMaxDevices) || v.has(-1)) return 6;
    std::printf("ok\n");
    return 0;
}
