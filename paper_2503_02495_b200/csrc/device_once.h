// Per-device one-time set-up bookkeeping (plain C++, no CUDA types, so that it can be compiled and tested on its own).
//
// Function attributes (the opt-in to more than 48 KB of dynamic shared memory), occupancy figures and the SM count
// belong to a device, not to the process: a process that drives several GPUs must repeat the set-up on each.  A
// launcher keeps one `static DeviceOnce` (and, where it caches a number, one `static DeviceValue`) and asks it with
// the ordinal of the current device.  Not thread-safe: two threads making the first call on the same device both
// run the set-up, which is harmless for idempotent set-up but is a data race on the flag.
#pragma once

namespace uoe {

constexpr int kMaxDevices = 64;

struct DeviceOnce {
    bool done[kMaxDevices] = {};
    // true when `dev` is a usable ordinal whose set-up has not run yet
    bool needs(int dev) const { return dev >= 0 && dev < kMaxDevices && !done[dev]; }
    void mark(int dev) { if (dev >= 0 && dev < kMaxDevices) done[dev] = true; }
    bool valid(int dev) const { return dev >= 0 && dev < kMaxDevices; }
};

struct DeviceValue {
    int value[kMaxDevices] = {};
    bool known[kMaxDevices] = {};
    bool has(int dev) const { return dev >= 0 && dev < kMaxDevices && known[dev]; }
    int get(int dev) const { return has(dev) ? value[dev] : 0; }
    void set(int dev, int v) { if (dev >= 0 && dev < kMaxDevices) { value[dev] = v; known[dev] = true; } }
};

}  // namespace uoe
