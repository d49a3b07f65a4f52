// Host-only check of the per-device bookkeeping (csrc/device_once.h): what is recorded for one device
// ordinal must not leak to another, and ordinals outside the table are never recorded.
#include <cstdio>

#include "device_once.h"

using namespace allocmoe;

static int fails = 0;
#define CHECK(c) do { if (!(c)) { std::printf("FAIL line %d: %s\n", __LINE__, #c); ++fails; } } while (0)

int main() {
  PerDeviceOnce once;
  for (int d = 0; d < kMaxDevices; ++d) CHECK(!once.done(d));
  once.mark(0);
  CHECK(once.done(0));
  CHECK(!once.done(1));                 // a second GPU of the same process still needs its own set-up
  once.mark(5);
  CHECK(once.done(5) && !once.done(4) && !once.done(6));
  once.mark(-1);
  once.mark(kMaxDevices);               // outside the table: ignored, and reported as not done
  CHECK(!once.done(-1) && !once.done(kMaxDevices));
  for (int d = 0; d < kMaxDevices; ++d) CHECK(once.done(d) == (d == 0 || d == 5));

  PerDeviceInt sms;
  CHECK(sms.get(0) == 0 && sms.get(3) == 0);
  sms.set(0, 148);
  sms.set(3, 132);
  CHECK(sms.get(0) == 148 && sms.get(3) == 132 && sms.get(1) == 0);
  sms.set(kMaxDevices + 2, 7);
  CHECK(sms.get(kMaxDevices + 2) == 0 && sms.get(-3) == 0);
  std::printf(fails ? "FAILED\n" : "ok\n");
  return fails ? 1 : 0;
}
