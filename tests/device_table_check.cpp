// Host-only check of the per-device cache that the launchers use for state CUDA keeps per device
// (opt-in shared-memory limits, SM counts).  Compiled and run by tests/test_device_table_host.py.
#include <cstdio>

#include "mq_device_table.h"

static int g_calls[128];

static bool make_ok(int dev, int* out) {
  if (dev >= 0 && dev < 128) ++g_calls[dev];
  *out = 100 + dev;
  return true;
}

static int g_fail_calls = 0;
static bool make_fail_once(int dev, int* out) {
  if (g_fail_calls++ == 0) return false;
  *out = 7 + dev;
  return true;
}

#define CHECK(cond)                                                  \
  do {                                                               \
    if (!(cond)) {                                                   \
      std::printf("FAILED line %d: %s\n", __LINE__, #cond);          \
      return 1;                                                      \
    }                                                                \
  } while (0)

int main() {
  mq::PerDeviceTable<int, 4> t;
  int v = 0;
  // every device is initialised on its own first use, exactly once
  CHECK(t.get(0, make_ok, &v) && v == 100);
  CHECK(t.get(1, make_ok, &v) && v == 101);
  CHECK(t.get(0, make_ok, &v) && v == 100);
  CHECK(t.get(1, make_ok, &v) && v == 101);
  CHECK(t.get(3, make_ok, &v) && v == 103);
  CHECK(g_calls[0] == 1 && g_calls[1] == 1 && g_calls[2] == 0 && g_calls[3] == 1);
  // a device beyond the table is served without caching
  CHECK(t.get(9, make_ok, &v) && v == 109);
  CHECK(t.get(9, make_ok, &v) && v == 109);
  CHECK(g_calls[9] == 2);
  CHECK(t.get(-1, make_ok, &v) && v == 99);
  // a failed set-up is reported and not remembered
  mq::PerDeviceTable<int, 4> u;
  CHECK(!u.get(2, make_fail_once, &v));
  CHECK(u.get(2, make_fail_once, &v) && v == 9);
  CHECK(u.get(2, make_fail_once, &v) && v == 9);
  CHECK(g_fail_calls == 2);
  std::printf("ok\n");
  return 0;
}
