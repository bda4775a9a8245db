"""The per-device bookkeeping of the launch code (csrc/device_once.h: settings made once per (device, kernel),
values cached per device) exercised on the CPU with made-up device ordinals: a small C++ program is compiled
with g++ and run."""
import os
import subprocess
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

PROGRAM = textwrap.dedent("""
    #include "device_once.h"
    #include <cstdio>
    #include <thread>
    #include <vector>
    #include <atomic>
    #define CHECK(c) do { if (!(c)) { std::printf("FAILED line %d: %s\\n", __LINE__, #c); return 1; } } while (0)
    int main() {
      sjd::DeviceOnce once;
      int calls[4] = {0, 0, 0, 0};
      // a sequence of calls on two devices in one process: each device is configured exactly once
      for (int step = 0; step < 6; ++step) {
        const int dev = step % 2;
        CHECK(once.run_once(dev, [&] { ++calls[dev]; return 0; }) == 0);
      }
      CHECK(calls[0] == 1 && calls[1] == 1);
      CHECK(once.done(0) && once.done(1) && !once.done(2));
      // a failure is passed through and retried next time
      int tries = 0;
      CHECK(once.run_once(2, [&] { ++tries; return 7; }) == 7);
      CHECK(!once.done(2));
      CHECK(once.run_once(2, [&] { ++tries; return 0; }) == 0);
      CHECK(once.run_once(2, [&] { ++tries; return 0; }) == 0);
      CHECK(tries == 2 && once.done(2));
      // ordinals outside the table are never remembered
      int outside = 0;
      once.run_once(-1, [&] { ++outside; return 0; });
      once.run_once(sjd::kMaxDevices, [&] { ++outside; return 0; });
      once.run_once(sjd::kMaxDevices, [&] { ++outside; return 0; });
      CHECK(outside == 3 && !once.done(-1) && !once.done(sjd::kMaxDevices));
      // many threads, four devices: still once per device
      sjd::DeviceOnce shared;
      std::atomic<int> n[4];
      for (auto& x : n) x = 0;
      std::vector<std::thread> pool;
      for (int t = 0; t < 16; ++t)
        pool.emplace_back([&, t] { for (int r = 0; r < 1000; ++r) shared.run_once((t + r) % 4, [&, t, r] { ++n[(t + r) % 4]; return 0; }); });
      for (auto& th : pool) th.join();
      for (auto& x : n) CHECK(x == 1);
      // cached values: per device, asked once, non-positive answers not kept
      sjd::DeviceValue sms;
      int asked = 0;
      CHECK(sms.get(0, [&] { ++asked; return 148; }) == 148);
      CHECK(sms.get(0, [&] { ++asked; return 1; }) == 148);
      CHECK(sms.get(1, [&] { ++asked; return 132; }) == 132);
      CHECK(sms.get(1, [&] { ++asked; return 1; }) == 132);
      CHECK(asked == 2);
      CHECK(sms.get(3, [&] { ++asked; return 0; }) == 0);
      CHECK(sms.get(3, [&] { ++asked; return 64; }) == 64);
      CHECK(asked == 4);
      std::printf("DEVICE_ONCE_OK\\n");
      return 0;
    }
""")


def test_launch_state_is_kept_per_device(tmp_path):
    src = tmp_path / "device_once_test.cpp"
    src.write_text(PROGRAM)
    exe = tmp_path / "device_once_test"
    inc = os.path.join(ROOT, "paper_2512_07503_b200", "csrc")
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-pthread", "-I", inc, str(src), "-o", str(exe)])
    out = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and "DEVICE_ONCE_OK" in out.stdout, out.stdout + out.stderr
