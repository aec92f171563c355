"""Host-side bookkeeping for set-up that CUDA keeps per device (shared-memory attribute of a kernel, SM count):
`csrc/aq_per_device.h` compiled with the host compiler alone and driven from a small C++ program."""
import os
import shutil
import subprocess
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HDR = os.path.join(ROOT, "paper_2605_24011_b200", "csrc")

SRC = textwrap.dedent(r"""
    #include <cstdio>
    #include "aq_per_device.h"
    using namespace aq;
    #define CHECK(c) do { if (!(c)) { std::printf("FAIL line %d: %s\n", __LINE__, #c); return 1; } } while (0)
    int main() {
        PerDeviceOnce once;
        int calls = 0;
        auto ok = [&] { ++calls; return 0; };
        CHECK(once.run(0, ok) == 0 && calls == 1);
        CHECK(once.run(0, ok) == 0 && calls == 1);          // device 0 is set up: not run again
        CHECK(once.run(1, ok) == 0 && calls == 2);          // a second device gets its own set-up
        CHECK(once.run(1, ok) == 0 && calls == 2);
        CHECK(once.is_done(0) && once.is_done(1) && !once.is_done(2));
        int tries = 0;
        auto fail_once = [&] { return ++tries == 1 ? 7 : 0; };
        CHECK(once.run(2, fail_once) == 7 && !once.is_done(2));   // a failed set-up is not recorded
        CHECK(once.run(2, fail_once) == 0 && once.is_done(2) && tries == 2);
        CHECK(once.run(-1, ok) == -1 && once.run(AQ_MAX_DEVICES, ok) == -1 && calls == 2);
        CHECK(once.run(AQ_MAX_DEVICES - 1, ok) == 0 && calls == 3);

        PerDeviceValue<int> val;
        int fills = 0, v = 0;
        auto fill = [&](int dev, int* out) { ++fills; *out = 100 + dev; return 0; };
        CHECK(val.get(3, &v, fill) == 0 && v == 103 && fills == 1);
        CHECK(val.get(3, &v, fill) == 0 && v == 103 && fills == 1);
        CHECK(val.get(5, &v, fill) == 0 && v == 105 && fills == 2);
        CHECK(val.get(3, &v, fill) == 0 && v == 103 && fills == 2);   // the first device's value is still its own
        CHECK(val.get(-1, &v, fill) == -1 && val.get(AQ_MAX_DEVICES, &v, fill) == -1);
        auto bad = [&](int, int*) { return 9; };
        CHECK(val.get(6, &v, bad) == 9);
        CHECK(val.get(6, &v, fill) == 0 && v == 106);
        std::printf("ok\n");
        return 0;
    }
""")


@pytest.mark.skipif(shutil.which("g++") is None, reason="needs a host C++ compiler")
def test_per_device_bookkeeping(tmp_path):
    src = tmp_path / "t.cpp"
    src.write_text(SRC)
    exe = tmp_path / "t"
    subprocess.run(["g++", "-std=c++17", "-O1", "-pthread", "-I", HDR, str(src), "-o", str(exe)], check=True)
    r = subprocess.run([str(exe)], capture_output=True, text=True)
    assert r.returncode == 0 and r.stdout.strip() == "ok", r.stdout + r.stderr
