"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol,
and rejects bad arguments before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2406_12018_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "citrus.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(citrus_[a-z_]+)\s*\(", text)))


def test_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_error_strings(lib):
    assert binding.strerror(0) == "ok"
    for code in range(-9, 0):
        assert binding.strerror(code) not in ("ok", "unknown error")
    assert binding.strerror(-99) == "unknown error"


def test_create_rejects_bad_geometry_without_a_device(lib):
    h = C.c_void_p()
    f = lib.citrus_create
    assert f(None, 1, 8, 2, 64, 64, 128, 2) == -1
    assert f(C.byref(h), 0, 8, 2, 64, 64, 128, 2) == -1           # layers
    assert f(C.byref(h), 1, 8, 3, 64, 64, 128, 2) == -2           # q_heads % kv_heads
    assert f(C.byref(h), 1, 8, 2, 96, 64, 128, 2) == -9           # head_dim
    assert f(C.byref(h), 1, 8, 2, 64, 64, 128, 0) == -9           # bf16 needs head_dim 128
    assert f(C.byref(h), 1, 8, 2, 128, 40000, 20000, 0) == -9     # too many candidates
    assert f(C.byref(h), 1, 8, 2, 128, 64, 128, 1 << 30) == -1    # unknown mode bits
    assert h.value is None


def test_null_and_unknown_handles(lib):
    assert lib.citrus_destroy(None) == 0
    bogus = C.c_void_p(0x1000)
    assert lib.citrus_destroy(bogus) == -1
    assert lib.citrus_reset(bogus) == -1
    assert lib.citrus_poll_status(None) == -1
    assert lib.citrus_process_chunk(bogus, 0, None, None, None, 1, None, 1, None, None) == -1


def test_per_device_setup_bookkeeping(tmp_path):
    # The kernels' shared-memory limits and the static scratch address are per-device facts: the record of which
    # devices have had their set-up (DeviceOnce in the library's internal header) is compiled here with the host
    # compiler alone and driven as the launchers drive it.
    import subprocess
    src = tmp_path / "once.cpp"
    src.write_text(r'''
#include "citrus_internal.h"
#include <cstdio>
int main() {
    citrus::DeviceOnce once;
    int setups = 0;
    const int order[] = {0, 0, 1, 0, 1, 63, 63};
    for (int dev : order) {
        if (once.needs_setup(dev)) { ++setups; once.mark(dev); }
    }
    if (setups != 3) { std::printf("setups %d\n", setups); return 1; }         // once per device, not once per process
    if (once.needs_setup(0) || once.needs_setup(1) || once.needs_setup(63)) return 2;
    if (!once.needs_setup(2)) return 3;                                         // an untouched device still needs it
    // out-of-range ids are never recorded: the set-up simply runs every time
    once.mark(64); once.mark(-1);
    if (!once.needs_setup(64) || !once.needs_setup(-1)) return 4;
    return 0;
}
''')
    exe = tmp_path / "once"
    inc = os.path.join(ROOT, "paper_2406_12018_b200", "csrc")
    r = subprocess.run(["g++", "-std=c++17", "-I", inc, "-I", "/usr/local/cuda/include", str(src), "-o", str(exe)],
                       capture_output=True, text=True)
    assert r.returncode == 0, r.stderr[-2000:]
    r = subprocess.run([str(exe)], capture_output=True, text=True)
    assert r.returncode == 0, (r.returncode, r.stdout)
