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
