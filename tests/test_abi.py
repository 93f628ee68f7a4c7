"""CPU-side checks of the C-ABI library: it builds, loads, exports everything the header declares,
and rejects bad arguments before touching a device.  No compute call is made here."""
import ctypes
import os
import re

import pytest

from paper_2510_04286_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "slicemoe.h")


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding._lib()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(slicemoe_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert "slicemoe_forward" in names and "slicemoe_route" in names and len(names) >= 12
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in slicemoe.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_status_strings(lib):
    assert binding.slicemoe_status_string(0) == "ok"
    seen = {binding.slicemoe_status_string(i) for i in range(10)}
    assert len(seen) == 10
    assert binding.slicemoe_status_string(99) == "unknown status"


def cfg(**kw):
    base = dict(T=64, d=512, S=8, E=16, k=2, F=256)
    base.update(kw)
    return binding.Config(**base)


def ws_bytes(lib, c):
    out = ctypes.c_size_t(0)
    cc = c.c()
    return lib.slicemoe_workspace_bytes(ctypes.byref(cc), ctypes.byref(out)), out.value


def test_workspace_sizing(lib):
    rc, small = ws_bytes(lib, cfg(T=64))
    assert rc == 0 and small > 0 and small % 256 == 0
    rc, big = ws_bytes(lib, cfg(T=16384))
    assert rc == 0 and big > small
    # stacked rows in and out dominate: 2 * R * ds * 2 bytes
    assert big >= 2 * 16384 * 8 * 2 * 64 * 2
    rc, empty = ws_bytes(lib, cfg(T=0))
    assert rc == 0 and empty > 0


@pytest.mark.parametrize("kw,status", [
    (dict(d=500), 2),            # d % S != 0
    (dict(k=17), 2),             # k > E
    (dict(k=0), 2),
    (dict(T=-1), 2),
    (dict(capacity=-5), 2),
    (dict(T=2 ** 28), 2),        # T*S*k overflows int32
    (dict(dtype=7), 3),
    (dict(act=9), 3),
    (dict(d=8 * 12), 3),         # ds = 12 is not a multiple of 8 (bf16 vectors)
    (dict(k=9, E=16), 3),
    (dict(E=512), 3),
    (dict(F=100), 3),
])
def test_bad_configs_are_rejected(lib, kw, status):
    rc, _ = ws_bytes(lib, cfg(**kw))
    assert rc == status


def test_argument_checks_come_before_any_device_work(lib):
    c = cfg().c()
    fake = ctypes.c_void_p(0x1000)          # aligned, never dereferenced: checks fail first
    odd = ctypes.c_void_p(0x1004)
    w = binding._Weights(*([0x1000] * 8))
    wnull = binding._Weights(*([None] * 8))
    big = ctypes.c_size_t(1 << 40)
    n = ctypes.c_void_p(None)
    f = lib.slicemoe_forward
    assert f(ctypes.byref(c), ctypes.byref(w), n, fake, n, n, n, n, fake, big, n) == 1          # h NULL
    assert f(ctypes.byref(c), ctypes.byref(wnull), fake, fake, n, n, n, n, fake, big, n) == 1   # weights NULL
    assert f(ctypes.byref(c), ctypes.byref(w), odd, fake, n, n, n, n, fake, big, n) == 4        # misaligned h
    assert f(ctypes.byref(c), ctypes.byref(w), fake, fake, n, n, n, n, fake, big, n) == 6       # h_out aliases h
    far = ctypes.c_void_p(0x1000 + (1 << 30))
    assert f(ctypes.byref(c), ctypes.byref(w), fake, far, n, n, n, n, n, big, n) == 5           # no workspace
    assert f(ctypes.byref(c), ctypes.byref(w), fake, far, n, n, n, n, fake, ctypes.c_size_t(16), n) == 5
    assert f(None, ctypes.byref(w), fake, far, n, n, n, n, fake, big, n) == 1
    assert lib.slicemoe_combine(ctypes.byref(c), n, fake, fake, n) == 1
    assert lib.slicemoe_dispatch(ctypes.byref(c), n, fake, fake, fake, fake, fake, fake, fake, fake, big, n) == 1
    assert lib.slicemoe_forward_profiled(ctypes.byref(c), ctypes.byref(w), fake, far, n, n, n, n, fake, big, n, n) == 1
    assert binding.slicemoe_launch_count() == 0


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_handle", None)
    monkeypatch.setattr(binding, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libslicemoe.so"))
    with pytest.raises(RuntimeError, match="missing"):
        binding.slicemoe_workspace_bytes(cfg())


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2510_04286_b200")
    for dirpath, _, files in os.walk(pkg):
        for name in files:
            if name.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, name)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b", text, flags=re.M), name
                assert "slicemoe_oracle" not in text, name
    oracle_dir = os.path.join(ROOT, "oracle")
    for name in os.listdir(oracle_dir):
        if name.endswith((".py", ".c")):
            text = open(os.path.join(oracle_dir, name)).read()
            assert "paper_2510_04286_b200" not in text and "libslicemoe.so" not in text, name
