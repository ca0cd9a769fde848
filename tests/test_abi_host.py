"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol and rejects bad
arguments on the host before touching the device (no compute call is made here)."""
import ctypes as C
import os
import re

import pytest

from paper_2609_15627_b200 import build_ext, moe

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build_ext.build()
    return moe.lib()


def test_every_declared_symbol_is_exported(L):
    header = open(os.path.join(ROOT, "include", "moe_b200.h")).read()
    declared = set(re.findall(r"\b(moe_[a-z0-9_]+)\s*\(", header))
    declared -= {"moe_status_t", "moe_shape_t"}
    assert {"moe_route", "moe_permute", "moe_expert_ffn", "moe_combine"} <= declared
    for name in sorted(declared):
        assert hasattr(L, name), name
    assert declared == set(moe.EXPORTS)


def test_workspace_and_status_strings(L):
    sh = moe.shape(64, 4096, 2048, 256, 8)
    assert moe.moe_workspace_bytes(sh) >= 64 * 8 * 2048 * 2
    assert moe.moe_workspace_bytes(moe.shape(64, 4000, 2048, 256, 8)) == 0   # H % 128
    assert moe.moe_workspace_bytes(moe.shape(64, 4096, 2048, 2048, 8)) == 0  # E > 1024
    assert moe.moe_workspace_bytes(moe.shape(64, 4096, 2048, 4, 8)) == 0     # k > E
    assert L.moe_status_string(0) == b"ok"
    assert len({L.moe_status_string(i) for i in range(6)}) == 6


def test_argument_errors_are_found_on_the_host(L):
    sh = moe.shape(4, 256, 128, 8, 2)
    fake = C.c_void_p(0x1000)           # never dereferenced: validation fails first
    odd = C.c_void_p(0x1004)
    null = C.c_void_p(0)
    assert L.moe_route(null, 4, 8, 2, fake, fake, fake, fake, 1 << 20, null) == 1
    assert L.moe_route(fake, 4, 8, 9, fake, fake, fake, fake, 1 << 20, null) == 1      # k > E
    assert L.moe_route(fake, 0, 8, 2, fake, fake, fake, fake, 1 << 20, null) == 1      # T < 1
    assert L.moe_route(fake, 4, 2048, 2, fake, fake, fake, fake, 1 << 20, null) == 2   # E > 1024
    assert L.moe_route(fake, 4, 64, 40, fake, fake, fake, fake, 1 << 20, null) == 2    # k > 32
    assert L.moe_route(odd, 4, 8, 2, fake, fake, fake, fake, 1 << 20, null) == 1       # misaligned
    assert L.moe_route(fake, 4, 8, 2, fake, fake, fake, fake, 16, null) == 3           # ws too small
    assert L.moe_route(fake, 4, 8, 2, fake, fake, fake, null, 1 << 20, null) == 3      # ws NULL
    assert L.moe_permute(fake, fake, fake, C.byref(sh), fake, fake, fake, fake, 8, null) == 3
    assert L.moe_permute(null, fake, fake, C.byref(sh), fake, fake, fake, fake, 1 << 20, null) == 1
    bad = moe.shape(4, 200, 128, 8, 2)
    assert L.moe_expert_ffn(fake, fake, fake, fake, fake, fake, C.byref(bad), fake, null, fake, 1 << 20, null) == 2
    assert L.moe_expert_ffn(fake, fake, fake, fake, fake, fake, C.byref(sh), odd, null, fake, 1 << 20, null) == 1
    assert L.moe_expert_ffn(fake, fake, fake, fake, fake, fake, C.byref(sh), fake, null, fake, 64, null) == 3
    assert L.moe_combine(fake, fake, fake, C.byref(sh), null, null) == 1
    assert L.moe_combine(fake, fake, fake, None, fake, null) == 1
    assert L.moe_validate_scales(null, 16, fake, null) == 1
    assert L.moe_forward_host(null, fake, fake, fake, fake, fake, C.byref(sh), fake, null, fake, 1 << 30, null) == 1


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(moe, "_lib", None)
    monkeypatch.setattr(moe, "LIB_PATH", "/nonexistent/libmoe_b200.so")
    with pytest.raises(moe.MoeError):
        moe.lib()
