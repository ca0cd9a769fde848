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
    header = "".join(open(os.path.join(ROOT, "include", h)).read() for h in ("moe_b200.h", "moe_b200_debug.h"))
    declared = set(re.findall(r"\b(moe_[a-z0-9_]+)\s*\(", header))
    public = open(os.path.join(ROOT, "include", "moe_b200.h")).read()
    assert not re.findall(r"\b(moe_debug_[a-z0-9_]+)\s*\(", public)      # diagnostics stay out of the layer's header
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
    big = C.c_void_p(0x10000)
    assert L.moe_forward(null, fake, fake, fake, fake, fake, C.byref(sh), fake, null, null, null, big, 1 << 30, null) == 1
    assert L.moe_forward(fake, fake, fake, fake, fake, fake, C.byref(sh), odd, null, null, null, big, 1 << 30, null) == 1
    assert L.moe_forward(fake, fake, fake, fake, fake, fake, C.byref(sh), fake, odd, null, null, big, 1 << 30, null) == 1   # topk_ids
    assert L.moe_forward(fake, fake, fake, fake, fake, fake, C.byref(bad), fake, null, null, null, big, 1 << 30, null) == 2
    assert L.moe_forward(fake, fake, fake, fake, fake, fake, C.byref(sh), fake, null, null, null, big, 64, null) == 3
    assert L.moe_forward(fake, fake, fake, fake, fake, fake, C.byref(sh), fake, null, null, null, null, 1 << 30, null) == 3


def test_prepack_sizes_and_argument_errors(L):
    sh = moe.shape(4, 1024, 512, 4, 2)
    n = 4 * 1024 * 512
    assert moe.moe_prepack_bytes(sh) == n + n // 16 + n // 2 + n // 32        # the same bytes, each tensor a multiple of 256
    assert moe.moe_prepack_bytes(moe.shape(4, 1000, 512, 4, 2)) == 0
    fake, odd, null = C.c_void_p(0x1000), C.c_void_p(0x1004), C.c_void_p(0)
    assert L.moe_prepack(null, fake, fake, fake, C.byref(sh), fake, 1 << 30, null) == 1
    assert L.moe_prepack(fake, fake, fake, fake, C.byref(sh), odd, 1 << 30, null) == 3
    assert L.moe_prepack(fake, fake, fake, fake, C.byref(sh), fake, 64, null) == 3
    assert L.moe_expert_ffn_packed(fake, fake, odd, C.byref(sh), fake, null, fake, 1 << 30, null) == 1
    assert L.moe_expert_ffn_packed(fake, fake, fake, C.byref(sh), fake, null, fake, 64, null) == 3
    assert L.moe_forward_packed(fake, fake, odd, C.byref(sh), fake, null, null, null, C.c_void_p(0x10000), 1 << 30, null) == 1
    assert L.moe_forward_host_packed(null, fake, fake, C.byref(sh), fake, null, fake, 1 << 30, null) == 1


def test_forward_workspace_sizes(L):
    """The workspace of moe_forward: the counter block, then room for the one-launch scratch or the four calls' buffers."""
    sync = moe.moe_forward_sync_bytes()
    assert sync >= 4 * (1024 + 64 + 2) and sync % 256 == 0
    for T, H, I, E, k in ((1, 4096, 2048, 256, 8), (4, 4096, 2048, 256, 8), (64, 4096, 2048, 256, 8), (16, 256, 128, 8, 2)):
        sh = moe.shape(T, H, I, E, k)
        S = T * k
        n = moe.moe_forward_workspace_bytes(sh)
        four = S * H * 2 + S * H * 4 + moe.moe_workspace_bytes(sh)        # x_perm, y_perm, the calls' own workspace
        one = S * H * 4 + 8 * S * (I // 2 + I // 32) + 8 * T * (H // 2 + H // 32)
        assert n >= sync + four and n >= sync + one and n % 256 == 0
        assert moe.moe_forward_host_workspace_bytes(sh) >= n + T * E * 4 + 2 * T * H * 2
    assert moe.moe_forward_workspace_bytes(moe.shape(64, 4000, 2048, 256, 8)) == 0


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(moe, "_lib", None)
    monkeypatch.setattr(moe, "LIB_PATH", "/nonexistent/libmoe_b200.so")
    with pytest.raises(moe.MoeError):
        moe.lib()


def test_decode_ffn_work_split_keeps_waits_pointing_down(L):
    """The decode-sized expert-FFN kernel runs both projections in one grid: a down item waits on the device for the
    gate/up items of its expert.  The split must cover every item exactly once, and every gate/up item an expert's
    down items wait for must belong to a CTA with a lower or equal index than theirs (CTAs start in index order, so
    such a wait can always end), with shares close to even."""
    n_ctas = 148
    for (H, I) in [(4096, 2048), (512, 512), (1024, 512), (512, 1024), (4096, 4096), (512, 4096)]:
        tiles0, tiles1 = 2 * I // 256, H // 256
        for n_touched in [0, 1, 2, 3, 7, 8, 9, 37, 74, 147, 148, 149, 224, 256, 1024]:
            shares = [moe.moe_debug_native_cta_share(n_ctas, c, n_touched, H, I) for c in range(n_ctas)]
            for ph, tiles in ((0, tiles0), (1, tiles1)):
                pos = 0
                for sh in shares:
                    b, e = sh[2 * ph], sh[2 * ph + 1]
                    assert b == min(pos, n_touched * tiles) or b == pos, (H, I, n_touched, ph, sh, pos)
                    assert e >= b
                    pos = e
                assert pos == n_touched * tiles
            owner0 = {}
            for c, sh in enumerate(shares):
                for it in range(sh[0], sh[1]):
                    owner0[it] = c
            for c, sh in enumerate(shares):
                for it in range(sh[2], sh[3]):
                    t = it // tiles1
                    assert max(owner0[g] for g in range(t * tiles0, (t + 1) * tiles0)) <= c, (H, I, n_touched, c, it)
            if n_touched:
                even1 = -(-n_touched * tiles1 // n_ctas)
                assert max(sh[3] - sh[2] for sh in shares) <= even1 + tiles1
    out = (C.c_int32 * 4)()
    assert L.moe_debug_native_cta_share(148, 148, 8, 4096, 2048, out) == 1
    assert L.moe_debug_native_cta_share(148, 0, 8, 4096, 100, out) == 1
