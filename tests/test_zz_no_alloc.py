"""The allocation-free entry point moe_expert_ffn_noalloc against moe_expert_ffn (GPU).

Some callers of this library may not call cudaMalloc where they run (inside another framework's
graph-managed section, a real-time loop, a host that only hands over input and output buffers), so they
cannot provide the workspace moe_expert_ffn wants.  moe_expert_ffn_noalloc keeps that scratch in a fixed
array inside the library.  This test calls it through the C ABI twice in a row (the array is shared and
keeps the previous call's contents) and checks each result against the regular entry point.
Collected last on purpose: a run that stops at the first failure has then already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2609_15627_b200 import inputs, moe

pytestmark = pytest.mark.gpu


def _dev(a):
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def _case(T, H, I, E, k, seed):
    w = [_dev(a) for a in inputs.make_expert_weights(H, I, E, seed=seed)]
    logits, x = inputs.make_logits(T, E, seed), inputs.make_x(T, H, seed)
    ids, _, off = O.route(logits, k)          # inputs of the call only; outputs are compared GPU to GPU
    x_perm, _, _ = O.permute(x, ids, off)
    return w, _dev(x_perm), _dev(off), moe.shape(T, H, I, E, k)


_NATIVE, _UMMA, _STREAM = "ffn_native_mxf4_block_scaled", "ffn_umma_tcgen05_grouped", "ffn_stream_bulk_ring_mma16816"

# Every kernel variant behind the entry point, each carving its own kind of scratch out of the fixed array: the
# decode-sized variant its E2M1 term rows, scale bytes and per-expert counters (read back through TMA tensor maps),
# the prefill-sized variant the bf16 intermediate behind a tensor map, the streaming variant the bf16 intermediate.
# Different shapes back to back: each call finds the previous call's data in the array.  The last case is the largest
# decode-sized batch at the production H and I whose scratch (26,112 bytes per slot) still fits the 16 MiB.
_CASES = [(64, 512, 384, 8, 2, 0, _STREAM), (8, 1024, 512, 32, 6, 3, _NATIVE), (16, 256, 128, 8, 2, 1, _STREAM),
          (256, 512, 512, 8, 6, 4, _UMMA), (4, 512, 512, 8, 2, 5, _NATIVE), (64, 512, 256, 8, 2, 2, _NATIVE),
          (80, 4096, 2048, 32, 8, 6, _NATIVE)]


def test_noalloc_matches_regular_entry_point_on_two_calls_in_a_row():
    assert torch.cuda.is_available()
    assert moe.moe_expert_ffn_noalloc_max_bytes() == 16 << 20
    for (T, H, I, E, k, seed, kernel) in _CASES:
        w, x_perm, off, sh = _case(T, H, I, E, k, seed)
        buf = moe.LayerBuffers(sh)
        moe.moe_expert_ffn(x_perm, off, *w, sh, buf.y_perm, buf.status, buf.ws)
        torch.cuda.synchronize()
        assert moe.moe_last_kernel_name() == kernel
        want = buf.y_perm.clone()
        for _ in range(2):
            got = torch.full_like(want, float("nan"))
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            moe.moe_expert_ffn_noalloc(x_perm, off, *w, sh, got, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert moe.moe_last_kernel_name() == kernel   # same kernel choice as the regular entry point
            # same kernels on the same inputs: the tolerance of the other tests is met with equality
            assert torch.equal(got, want)
            rel = float((got - want).norm() / want.norm())
            assert rel <= 5e-4
        # and against the oracle, within the tolerance of the fp32 per-slot rows
        ref = O.expert_ffn(x_perm.view(torch.int16).cpu().numpy().view(np.uint16), off.cpu().numpy(),
                           *[a.cpu().numpy() for a in w], k)
        g = got.cpu().numpy().astype(np.float64)
        r = ref.astype(np.float64)
        rms = np.sqrt(np.mean(r ** 2))
        assert np.linalg.norm(g - r) / np.linalg.norm(r) <= 5e-4 and np.abs(g - r).max() <= 2e-2 * rms


def test_noalloc_rejects_a_misaligned_status_word():
    L = moe.lib()
    w, x_perm, off, sh = _case(16, 256, 128, 8, 2, 1)
    y = torch.empty((32, 256), dtype=torch.float32, device="cuda")
    st = torch.zeros(2, dtype=torch.int32, device="cuda")
    args = [C.c_void_p(t.data_ptr()) for t in (x_perm, off, *w)]
    bad = C.c_void_p(st.data_ptr() + 2)
    assert L.moe_expert_ffn_noalloc(*args, C.byref(sh), C.c_void_p(y.data_ptr()), bad, None) == 1


def test_noalloc_rejects_sizes_beyond_the_fixed_array():
    L = moe.lib()
    fake = C.c_void_p(0x1000)  # never dereferenced: the size check comes first
    big = moe.shape(4096, 4096, 2048, 256, 8)   # 2*T*k*I = 128 MiB > 16 MiB
    assert L.moe_expert_ffn_noalloc(fake, fake, fake, fake, fake, fake, C.byref(big), fake, None, None) == 3
    assert L.moe_expert_ffn_noalloc(fake, fake, fake, fake, fake, fake, None, fake, None, None) == 1
