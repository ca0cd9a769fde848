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


def test_noalloc_matches_regular_entry_point_on_two_calls_in_a_row():
    assert torch.cuda.is_available()
    assert moe.moe_expert_ffn_noalloc_max_bytes() == 16 << 20
    # two different shapes back to back: the second call finds the first call's data in the array
    for (T, H, I, E, k, seed) in [(64, 512, 256, 8, 2, 0), (16, 256, 128, 8, 2, 1), (64, 512, 256, 8, 2, 2)]:
        w, x_perm, off, sh = _case(T, H, I, E, k, seed)
        buf = moe.LayerBuffers(sh)
        moe.moe_expert_ffn(x_perm, off, *w, sh, buf.y_perm, buf.status, buf.ws)
        torch.cuda.synchronize()
        want = buf.y_perm.clone()
        for _ in range(2):
            got = torch.full_like(want, float("nan"))
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            moe.moe_expert_ffn_noalloc(x_perm, off, *w, sh, got, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            # same kernels on the same inputs: the tolerance of the other tests is met with equality
            assert torch.equal(got, want)
            rel = float((got - want).norm() / want.norm())
            assert rel <= 5e-4


def test_noalloc_rejects_sizes_beyond_the_fixed_array():
    L = moe.lib()
    fake = C.c_void_p(0x1000)  # never dereferenced: the size check comes first
    big = moe.shape(4096, 4096, 2048, 256, 8)   # 2*T*k*I = 128 MiB > 16 MiB
    assert L.moe_expert_ffn_noalloc(fake, fake, fake, fake, fake, fake, C.byref(big), fake, None, None) == 3
    assert L.moe_expert_ffn_noalloc(fake, fake, fake, fake, fake, fake, None, fake, None, None) == 1
