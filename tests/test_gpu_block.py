"""GPU parity of the steps either side of the routed path - router projection, shared expert, join - and of the FFN block
they make with it (paper, figure "Execution structure"), against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from _gpu_util import bits, check_out, check_y, dev, weights_dev
from oracle import moe_oracle as O
from paper_2609_15627_b200 import inputs, moe

pytestmark = pytest.mark.gpu

bf = inputs.bf16_bits_to_f32


def _router_weights(E, H, seed):
    return inputs.f32_to_bf16_bits(bf(inputs.make_x(E, H, seed)) * np.float32(0.03))


@pytest.mark.parametrize("T,H,E,kernel", [
    (1, 4096, 256, "router_gemv_warp_per_expert"), (7, 512, 8, "router_gemv_warp_per_expert"),
    (16, 1024, 100, "router_gemv_warp_per_expert"), (17, 512, 64, "router_gemm_tcgen05_128x64"),
    (200, 512, 40, "router_gemm_tcgen05_128x64"), (1000, 1024, 256, "router_gemm_tcgen05_128x64"),
    (64, 4096, 256, "router_gemm_tcgen05_128x64"), (300, 256, 1024, "router_gemm_tcgen05_128x64")])
def test_router_logits_against_oracle(T, H, E, kernel):
    x, wr = inputs.make_x(T, H, 3), _router_weights(E, H, 4)
    lg = torch.full((T, E), float("nan"), dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    moe.moe_router_logits(dev(x), dev(wr), lg, st)
    torch.cuda.synchronize()
    assert moe.moe_last_kernel_name() == kernel and int(st.item()) == 0
    ref = O.router_logits(x, wr)
    got = lg.cpu().numpy()
    # both sum exact products in fp32, in different orders: each is within H * 2^-24 * sum |terms| of the true value
    bound = 2 * H * 2.0 ** -24 * (np.abs(bf(x).astype(np.float64)) @ np.abs(bf(wr).astype(np.float64)).T) + 1e-30
    assert np.isfinite(got).all() and np.all(np.abs(got.astype(np.float64) - ref) <= bound)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 1e-5


def test_router_logits_exact_on_small_integers():
    # every partial sum is an integer below 2^24: any summation order gives the exact result
    rng = np.random.default_rng(0)
    for T in (3, 150):
        xi = rng.integers(-8, 9, (T, 512)).astype(np.float32)
        wi = rng.integers(-8, 9, (72, 512)).astype(np.float32)
        lg = torch.empty((T, 72), dtype=torch.float32, device="cuda")
        moe.moe_router_logits(dev(inputs.f32_to_bf16_bits(xi)), dev(inputs.f32_to_bf16_bits(wi)), lg)
        torch.cuda.synchronize()
        assert np.array_equal(lg.cpu().numpy().astype(np.int64), xi.astype(np.int64) @ wi.astype(np.int64).T)


@pytest.mark.parametrize("T,H,k", [(16, 256, 2), (1, 4096, 8), (1000, 512, 6)])
def test_combine_shared_bit_exact_given_oracle_inputs(T, H, k):
    rng = np.random.default_rng(1)
    y = (rng.standard_normal((T * k, H)) * 10).astype(np.float32)
    ys = (rng.standard_normal((T, H)) * 10).astype(np.float32)
    w = rng.random((T, k)).astype(np.float32)
    inv = rng.permutation(T * k).astype(np.int32)
    out = torch.empty((T, H), dtype=torch.bfloat16, device="cuda")
    moe.moe_combine_shared(dev(y), dev(inv), dev(w), dev(ys), moe.shape(T, H, 128, 8, k), out)
    torch.cuda.synchronize()
    ref, _ = O.combine_shared(y, inv, w, ys)
    assert np.array_equal(bits(out), ref)


def _run_block(wl, x, wr, routed, shared, rdev=None):
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    ws = moe.alloc_block_workspace(sh)
    out = torch.full((wl.T, wl.H), float("nan"), dtype=torch.bfloat16, device="cuda")
    ids = torch.empty((wl.T, wl.k), dtype=torch.int32, device="cuda")
    w = torch.empty((wl.T, wl.k), dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    rdev = rdev if rdev is not None else tuple(dev(a) for a in routed)
    sdev = tuple(dev(a) for a in shared)
    xd, wrd = dev(x), dev(wr)
    for _ in range(2):   # twice on one workspace
        moe.moe_ffn_block(xd, wrd, rdev, sdev, sh, out, ids, w, st, ws)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
    logits = ws[:wl.T * wl.E * 4].view(torch.float32).reshape(wl.T, wl.E).cpu().numpy()   # the block keeps them first in ws
    return out, ids.cpu().numpy(), w.cpu().numpy(), logits


def _check_block(wl, seed, routed=None, rdev=None, sample=None):
    routed = routed if routed is not None else inputs.make_expert_weights(wl.H, wl.I, wl.E, seed=0)
    shared = inputs.make_expert_weights(wl.H, wl.I, 1, seed=21)
    x, wr = inputs.make_x(wl.T, wl.H, seed), _router_weights(wl.E, wl.H, seed + 1)
    out, ids, w, logits = _run_block(wl, x, wr, routed, shared, rdev)
    ref_logits = O.router_logits(x, wr)
    assert np.linalg.norm(logits - ref_logits) / np.linalg.norm(ref_logits) < 1e-5
    # everything after the projection is checked on the logits the GPU computed (a last-bit difference in a logit may
    # legitimately change a near-tie of the Top-k)
    if sample is None:
        r = O.ffn_block(x, wr, *routed, *shared, wl.k, logits=logits)
        assert np.array_equal(ids, r["ids"]) and np.array_equal(w.view(np.uint32), r["w"].view(np.uint32))
        return check_out(bits(out), r["out"], r["out_f32"], wl.name)
    rids, rw, _ = O.route(logits, wl.k)
    assert np.array_equal(ids, rids) and np.array_equal(w.view(np.uint32), rw.view(np.uint32))
    tok = np.array(sample, np.int32)
    rt = O.forward_tokens(logits, x, *routed, wl.k, tok)
    ys = O.shared_expert(np.ascontiguousarray(x[tok]), *shared)
    want_f32 = (rt["out_f32"].astype(np.float64) + ys.astype(np.float64)).astype(np.float32)
    got = bits(out[torch.from_numpy(tok.astype(np.int64)).cuda()])
    return check_out(got, inputs.f32_to_bf16_bits(want_f32), want_f32, wl.name)


@pytest.mark.parametrize("T,H,I,E,k", [
    (16, 256, 128, 8, 2),      # streaming expert kernel for both calls
    (4, 512, 512, 8, 2),       # decode-sized kernel, router by warps
    (24, 1024, 512, 32, 6),    # decode-sized routed call, shared call of 24 rows on one expert
    (512, 512, 512, 8, 2),     # prefill-sized routed call, router GEMM
    (1100, 512, 512, 16, 6),   # prefill-sized kernel for both calls
    (1, 512, 512, 8, 2),       # one token: the router projection, then one launch with the shared expert as a third slot
    (1, 1024, 512, 16, 6),
    (1, 512, 1024, 4, 4)])
def test_ffn_block_small_shapes(T, H, I, E, k):
    _check_block(inputs.Workload("block", T, H, I, E, k), seed=5)
    if T == 1:
        assert moe.moe_last_kernel_name() == "block_one_launch_mxf4_pair_split_k"


@pytest.mark.parametrize("name", ["decode_c1", "decode_c64"])
def test_ffn_block_production_decode(name):
    wl = inputs.WORKLOADS[name]
    _check_block(wl, seed=7)
    if wl.T == 1:   # 9 slots x 16 CTAs on 144 of the 148 SMs
        assert moe.moe_last_kernel_name() == "block_one_launch_mxf4_pair_split_k"


def test_ffn_block_prefill_8k_sampled():
    wl = inputs.WORKLOADS["prefill_8k"]
    rng = np.random.default_rng(0)
    _check_block(wl, seed=9, sample=sorted(set([0, wl.T - 1] + rng.integers(0, wl.T, 30).tolist())))
