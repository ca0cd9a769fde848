"""GPU parity: every C-ABI call against the CPU oracle on the same seeded inputs.

Bit-exact: routing ids, routing weights, offsets, perm, inv_perm, x_perm, and moe_combine given the
oracle's y and w.  Within the stated tolerance: y_perm and out through the GPU expert FFN
(rel-Frobenius <= 5e-3 and max|diff| <= 2e-2 * rms(reference) on bf16 outputs).
"""
import numpy as np
import pytest
import torch

from _gpu_util import assert_same_up_to_rounding, bits, check_out, check_y, dev, run_layer, weights_dev
from oracle import moe_oracle as O
from paper_2609_15627_b200 import inputs, moe

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    moe.lib()


@pytest.fixture(scope="module")
def prod_weights():
    """Production-shape expert weights (H=4096, I=2048, E=256), host and device."""
    w = inputs.make_expert_weights(4096, 2048, 256, seed=0)
    return w, tuple(dev(a) for a in w)


# ---- moe_route --------------------------------------------------------------------------------

def _gpu_route(logits, k):
    T, E = logits.shape
    ids = torch.empty((T, k), dtype=torch.int32, device="cuda")
    w = torch.empty((T, k), dtype=torch.float32, device="cuda")
    off = torch.empty(E + 1, dtype=torch.int32, device="cuda")
    ws = torch.empty(1 << 16, dtype=torch.uint8, device="cuda")
    moe.moe_route(dev(logits), k, ids, w, off, ws)
    torch.cuda.synchronize()
    return ids.cpu().numpy(), w.cpu().numpy(), off.cpu().numpy()


@pytest.mark.parametrize("T,E,k,seed,skew", [
    (16, 8, 2, 0, False), (1, 256, 8, 0, False), (64, 256, 8, 0, False), (128, 256, 8, 1, False),
    (129, 256, 8, 2, False), (777, 256, 6, 3, False), (8192, 256, 8, 0, False), (32768, 256, 8, 0, True),
    (50, 1024, 32, 4, False), (33, 40, 32, 5, False), (9, 100, 1, 6, False), (300, 7, 3, 7, False)])
def test_route_bit_exact(T, E, k, seed, skew):
    l = inputs.make_logits(T, E, seed=seed, skew=skew)
    ids, w, off = _gpu_route(l, k)
    rids, rw, roff = O.route(l, k)
    assert np.array_equal(ids, rids)
    assert np.array_equal(w.view(np.uint32), rw.view(np.uint32))
    assert np.array_equal(off, roff)


def test_route_ties_and_signed_zero():
    E, k = 256, 8
    rng = np.random.default_rng(5)
    l = rng.integers(-3, 4, size=(300, E)).astype(np.float32) * 0.25  # many exact ties
    l[0, :] = 1.5
    l[1, ::2] = 0.0
    l[1, 1::2] = -0.0
    ids, w, off = _gpu_route(l, k)
    rids, rw, roff = O.route(l, k)
    assert np.array_equal(ids, rids) and np.array_equal(off, roff)
    assert np.array_equal(w.view(np.uint32), rw.view(np.uint32))
    assert ids[0].tolist() == list(range(k)) and ids[1].tolist() == list(range(k))


def test_route_nonfinite_logits_still_give_distinct_valid_ids():
    l = inputs.make_logits(64, 256, seed=9)
    l[3, 10] = np.nan
    l[4, :] = np.nan
    l[5, 7] = np.inf
    l[6, :] = -np.inf
    ids, _, off = _gpu_route(l, 8)
    assert ids.min() >= 0 and ids.max() < 256
    assert all(len(set(r)) == 8 for r in ids.tolist())
    assert off[-1] == 64 * 8


# ---- moe_permute ------------------------------------------------------------------------------

@pytest.mark.parametrize("T,H,E,k,seed,skew", [
    (16, 256, 8, 2, 0, False), (1, 4096, 256, 8, 0, False), (64, 4096, 256, 8, 0, False),
    (512, 256, 256, 8, 1, False), (513, 128, 256, 8, 2, False), (4100, 128, 64, 6, 3, True),
    (8192, 128, 256, 8, 0, False), (5000, 256, 1024, 3, 4, False)])
def test_permute_bit_exact(T, H, E, k, seed, skew):
    l = inputs.make_logits(T, E, seed=seed, skew=skew)
    x = inputs.make_x(T, H, seed=seed)
    ids, w, off = O.route(l, k)
    rx, rperm, rinv = O.permute(x, ids, off)
    sh = moe.shape(T, H, 128, E, k)
    buf = moe.LayerBuffers(sh)
    moe.moe_permute(dev(x), dev(ids), dev(off), sh, buf.x_perm, buf.perm, buf.inv_perm, buf.ws)
    torch.cuda.synchronize()
    assert np.array_equal(buf.perm.cpu().numpy(), rperm)
    assert np.array_equal(buf.inv_perm.cpu().numpy(), rinv)
    assert np.array_equal(bits(buf.x_perm), rx)


def test_permute_all_slots_to_one_expert():
    T, H, E, k = 3000, 128, 16, 2
    l = np.zeros((T, E), np.float32)
    l[:, 5] = 2.0
    l[:, 11] = 1.0
    x = inputs.make_x(T, H, seed=1)
    ids, w, off = O.route(l, k)
    rx, rperm, rinv = O.permute(x, ids, off)
    sh = moe.shape(T, H, 128, E, k)
    buf = moe.LayerBuffers(sh)
    moe.moe_permute(dev(x), dev(ids), dev(off), sh, buf.x_perm, buf.perm, buf.inv_perm, buf.ws)
    torch.cuda.synchronize()
    assert np.array_equal(buf.perm.cpu().numpy(), rperm) and np.array_equal(bits(buf.x_perm), rx)


# ---- moe_combine ------------------------------------------------------------------------------

@pytest.mark.parametrize("T,H,k", [(16, 256, 2), (1, 4096, 8), (64, 4096, 8), (1000, 512, 6), (7, 128, 1)])
def test_combine_bit_exact_given_oracle_inputs(T, H, k):
    rng = np.random.default_rng(T)
    S = T * k
    y = (rng.standard_normal((S, H)) * 19).astype(np.float32)
    inv = rng.permutation(S).astype(np.int32)
    w = rng.random((T, k)).astype(np.float32)
    w /= w.sum(axis=1, keepdims=True)
    rout, rout32 = O.combine(y, inv, w)
    sh = moe.shape(T, H, 128, max(k, 8), k)
    out = torch.empty((T, H), dtype=torch.bfloat16, device="cuda")
    moe.moe_combine(dev(y), dev(inv), dev(w), sh, out)
    torch.cuda.synchronize()
    assert np.array_equal(bits(out), rout)


# ---- moe_expert_ffn ----------------------------------------------------------------------------

def _gpu_ffn(wl, x_perm, off, w):
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    buf = moe.LayerBuffers(sh)
    moe.moe_expert_ffn(dev(x_perm), dev(off), *[dev(a) for a in w], sh, buf.y_perm, buf.status, buf.ws)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    return buf.y_perm.cpu().numpy()


def _staged_inputs(wl, seed, w=None):
    d = inputs.make_workload(wl, seed=seed) if w is None else None
    logits = inputs.make_logits(wl.T, wl.E, seed, wl.skew)
    x = inputs.make_x(wl.T, wl.H, seed)
    if w is None:
        w = (d["w13"], d["s13"], d["w2"], d["s2"])
    ids, tw, off = O.route(logits, wl.k)
    x_perm, perm, inv = O.permute(x, ids, off)
    return logits, x, w, ids, tw, off, x_perm, perm, inv


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_ffn_tiny_against_oracle(seed):
    wl = inputs.WORKLOADS["tiny"]
    logits, x, w, ids, tw, off, x_perm, perm, inv = _staged_inputs(wl, seed)
    y = _gpu_ffn(wl, x_perm, off, w)
    ry = O.expert_ffn(x_perm, off, *w, wl.k)
    check_y(y, ry, "tiny seed %d" % seed)


def test_ffn_nonconstant_scales_and_fingerprint_codes():
    # index-dependent scale bytes and row-fingerprint codes: a scale or row read from the wrong
    # place, or a permuted tile, changes the result far beyond the tolerance
    wl = inputs.Workload("fixture", 24, 512, 256, 4, 2)
    w13 = inputs.fingerprint_codes(2 * wl.I, wl.H, wl.E)
    w2 = inputs.fingerprint_codes(wl.H, wl.I, wl.E)
    s13 = inputs.index_scales(2 * wl.I, wl.H, wl.E, lo=116, span=8)
    s2 = inputs.index_scales(wl.H, wl.I, wl.E, lo=118, span=7)
    w = (w13, s13, w2, s2)
    logits, x, w, ids, tw, off, x_perm, perm, inv = _staged_inputs(wl, 3, w)
    y = _gpu_ffn(wl, x_perm, off, w)
    ry = O.expert_ffn(x_perm, off, *w, wl.k)
    check_y(y, ry, "fixture")


def test_ffn_every_code_and_scale_byte_exactly():
    # one non-zero weight per matrix row: each stage is a single product, so dequantisation is
    # checked value by value (all 16 codes, scale bytes from 2^-127 up to 2^1)
    T, H, I, E, k = 8, 128, 128, 1, 1
    wl = inputs.Workload("codes", T, H, I, E, k)
    x = inputs.make_x(T, H, seed=2)
    off = np.array([0, T], np.int32)
    for sb2 in (90, 110, 119, 122, 127, 128):
        w13 = np.zeros((E, 2 * I, H // 2), np.uint8)
        s13 = np.full((E, 2 * I, H // 32), 127, np.uint8)
        w2 = np.zeros((E, H, I // 2), np.uint8)
        s2 = np.full((E, H, I // 32), sb2, np.uint8)
        for i in range(I):
            w13[0, i, i // 2] = 0x2 << (4 * (i & 1))            # gate: 1.0 * x[i]
            w13[0, I + i, i // 2] = 0x4 << (4 * (i & 1))        # up:   2.0 * x[i]
        for n in range(H):
            code = n % 16
            i = (5 * n + 3) % I
            w2[0, n, i // 2] = code << (4 * (i & 1))
        y = _gpu_ffn(wl, x, off, (w13, s13, w2, s2))
        ry, ract = O.expert_ffn(x, off, w13, s13, w2, s2, k, want_act=True)
        # the activations may differ in the last bf16 bit (different exp), so compare y against
        # its own definition from the oracle's table: y[n] = value(code) * 2^(sb2-127) * act
        with np.errstate(over="ignore"):
            close = np.isclose(y, ry, rtol=2.0 ** -6, atol=0.0)
        assert close.all(), sb2
        for n in range(H):
            if n % 16 in (0, 8):
                assert np.all(y[:, n] == 0.0)
    # and the gate/up side: scale bytes on w13, identity-like w2
    for sb1 in (100, 119, 122, 127, 128):
        w13 = np.zeros((E, 2 * I, H // 2), np.uint8)
        s13 = np.full((E, 2 * I, H // 32), sb1, np.uint8)
        w2 = np.zeros((E, H, I // 2), np.uint8)
        s2 = np.full((E, H, I // 32), 127, np.uint8)
        for i in range(I):
            h = (3 * i + 1) % H
            w13[0, i, h // 2] = (i % 16) << (4 * (h & 1))
            w13[0, I + i, i // 2] = 0x2 << (4 * (i & 1))
        for n in range(H):
            w2[0, n, n // 2] = 0x2 << (4 * (n & 1))             # y[n] = act[n]
        y = _gpu_ffn(wl, x, off, (w13, s13, w2, s2))
        ry = O.expert_ffn(x, off, w13, s13, w2, s2, k)
        assert np.allclose(y, ry, rtol=2.0 ** -6, atol=1e-30), sb1


def test_ffn_zero_codes_give_zero():
    wl = inputs.WORKLOADS["tiny"]
    logits, x, w, ids, tw, off, x_perm, perm, inv = _staged_inputs(wl, 0)
    w13 = np.zeros_like(w[0])
    w13[:, :, ::2] = 0x80
    w2 = np.full_like(w[2], 0x08)
    y = _gpu_ffn(wl, x_perm, off, (w13, w[1], w2, w[3]))
    assert np.all(y == 0.0)


def test_ffn_w2_scale_plus_one_doubles_exactly():
    wl = inputs.WORKLOADS["tiny"]
    logits, x, w, ids, tw, off, x_perm, perm, inv = _staged_inputs(wl, 4)
    y1 = _gpu_ffn(wl, x_perm, off, w)
    y2 = _gpu_ffn(wl, x_perm, off, (w[0], w[1], w[2], w[3] + 1))
    assert np.array_equal(y2, 2.0 * y1)


@pytest.mark.parametrize("T,E,k,hot", [(40, 4, 2, True), (96, 8, 1, True), (37, 8, 3, False)])
def test_ffn_many_rows_per_expert_and_empty_experts(T, E, k, hot):
    # experts with more than 8 rows (several token tiles), ragged tails and experts with no rows
    wl = inputs.Workload("ragged", T, 256, 128, E, k)
    w = inputs.make_expert_weights(wl.H, wl.I, wl.E, seed=7)
    logits = inputs.make_logits(T, E, seed=7)
    if hot:
        logits[:, 1] += 6.0
        logits[:, E - 1] -= 50.0  # never chosen
    x = inputs.make_x(T, wl.H, seed=7)
    ids, tw, off = O.route(logits, k)
    assert np.diff(off).max() > 8
    x_perm, perm, inv = O.permute(x, ids, off)
    y = _gpu_ffn(wl, x_perm, off, w)
    ry = O.expert_ffn(x_perm, off, *w, k)
    check_y(y, ry, "ragged")


def test_ffn_mutations_and_replay_determinism():
    # seeded mutations of inputs, routes, weights and scales; repeated launches are bit-identical
    wl = inputs.WORKLOADS["tiny"]
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    buf = moe.LayerBuffers(sh)
    rng = np.random.default_rng(0)
    for m in range(100):  # the size of the paper's component fixture: 100 mutations per shape
        d = inputs.make_workload(wl, seed=100 + m)
        w = [d["w13"].copy(), d["s13"].copy(), d["w2"].copy(), d["s2"].copy()]
        w[1].reshape(-1)[rng.integers(0, w[1].size, 64)] = rng.integers(110, 129, 64)
        w[3].reshape(-1)[rng.integers(0, w[3].size, 64)] = rng.integers(110, 129, 64)
        w[0].reshape(-1)[rng.integers(0, w[0].size, 64)] = rng.integers(0, 256, 64)
        w[2].reshape(-1)[rng.integers(0, w[2].size, 64)] = rng.integers(0, 256, 64)
        r = O.forward_staged(d["logits"], d["x"], *w, wl.k)
        wdev = tuple(dev(a) for a in w)
        out = moe.moe_layer(dev(d["logits"]), dev(d["x"]), wdev, buf)
        torch.cuda.synchronize()
        first = bits(out).copy()
        check_out(first, r["out"], r["out_f32"], "mutation %d" % m)
        assert np.array_equal(buf.topk_ids.cpu().numpy(), r["ids"])
        for _ in range(5):
            out = moe.moe_layer(dev(d["logits"]), dev(d["x"]), wdev, buf)
            torch.cuda.synchronize()
            assert np.array_equal(bits(out), first)


@pytest.mark.parametrize("one_call", [True, False])
def test_replay_determinism_1000_graph_replays(one_call, prod_weights):
    """The paper's fixture replays a captured graph 1000 times and checks every replay.  Here: the single-token
    production call - as moe_forward (one launch, CTAs handing work over through global counters) and as the four
    calls - captured once and replayed 1000 times; every replay's output is compared on the device with the first."""
    wl = inputs.WORKLOADS["decode_c1"]
    (w13, s13, w2, s2), wdev = prod_weights
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    ws = moe.alloc_forward_workspace(sh)
    buf = moe.LayerBuffers(sh)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    lg, x = dev(inputs.make_logits(wl.T, wl.E, 77)), dev(inputs.make_x(wl.T, wl.H, 77))
    out = buf.out

    def call(stream=None):
        if one_call:
            moe.moe_forward(lg, x, *wdev, sh, out, None, None, st, ws, stream)
        else:
            moe.moe_layer(lg, x, wdev, buf, stream)

    call()
    torch.cuda.synchronize()
    assert (moe.moe_last_kernel_name() in _ONE_KERNELS) == one_call
    first = out.view(torch.int16).clone()
    r = O.forward_staged(lg.cpu().numpy(), bits(x), w13, s13, w2, s2, wl.k)
    check_out(bits(out), r["out"], r["out_f32"], "replay source")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        call()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        call()
    bad = torch.zeros((), dtype=torch.int32, device="cuda")
    for _ in range(1000):
        out.zero_()
        g.replay()
        bad += (out.view(torch.int16) != first).any().int()
    torch.cuda.synchronize()
    assert int(bad.item()) == 0 and int(st.item()) == 0 and int(buf.status.item()) == 0


# ---- the five workloads end to end ----------------------------------------------------------------

def _check_layer_full(wl, d, wdev):
    buf, out = run_layer(wl, d, wdev)
    r = O.forward_staged(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"], wl.k)
    assert np.array_equal(buf.topk_ids.cpu().numpy(), r["ids"])
    assert np.array_equal(buf.topk_w.cpu().numpy().view(np.uint32), r["w"].view(np.uint32))
    assert np.array_equal(buf.expert_offsets.cpu().numpy(), r["offsets"])
    assert np.array_equal(buf.perm.cpu().numpy(), r["perm"])
    assert np.array_equal(buf.inv_perm.cpu().numpy(), r["inv_perm"])
    assert np.array_equal(bits(buf.x_perm), r["x_perm"])
    check_y(buf.y_perm.cpu().numpy(), r["y_perm"], wl.name)
    return check_out(bits(out), r["out"], r["out_f32"], wl.name)


def test_layer_tiny():
    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl, seed=0)
    _check_layer_full(wl, d, None)


@pytest.mark.parametrize("T,H,I,E,k,kernel", [
    (8, 1024, 512, 32, 6, "ffn_native_mxf4_block_scaled"),   # the paper's own top-k (6), decode-sized
    (24, 512, 256, 16, 6, "ffn_native_mxf4_block_scaled"),   # top-6 with I = 256, the paper's TP8 shard of I
    (24, 512, 384, 16, 6, "ffn_stream_bulk_ring_mma16816"),  # an I the tensor-core kernels do not take
    (256, 512, 512, 8, 6, "ffn_umma_tcgen05_grouped"),       # top-6, prefill-sized
])
def test_layer_full_with_top6(T, H, I, E, k, kernel):
    wl = inputs.Workload("top6", T, H, I, E, k)
    d = inputs.make_workload(wl, seed=3)
    _check_layer_full(wl, d, None)   # `kernel`: the expert-FFN variant this shape selects (see the kernel-choice test)


@pytest.mark.parametrize("name", ["decode_c1", "decode_c64"])
def test_layer_decode_full(name, prod_weights):
    wl = inputs.WORKLOADS[name]
    (w13, s13, w2, s2), wdev = prod_weights
    d = dict(logits=inputs.make_logits(wl.T, wl.E, 0), x=inputs.make_x(wl.T, wl.H, 0), w13=w13, s13=s13, w2=w2, s2=s2)
    _check_layer_full(wl, d, wdev)


# ---- moe_forward: the whole layer as one call (one kernel launch for a handful of tokens) -------------------

_ONE_LAUNCH = "layer_one_launch_mxf4_block_scaled"       # the general one-launch kernel (up to 4 tokens)
_ONE_TOKEN = "layer_one_launch_mxf4_pair_split_k"         # one token: down projection split along K over pairs of CTAs
_ONE_KERNELS = (_ONE_LAUNCH, _ONE_TOKEN)


def _run_forward(wl, d, wdev, reps=1, force_one_launch=False):
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    ws = moe.alloc_forward_workspace(sh)
    out = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device="cuda")
    ids = torch.empty((wl.T, wl.k), dtype=torch.int32, device="cuda")
    w = torch.empty((wl.T, wl.k), dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    lg, x = dev(d["logits"]), dev(d["x"])
    for _ in range(reps):
        out.fill_(float("nan"))
        (moe.moe_debug_forward_one_launch if force_one_launch else moe.moe_forward)(lg, x, *wdev, sh, out, ids, w, st, ws)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        # the counter block is left clear for the next call
        assert int(ws[:moe.moe_forward_sync_bytes()].view(torch.int32).abs().sum().item()) == 0
    return out, ids, w, moe.moe_last_kernel_name()


def _check_forward(wl, d, wdev, one_launch, force_one_launch=False):
    wdev = wdev if wdev is not None else weights_dev(d)
    out, ids, w, kernel = _run_forward(wl, d, wdev, reps=3, force_one_launch=force_one_launch)
    assert (kernel in _ONE_KERNELS) == one_launch, kernel
    assert (kernel == _ONE_TOKEN) == (one_launch and wl.T == 1 and not force_one_launch), kernel
    # against the oracle: routing bit for bit, the output within the stated tolerance
    r = O.forward_staged(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"], wl.k)
    assert np.array_equal(ids.cpu().numpy(), r["ids"])
    assert np.array_equal(w.cpu().numpy().view(np.uint32), r["w"].view(np.uint32))
    check_out(bits(out), r["out"], r["out_f32"], wl.name)
    # against the four calls: the general kernel does the same arithmetic in the same order, so the same bits; the
    # one-token kernel adds the down projection's partial sums in another order
    buf, out4 = run_layer(wl, d, wdev)
    if kernel == _ONE_TOKEN:
        assert_same_up_to_rounding(bits(out), bits(out4), wl.name)
    else:
        assert np.array_equal(bits(out), bits(out4))


@pytest.mark.parametrize("T,H,I,E,k,one_launch", [
    (1, 512, 512, 8, 2, True), (1, 1024, 512, 16, 4, True), (1, 2048, 1024, 64, 8, True), (1, 1024, 512, 32, 6, True),
    (1, 512, 512, 4, 4, True),      # every expert touched
    (1, 512, 512, 32, 32, True),    # 32 slots
    (1, 512, 512, 1024, 8, True),   # the largest expert count
    (2, 1024, 512, 16, 4, False),   # more than one token: the four calls are faster
    (16, 256, 128, 8, 2, False),    # not a shape of the decode-sized expert kernel
    (64, 1024, 512, 32, 6, False)])
def test_forward_small_shapes(T, H, I, E, k, one_launch):
    wl = inputs.Workload("fwd", T, H, I, E, k)
    d = inputs.make_workload(wl, seed=5)
    _check_forward(wl, d, None, one_launch)


@pytest.mark.parametrize("T,H,I,E,k", [
    (2, 1024, 512, 16, 4), (2, 2048, 1024, 64, 8), (3, 1024, 512, 32, 6), (4, 512, 512, 8, 2), (4, 1024, 512, 32, 8),
    (2, 512, 512, 16, 16),          # 32 slots, every expert touched by both tokens
    (4, 2048, 1024, 8, 8),          # every expert touched by all four tokens
    (3, 512, 512, 4, 1)])
def test_one_launch_kernel_with_several_tokens(T, H, I, E, k):
    """moe_forward keeps the one-launch kernel for one token; the kernel itself takes up to four."""
    wl = inputs.Workload("fwd_n", T, H, I, E, k)
    d = inputs.make_workload(wl, seed=7)
    _check_forward(wl, d, None, True, force_one_launch=True)


def test_one_launch_kernel_refuses_what_it_cannot_take():
    for T, H, I, E, k in ((5, 512, 512, 8, 2), (2, 512, 512, 32, 32), (2, 512, 512, 512, 8), (2, 256, 128, 8, 2)):
        wl = inputs.Workload("fwd_no", T, H, I, E, k)
        d = inputs.make_workload(wl, seed=7)
        wdev = weights_dev(d)
        sh = moe.shape(T, H, I, E, k)
        ws = moe.alloc_forward_workspace(sh)
        out = torch.empty((T, H), dtype=torch.bfloat16, device="cuda")
        with pytest.raises(moe.MoeError, match="unsupported shape"):
            moe.moe_debug_forward_one_launch(dev(d["logits"]), dev(d["x"]), *wdev, sh, out, None, None, None, ws)


@pytest.mark.parametrize("T,k,seed,force", [(1, 8, 0, False), (1, 8, 1, False), (1, 6, 2, False), (2, 8, 0, False),
                                             (2, 6, 3, True), (3, 8, 5, True), (4, 8, 4, True)])
def test_forward_production_shape(T, k, seed, force, prod_weights):
    wl = inputs.Workload("fwd_prod", T, 4096, 2048, 256, k)
    (w13, s13, w2, s2), wdev = prod_weights
    d = dict(logits=inputs.make_logits(T, wl.E, seed), x=inputs.make_x(T, wl.H, seed), w13=w13, s13=s13, w2=w2, s2=s2)
    _check_forward(wl, d, wdev, T == 1 or force, force_one_launch=force)


def test_forward_tokens_sharing_experts():
    """Four tokens with the same logits: every touched expert gets all four rows."""
    wl = inputs.Workload("fwd_same", 4, 1024, 512, 16, 4)
    d = inputs.make_workload(wl, seed=6)
    d["logits"][:] = d["logits"][0]
    _check_forward(wl, d, None, True, force_one_launch=True)


def test_forward_without_routing_outputs_and_in_a_graph(prod_weights):
    """topk_ids / topk_w may be NULL; graph replays of several calls sharing one workspace give the eager result."""
    wl = inputs.WORKLOADS["decode_c1"]
    (w13, s13, w2, s2), wdev = prod_weights
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    ws = moe.alloc_forward_workspace(sh)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    batches = [(dev(inputs.make_logits(wl.T, wl.E, 40 + i)), dev(inputs.make_x(wl.T, wl.H, 40 + i))) for i in range(4)]
    outs = [torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device="cuda") for _ in batches]
    eager = []
    for (lg, x), o in zip(batches, outs):
        moe.moe_forward(lg, x, *wdev, sh, o, None, None, st, ws)
        torch.cuda.synchronize()
        eager.append(bits(o).copy())
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        moe.moe_forward(batches[0][0], batches[0][1], *wdev, sh, outs[0], None, None, st, ws, None)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for (lg, x), o in zip(batches, outs):
            moe.moe_forward(lg, x, *wdev, sh, o, None, None, st, ws, None)
    for _ in range(3):
        for o in outs:
            o.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        for o, e in zip(outs, eager):
            assert np.array_equal(bits(o), e)


def test_forward_with_a_workspace_that_was_never_cleared():
    """The one-launch kernel finds its two untouched words non-zero, reports it and does nothing; after a clear the
    same workspace works."""
    wl = inputs.Workload("fwd_dirty", 1, 1024, 512, 16, 4)
    d = inputs.make_workload(wl, seed=9)
    wdev = weights_dev(d)
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    ws = moe.alloc_forward_workspace(sh)
    ws.fill_(0x5A)
    out = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    moe.moe_forward(dev(d["logits"]), dev(d["x"]), *wdev, sh, out, None, None, st, ws)
    torch.cuda.synchronize()
    assert moe.moe_last_kernel_name() in _ONE_KERNELS
    assert int(st.item()) == 3                      # MOE_ERR_WORKSPACE
    assert int(out.view(torch.int16).abs().sum().item()) == 0
    ws[:moe.moe_forward_sync_bytes()].zero_()
    st.zero_()
    moe.moe_forward(dev(d["logits"]), dev(d["x"]), *wdev, sh, out, None, None, st, ws)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    buf, out4 = run_layer(wl, d, wdev)
    assert_same_up_to_rounding(bits(out), bits(out4))


def test_forward_bounded_wait_runs_out_and_the_next_call_works():
    """A wait that nothing can satisfy: the count of stored partial sums of the first column tile (word 1024 of the
    counter block) starts far below zero, so it never reaches its target.  The wait gives up after its limit (about two seconds), the
    kernel reports MOE_ERR_TIMEOUT through the status word and runs to its end, the last CTA clears the block as
    always, and the same workspace then serves a correct call."""
    wl = inputs.Workload("fwd_wait", 1, 1024, 512, 16, 4)
    d = inputs.make_workload(wl, seed=10)
    wdev = weights_dev(d)
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    ws = moe.alloc_forward_workspace(sh)
    ws[:moe.moe_forward_sync_bytes()].view(torch.int32)[1024] = -100000
    out = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    lg, x = dev(d["logits"]), dev(d["x"])
    moe.moe_forward(lg, x, *wdev, sh, out, None, None, st, ws)
    torch.cuda.synchronize()
    assert moe.moe_last_kernel_name() in _ONE_KERNELS
    assert int(st.item()) == 5                      # MOE_ERR_TIMEOUT
    assert int(ws[:moe.moe_forward_sync_bytes()].view(torch.int32).abs().sum().item()) == 0
    st.zero_()
    moe.moe_forward(lg, x, *wdev, sh, out, None, None, st, ws)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    buf, out4 = run_layer(wl, d, wdev)
    assert_same_up_to_rounding(bits(out), bits(out4))


def test_forward_bounded_wait_runs_out_without_a_status_word():
    """The same run-out with status_word = NULL: the kernels then report to a word inside the library, so that after the
    first wait has given up (about two seconds) every later wait of the grid drains after a short spin instead of
    waiting out its own two seconds - the call ends within seconds, nothing is reported (the caller asked for nothing),
    the counter block is left clear, and the next call, again without a status word, is correct."""
    import time
    wl = inputs.Workload("fwd_wait_null", 1, 1024, 512, 16, 4)
    d = inputs.make_workload(wl, seed=11)
    wdev = weights_dev(d)
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    ws = moe.alloc_forward_workspace(sh)
    ws[:moe.moe_forward_sync_bytes()].view(torch.int32)[1024] = -100000
    out = torch.zeros((wl.T, wl.H), dtype=torch.bfloat16, device="cuda")
    lg, x = dev(d["logits"]), dev(d["x"])
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    moe.moe_forward(lg, x, *wdev, sh, out, None, None, None, ws)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 8.0
    assert moe.moe_last_kernel_name() in _ONE_KERNELS
    assert int(ws[:moe.moe_forward_sync_bytes()].view(torch.int32).abs().sum().item()) == 0
    moe.moe_forward(lg, x, *wdev, sh, out, None, None, None, ws)
    torch.cuda.synchronize()
    buf, out4 = run_layer(wl, d, wdev)
    assert_same_up_to_rounding(bits(out), bits(out4))
    # the four calls without a status word, on every expert-FFN variant (decode-sized, prefill-sized, streaming)
    for T, H, I, E, k in [(4, 512, 512, 8, 2), (512, 512, 512, 8, 2), (16, 256, 128, 8, 2)]:
        wl2 = inputs.Workload("null_status", T, H, I, E, k)
        d2 = inputs.make_workload(wl2, seed=12)
        w2dev = weights_dev(d2)
        buf2, want = run_layer(wl2, d2, w2dev)
        want = bits(want).copy()
        moe.moe_expert_ffn(buf2.x_perm, buf2.expert_offsets, *w2dev, buf2.sh, buf2.y_perm, None, buf2.ws)
        moe.moe_combine(buf2.y_perm, buf2.inv_perm, buf2.topk_w, buf2.sh, buf2.out)
        torch.cuda.synchronize()
        assert np.array_equal(bits(buf2.out), want)


def test_forward_host_uses_it():
    """moe_forward_host clears the counter block itself: a workspace full of ones still gives the layer's result."""
    wl = inputs.Workload("fwd_host", 1, 1024, 512, 16, 4)
    d = inputs.make_workload(wl, seed=8)
    wdev = weights_dev(d)
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    ws = moe.alloc_workspace(sh, host_path=True)
    ws.fill_(1)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    lh = torch.from_numpy(d["logits"]).pin_memory()
    xh = torch.from_numpy(d["x"].view(np.int16)).pin_memory()
    oh = torch.empty((wl.T, wl.H), dtype=torch.int16).pin_memory()
    moe.moe_forward_host(lh, xh, *wdev, sh, oh, st, ws)
    assert int(st.item()) == 0 and moe.moe_last_kernel_name() in _ONE_KERNELS
    buf, out4 = run_layer(wl, d, wdev)
    assert_same_up_to_rounding(oh.numpy().view(np.uint16), bits(out4))


def test_forward_host_sequence_of_shapes_and_pageable_buffers():
    """The host entry point on one thread: a batch whose logits fill the staging buffer, then a single token (whose
    counter block's zeros travel behind 1 KB of logits in the same buffer), twice, then the same from pageable memory
    (no page-locked buffer for the kernel to read or write in place)."""
    big = inputs.Workload("host_big", 64, 512, 512, 256, 4)     # 64 KB of logits
    one = inputs.Workload("host_one", 1, 1024, 512, 256, 4)
    for pinned in (True, False):
        for wl in (big, one, big, one):
            d = inputs.make_workload(wl, seed=11)
            wdev = weights_dev(d)
            sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
            ws = moe.alloc_workspace(sh, host_path=True)
            ws.fill_(0x5A)
            st = torch.zeros(1, dtype=torch.int32, device="cuda")
            lh, xh = torch.from_numpy(d["logits"].copy()), torch.from_numpy(d["x"].view(np.int16).copy())
            oh = torch.zeros((wl.T, wl.H), dtype=torch.int16)
            if pinned:
                lh, xh, oh = lh.pin_memory(), xh.pin_memory(), oh.pin_memory()
            moe.moe_forward_host(lh, xh, *wdev, sh, oh, st, ws)
            assert int(st.item()) == 0
            buf, out4 = run_layer(wl, d, wdev)
            assert_same_up_to_rounding(oh.numpy().view(np.uint16), bits(out4))


# ---- moe_prepack and the calls that take its result ------------------------------------------------------

def _tiles(a, tile_bytes):
    """[R, B] bytes -> tiles of [128 rows][tile_bytes], tile (row // 128, byte // tile_bytes), flattened in that order."""
    R, B = a.shape
    return a.reshape(R // 128, 128, B // tile_bytes, tile_bytes).transpose(0, 2, 1, 3).ravel()


def _align(n, a=256):
    return (n + a - 1) // a * a


@pytest.mark.parametrize("H,I,E,tiled", [(1024, 512, 4, True), (512, 1536, 3, True), (256, 128, 8, False), (512, 384, 2, False)])
def test_prepack_layout(H, I, E, tiled):
    w13, s13, w2, s2 = inputs.make_expert_weights(H, I, E, seed=11)
    sh = moe.shape(4, H, I, E, 1)
    packed = moe.moe_prepack(dev(w13), dev(s13), dev(w2), dev(s2), sh)
    torch.cuda.synchronize()
    got = packed.cpu().numpy()
    parts = [(w13.reshape(E * 2 * I, H // 2), 128), (s13.reshape(E * 2 * I, H // 32), 16),
             (w2.reshape(E * H, I // 2), 128), (s2.reshape(E * H, I // 32), 16)]
    off = 0
    for a, tb in parts:
        want = _tiles(a, tb) if tiled else a.ravel()
        assert np.array_equal(got[off:off + want.size], want)
        off += _align(want.size)
    assert moe.moe_prepack_bytes(sh) == off == got.size


@pytest.mark.parametrize("T,H,I,E,k,same_kernel", [
    (8, 1024, 512, 32, 6, True),      # decode-sized kernel
    (3, 512, 512, 8, 2, True),
    (256, 512, 512, 8, 6, True),      # prefill-sized kernel
    (300, 1024, 1024, 4, 4, True),
    (64, 512, 512, 2, 2, False),      # raw: row-streaming kernel; packed: grouped GEMM
    (16, 256, 128, 8, 2, True),       # no tiled layout for this shape: plain copy, same kernel
])
def test_expert_ffn_packed(T, H, I, E, k, same_kernel):
    wl = inputs.Workload("packed", T, H, I, E, k)
    d = inputs.make_workload(wl, seed=12)
    wdev = weights_dev(d)
    buf, out = run_layer(wl, d, wdev)
    sh = buf.sh
    raw_kernel_y = buf.y_perm.clone()
    packed = moe.moe_prepack(*wdev, sh)
    y = torch.empty_like(buf.y_perm)
    moe.moe_expert_ffn(buf.x_perm, buf.expert_offsets, *wdev, sh, raw_kernel_y, buf.status, buf.ws)
    k_raw = moe.moe_last_kernel_name()
    moe.moe_expert_ffn_packed(buf.x_perm, buf.expert_offsets, packed, sh, y, buf.status, buf.ws)
    k_packed = moe.moe_last_kernel_name()
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    assert (k_raw == k_packed) == same_kernel, (k_raw, k_packed)
    r = O.forward_staged(d["logits"], d["x"], d["w13"], d["s13"], d["w2"], d["s2"], wl.k)
    check_y(y.cpu().numpy(), r["y_perm"], wl.name)
    if same_kernel:
        assert torch.equal(y.view(torch.int32), raw_kernel_y.view(torch.int32))


@pytest.mark.parametrize("T,k,seed", [(1, 8, 0), (2, 6, 1), (64, 8, 2)])
def test_forward_packed_production_shape(T, k, seed, prod_weights):
    wl = inputs.Workload("fwd_packed", T, 4096, 2048, 256, k)
    (w13, s13, w2, s2), wdev = prod_weights
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    packed = moe.moe_prepack(*wdev, sh)
    lg, x = dev(inputs.make_logits(T, wl.E, seed)), dev(inputs.make_x(T, wl.H, seed))
    ws = moe.alloc_forward_workspace(sh)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out_raw = torch.empty((T, wl.H), dtype=torch.bfloat16, device="cuda")
    out_packed = torch.empty_like(out_raw)
    ids = torch.empty((T, k), dtype=torch.int32, device="cuda")
    w = torch.empty((T, k), dtype=torch.float32, device="cuda")
    moe.moe_forward(lg, x, *wdev, sh, out_raw, None, None, st, ws)
    k_raw = moe.moe_last_kernel_name()
    moe.moe_forward_packed(lg, x, packed, sh, out_packed, ids, w, st, ws)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and moe.moe_last_kernel_name() == k_raw
    assert (k_raw in _ONE_KERNELS) == (T == 1)
    assert torch.equal(out_raw.view(torch.int16), out_packed.view(torch.int16))
    d = dict(logits=lg.cpu().numpy(), x=bits(x), w13=w13, s13=s13, w2=w2, s2=s2)
    r = O.forward_staged(d["logits"], d["x"], w13, s13, w2, s2, k)
    assert np.array_equal(ids.cpu().numpy(), r["ids"])
    check_out(bits(out_packed), r["out"], r["out_f32"], wl.name)
    # and through the host-buffer call
    ws_h = moe.alloc_workspace(sh, host_path=True)
    oh = torch.empty((T, wl.H), dtype=torch.int16).pin_memory()
    moe.moe_forward_host_packed(lg.cpu().pin_memory(), x.view(torch.int16).cpu().pin_memory(), packed, sh, oh, st, ws_h)
    assert int(st.item()) == 0
    assert np.array_equal(oh.numpy().view(np.uint16), bits(out_packed))


def test_forward_packed_on_the_benchmark_batches(prod_weights):
    """decode_c1 as bench.py runs it: the 32 seeded batches of its cycle through moe_forward_packed back to back on one
    workspace (the one-launch kernel), each compared with the four calls on the row-layout weights (equal up to rounding flips), and
    the first and last with the oracle."""
    wl = inputs.WORKLOADS["decode_c1"]
    (w13, s13, w2, s2), wdev = prod_weights
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    packed = moe.moe_prepack(*wdev, sh)
    ws = moe.alloc_forward_workspace(sh)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    batches = [(inputs.make_logits(wl.T, wl.E, 7000 + i), inputs.make_x(wl.T, wl.H, 7000 + i)) for i in range(32)]
    dev_batches = [(dev(l), dev(x)) for l, x in batches]
    outs = [torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device="cuda") for _ in batches]
    for (lg, x), o in zip(dev_batches, outs):
        moe.moe_forward_packed(lg, x, packed, sh, o, None, None, st, ws)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and moe.moe_last_kernel_name() in _ONE_KERNELS
    buf = moe.LayerBuffers(sh)
    for i, ((lg, x), o) in enumerate(zip(dev_batches, outs)):
        out4 = moe.moe_layer(lg, x, wdev, buf)
        torch.cuda.synchronize()
        assert_same_up_to_rounding(bits(o), bits(out4), "batch %d" % i)
    for i in (0, 31):
        r = O.forward_staged(batches[i][0], batches[i][1], w13, s13, w2, s2, wl.k)
        check_out(bits(outs[i]), r["out"], r["out_f32"], "decode_c1 batch %d" % i)


def _pass_ranges(m, max_tok=256):
    """Row ranges [begin, end) inside an expert of m rows, as the prefill-sized kernel cuts them: the fewest passes of
    at most max_tok tokens, of equal size rounded up to 16."""
    n_pass = (m + max_tok - 1) // max_tok
    tp = (((m + n_pass - 1) // n_pass) + 15) // 16 * 16
    return [(p * tp, min((p + 1) * tp, m)) for p in range(n_pass) if p * tp < m]


def _sample_tokens(wl, ids, off, n):
    """The sample the FFN and combine are checked on at sizes the oracle cannot do in full: the first and last row of
    the heaviest expert; for three experts (the heaviest, the lightest with more than one pass, the one in the middle)
    the rows on both sides of every pass boundary and of the 64- and 128-row boundaries inside a pass (TMA boxes,
    M tiles) and the first and last 16-row chunk; at least one row of every touched expert; the batch's first and
    last token; the rest seeded, up to n tokens (more if the boundaries ask for more)."""
    rng = np.random.default_rng(0)
    perm = np.argsort(ids.ravel(), kind="stable")
    rows = np.diff(off)
    touched = np.nonzero(rows)[0]
    pick = []

    def add_row(p):
        t = int(perm[p]) // wl.k
        if t not in pick:
            pick.append(t)

    heavy = int(np.argmax(rows))
    add_row(off[heavy])
    add_row(off[heavy + 1] - 1)
    multi = [e for e in touched if rows[e] > 256]
    three = [heavy]
    if multi:
        by_rows = sorted(multi, key=lambda e: rows[e])
        three += [by_rows[0], by_rows[len(by_rows) // 2]]
    else:
        by_rows = sorted(touched, key=lambda e: rows[e])
        three += [by_rows[-2], by_rows[len(by_rows) // 2]]
    for e in dict.fromkeys(int(e) for e in three):
        ranges = _pass_ranges(int(rows[e]))
        if len(ranges) > 5:  # a very heavy expert: its first two, middle and last two passes
            ranges = ranges[:2] + [ranges[len(ranges) // 2]] + ranges[-2:]
        for b, en in ranges:
            edge = {b, en - 1, min(b + 15, en - 1), min(b + 16, en - 1), max(en - 17, b), max(en - 16, b)}
            for cut in (64, 128, 192):
                if b + cut < en:
                    edge.update((b + cut - 1, b + cut))
            for r in sorted(edge):
                add_row(off[e] + r)
    if n < 64:  # small samples (mid-size decode batches): the heaviest expert's ends and a row of every eighth expert
        pick = pick[:2]
        for e in touched[:: max(1, len(touched) // 8)]:
            add_row(off[e])
    covered = set(int(e) for t in pick for e in ids[t])
    for e in (touched if n >= 64 else []):
        if int(e) not in covered:
            t = int(perm[off[e]]) // wl.k
            pick.append(t)
            covered.update(int(x) for x in ids[t])
    for t in (0, wl.T - 1):
        if t not in pick:
            pick.append(t)
    pick_set = set(pick)
    while len(pick_set) < n:
        pick_set.add(int(rng.integers(0, wl.T)))
    assert n < 64 or covered >= set(int(e) for e in touched)
    return np.array(sorted(pick_set), np.int32)


# decode_c256 / c512 / c768: not benchmark workloads; mid-size batches up to the largest the decode-sized expert-FFN kernel takes at the
# production shape (8, 16 and 24 rows per expert on average: passes of 16 tokens, experts with two or three passes)
_EXTRA = {"decode_c256": inputs.Workload("decode_c256", 256, 4096, 2048, 256, 8),
          "decode_c512": inputs.Workload("decode_c512", 512, 4096, 2048, 256, 8),
          "decode_c768": inputs.Workload("decode_c768", 768, 4096, 2048, 256, 8)}


@pytest.mark.parametrize("name,n_tokens", [("prefill_8k", 256), ("prefill_32k_skewed", 256), ("decode_c256", 16),
                                           ("decode_c512", 16), ("decode_c768", 16)])
def test_layer_prefill_sampled(name, n_tokens, prod_weights):
    wl = inputs.WORKLOADS[name] if name in inputs.WORKLOADS else _EXTRA[name]
    (w13, s13, w2, s2), wdev = prod_weights
    logits = inputs.make_logits(wl.T, wl.E, 0, wl.skew)
    x = inputs.make_x(wl.T, wl.H, 0)
    d = dict(logits=logits, x=x, w13=w13, s13=s13, w2=w2, s2=s2)
    buf, out = run_layer(wl, d, wdev)
    # routing and permutation in full (bit-exact)
    rids, rw, roff = O.route(logits, wl.k)
    assert np.array_equal(buf.topk_ids.cpu().numpy(), rids)
    assert np.array_equal(buf.topk_w.cpu().numpy().view(np.uint32), rw.view(np.uint32))
    assert np.array_equal(buf.expert_offsets.cpu().numpy(), roff)
    _, rperm, rinv = O.permute(x, rids, roff)
    assert np.array_equal(buf.perm.cpu().numpy(), rperm)
    assert np.array_equal(buf.inv_perm.cpu().numpy(), rinv)
    nx = min(4096, wl.T * wl.k)
    xp = bits(buf.x_perm[:nx]), bits(buf.x_perm[-nx:])
    assert np.array_equal(xp[0], x[rperm[:nx] // wl.k]) and np.array_equal(xp[1], x[rperm[-nx:] // wl.k])
    # FFN + combine on sampled tokens by the per-token definition
    tokens = _sample_tokens(wl, rids, roff, n_tokens)
    r = O.forward_tokens(logits, x, w13, s13, w2, s2, wl.k, tokens)
    got = bits(out[torch.from_numpy(tokens.astype(np.int64)).cuda()])
    check_out(got, r["out"], r["out_f32"], name)
    rows = torch.from_numpy(rinv.reshape(wl.T, wl.k)[tokens].ravel().astype(np.int64)).cuda()
    check_y(buf.y_perm[rows].cpu().numpy(), r["y"].reshape(-1, wl.H), name)
    # properties that hold at any size: finite outputs, plausible scale
    o = out.float()
    assert torch.isfinite(o).all()
    rms = float(o.pow(2).mean().sqrt())
    assert 4.0 < rms < 20.0, rms


@pytest.mark.parametrize("name,variant", [("prefill_8k", moe.VARIANT_UMMA), ("decode_c64", moe.VARIANT_NATIVE),
                                          ("decode_c768", moe.VARIANT_NATIVE)])
def test_ffn_variants_agree_over_the_whole_tensor(name, variant, prod_weights):
    """Where the oracle can only be sampled: every element of y_perm from the variant the shape selects against the
    streaming variant on the same inputs (the streaming variant is checked against the oracle in full on the small
    shapes and shares no tile scheduler with the other two), within the tolerance of the fp32 per-slot rows.  A fault
    confined to particular work shares, passes or row tiles of the full-size launch shows up here."""
    wl = inputs.WORKLOADS[name] if name in inputs.WORKLOADS else _EXTRA[name]
    (w13, s13, w2, s2), wdev = prod_weights
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    buf = moe.LayerBuffers(sh)
    lg, x = dev(inputs.make_logits(wl.T, wl.E, 5, wl.skew)), dev(inputs.make_x(wl.T, wl.H, 5))
    moe.moe_route(lg, wl.k, buf.topk_ids, buf.topk_w, buf.expert_offsets, buf.ws)
    moe.moe_permute(x, buf.topk_ids, buf.expert_offsets, sh, buf.x_perm, buf.perm, buf.inv_perm, buf.ws)
    moe.moe_expert_ffn(buf.x_perm, buf.expert_offsets, *wdev, sh, buf.y_perm, buf.status, buf.ws)
    torch.cuda.synchronize()
    chosen = moe.moe_last_kernel_name()
    y_sel = buf.y_perm.clone()
    moe.moe_debug_expert_ffn_variant(buf.x_perm, buf.expert_offsets, *wdev, sh, buf.y_perm, buf.status, buf.ws, variant)
    torch.cuda.synchronize()
    assert moe.moe_last_kernel_name() == chosen and torch.equal(buf.y_perm, y_sel)   # the named variant IS the chosen one
    moe.moe_debug_expert_ffn_variant(buf.x_perm, buf.expert_offsets, *wdev, sh, buf.y_perm, buf.status, buf.ws,
                                     moe.VARIANT_STREAM)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0 and moe.moe_last_kernel_name() == "ffn_stream_bulk_ring_mma16816"
    diff = (y_sel.double() - buf.y_perm.double())
    ref = buf.y_perm.double()
    rms = float(ref.pow(2).mean().sqrt())
    assert float(diff.norm() / ref.norm()) <= 5e-4
    assert float(diff.abs().max()) <= 2e-2 * rms
    # per row as well: a single wrong row is invisible in the Frobenius norm of 65,536 rows
    row_rel = diff.norm(dim=1) / ref.norm(dim=1).clamp_min(1e-30)
    assert float(row_rel.max()) <= 5e-3, int(row_rel.argmax())


def test_forward_host_matches_device_path(prod_weights):
    wl = inputs.WORKLOADS["decode_c64"]
    (w13, s13, w2, s2), wdev = prod_weights
    logits = inputs.make_logits(wl.T, wl.E, 3)
    x = inputs.make_x(wl.T, wl.H, 3)
    d = dict(logits=logits, x=x)
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    buf = moe.LayerBuffers(sh)
    out = moe.moe_layer(dev(logits), dev(x), wdev, buf)
    torch.cuda.synchronize()
    ws = moe.alloc_workspace(sh, host_path=True)
    lh = torch.from_numpy(logits).pin_memory()
    xh = torch.from_numpy(x.view(np.int16)).pin_memory()
    oh = torch.empty((wl.T, wl.H), dtype=torch.int16).pin_memory()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    moe.moe_forward_host(lh, xh, *wdev, sh, oh, status, ws)
    assert int(status.item()) == 0
    assert np.array_equal(oh.numpy().view(np.uint16), bits(out))


def test_validate_scales_counts_out_of_range_bytes():
    s = np.full(5000, 120, np.uint8)
    s[[3, 77, 4999]] = [129, 255, 200]
    bad = torch.zeros(1, dtype=torch.int32, device="cuda")
    moe.moe_validate_scales(dev(s), bad)
    torch.cuda.synchronize()
    assert int(bad.item()) == 3


# ---- the tensor-core (tcgen05) expert FFN, reached when T*k >= 1024 and H, I are multiples of 512 ----

@pytest.mark.parametrize("T,H,I,E,k,hot,seed", [
    (600, 512, 512, 8, 2, False, 0),     # ~150 rows per expert: one accumulator, ragged N
    (700, 512, 512, 4, 2, False, 1),     # ~350 rows per expert: second accumulator and a second pass
    (1100, 512, 512, 8, 1, True, 2),     # one hot expert with ~1000 rows (4 passes), empty experts
    (520, 1024, 512, 16, 2, False, 3),   # K = 1024 (several packed stages), few rows per expert
])
def test_ffn_tensor_core_path_against_oracle(T, H, I, E, k, hot, seed):
    wl = inputs.Workload("umma", T, H, I, E, k)
    w = inputs.make_expert_weights(H, I, E, seed=seed)
    s13 = inputs.index_scales(2 * I, H, E, lo=117, span=6)
    s2 = inputs.index_scales(H, I, E, lo=118, span=5)
    w = (w[0], s13, w[2], s2)
    logits = inputs.make_logits(T, E, seed=seed)
    if hot:
        logits[:, 2] += 8.0
        logits[:, [5, 6]] -= 50.0
    x = inputs.make_x(T, H, seed=seed)
    ids, tw, off = O.route(logits, k)
    x_perm, perm, inv = O.permute(x, ids, off)
    sh = moe.shape(T, H, I, E, k)
    buf = moe.LayerBuffers(sh)
    moe.moe_expert_ffn(dev(x_perm), dev(off), *[dev(a) for a in w], sh, buf.y_perm, buf.status, buf.ws)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    assert moe.moe_last_kernel_name() == "ffn_umma_tcgen05_grouped"
    ry = O.expert_ffn(x_perm, off, *w, k)
    check_y(buf.y_perm.cpu().numpy(), ry, "tensor-core path")


def test_kernel_choice_is_a_function_of_the_shape():
    for (T, H, I, E, k, want) in [(16, 256, 128, 8, 2, "ffn_stream_bulk_ring_mma16816"),
                                  (64, 512, 256, 8, 2, "ffn_native_mxf4_block_scaled"),   # I = 256: native since H, I % 256
                                  (64, 512, 384, 8, 2, "ffn_stream_bulk_ring_mma16816"),
                                  (64, 512, 512, 8, 2, "ffn_native_mxf4_block_scaled"),
                                  (512, 512, 512, 8, 2, "ffn_umma_tcgen05_grouped"),
                                  (512, 512, 256, 8, 2, "ffn_stream_bulk_ring_mma16816")]:
        wl = inputs.Workload("choice", T, H, I, E, k)
        w = inputs.make_expert_weights(H, I, E, seed=0)
        logits, x = inputs.make_logits(T, E, 0), inputs.make_x(T, H, 0)
        ids, tw, off = O.route(logits, k)
        x_perm, _, _ = O.permute(x, ids, off)
        sh = moe.shape(T, H, I, E, k)
        buf = moe.LayerBuffers(sh)
        moe.moe_expert_ffn(dev(x_perm), dev(off), *[dev(a) for a in w], sh, buf.y_perm, buf.status, buf.ws)
        torch.cuda.synchronize()
        assert moe.moe_last_kernel_name() == want


# ---- the native block-scaled FP4 expert FFN, reached when T*k <= 32*E (decode-sized) and H, I are multiples of 256 ----

@pytest.mark.parametrize("T,H,I,E,k,hot,seed", [
    (16, 512, 512, 8, 2, False, 0),      # a few rows per expert: term-row boxes of 16 to 64 rows
    (1, 512, 512, 16, 4, False, 1),      # one token: every expert has at most one row
    (8, 512, 512, 8, 2, False, 4),       # two rows per expert on average
    (64, 1024, 512, 8, 2, False, 2),     # ~16 rows per expert: 128-row boxes, some experts need two passes of 16 tokens
    (64, 512, 512, 4, 2, False, 5),      # ~32 rows per expert: two or three passes each
    (40, 512, 1024, 8, 1, True, 3),      # one hot expert with most rows, several empty experts
    (8, 512, 256, 8, 2, False, 6),       # I = 256 (the paper's TP8 shard of the intermediate): one K step in the down
    (12, 768, 256, 4, 2, False, 7),      #   projection, scale rows of 8 bytes; H = 768: three K steps, rows of 24 bytes
    (5, 1280, 768, 6, 3, False, 8),      # both reductions odd multiples of 256
    (33, 4096, 256, 16, 4, False, 9),    # the model's H with the TP8 shard
])
def test_ffn_native_fp4_path_against_oracle(T, H, I, E, k, hot, seed):
    w = inputs.make_expert_weights(H, I, E, seed=seed)
    s13 = inputs.index_scales(2 * I, H, E, lo=117, span=6)
    s2 = inputs.index_scales(H, I, E, lo=118, span=5)
    w = (w[0], s13, w[2], s2)
    logits = inputs.make_logits(T, E, seed=seed)
    if hot:
        logits[:, 2] += 8.0
        logits[:, [5, 6]] -= 50.0
    x = inputs.make_x(T, H, seed=seed)
    # activations with a wide dynamic range inside a 32-block exercise the split into E2M1 terms
    xf = inputs.bf16_bits_to_f32(x)
    xf[:, ::7] *= 2.0 ** -9
    xf[:, 5::11] *= 64.0
    x = inputs.f32_to_bf16_bits(xf)
    ids, tw, off = O.route(logits, k)
    x_perm, perm, inv = O.permute(x, ids, off)
    sh = moe.shape(T, H, I, E, k)
    buf = moe.LayerBuffers(sh)
    moe.moe_expert_ffn(dev(x_perm), dev(off), *[dev(a) for a in w], sh, buf.y_perm, buf.status, buf.ws)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    assert moe.moe_last_kernel_name() == "ffn_native_mxf4_block_scaled"
    ry = O.expert_ffn(x_perm, off, *w, k)
    check_y(buf.y_perm.cpu().numpy(), ry, "native fp4 path")


# ---- consecutive layer calls on one stream, sharing every buffer but the output ----
# With programmatic dependent launch the next call's router may start while this call's combine is still
# running; it must not overwrite the routing weights and the inverse permutation that combine reads.

@pytest.mark.parametrize("T,H,I,E,k", [(4, 512, 512, 8, 2), (1, 4096, 2048, 256, 8)])
def test_back_to_back_calls_sharing_buffers(T, H, I, E, k, prod_weights):
    if (H, I, E) == (4096, 2048, 256):
        wdev = prod_weights[1]
    else:
        wdev = tuple(dev(a) for a in inputs.make_expert_weights(H, I, E, seed=1))
    sh = moe.shape(T, H, I, E, k)
    buf = moe.LayerBuffers(sh)
    n = 12
    batches = [(dev(inputs.make_logits(T, E, 300 + i)), dev(inputs.make_x(T, H, 300 + i))) for i in range(n)]

    def run(outs, sync_each):
        for (l, x), o in zip(batches, outs):
            moe.moe_route(l, k, buf.topk_ids, buf.topk_w, buf.expert_offsets, buf.ws)
            moe.moe_permute(x, buf.topk_ids, buf.expert_offsets, sh, buf.x_perm, buf.perm, buf.inv_perm, buf.ws)
            moe.moe_expert_ffn(buf.x_perm, buf.expert_offsets, *wdev, sh, buf.y_perm, buf.status, buf.ws)
            moe.moe_combine(buf.y_perm, buf.inv_perm, buf.topk_w, sh, o)
            if sync_each:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        assert int(buf.status.item()) == 0

    ref = [torch.empty_like(buf.out) for _ in range(n)]
    got = [torch.empty_like(buf.out) for _ in range(n)]
    run(ref, True)
    for rep in range(3):
        run(got, False)
        for i in range(n):
            assert torch.equal(got[i].view(torch.int16), ref[i].view(torch.int16)), "call %d of a back-to-back run differs" % i
