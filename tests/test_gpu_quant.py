"""GPU parity of the quantised-activation variant (moe_expert_ffn_q) against its own oracle (oracle.expert_ffn_q).

Tolerance.  Every product of the variant is an E2M1 value times an E2M1 value times a power of two; the fp32 sums of such
terms are exact, whatever their order, as long as the terms of one sum span fewer than 24 bits - which is the rule on the
seeded inputs, so most rows are bit-identical to the oracle.  Where a sum does round, the kernel's order may differ from
the oracle's ascending order by a few units in the last place, and the kernel's SwiGLU uses the fast exponential and
division (relative 1e-6).  Such a difference can flip the bf16 rounding of an intermediate value (about 3e-4 of the
elements) and then, where the value sits at a rounding boundary of the 4-bit format, its E2M1 code (about 1 % of those):
about one row in two hundred has one element of its intermediate off by one code step - up to a third of its block's
largest magnitude - and every output of that row moves by that step times a weight (seen: 0.13 of the row's rms, on one
row of 774).  The comparison therefore asks: every row within 0.25 of its rms, element by element, and all rows but one
(or 3 % of them) within 1e-5 of it.  `test_ffn_q_stage_by_stage` takes the call apart instead: the token rows' codes
bit-exact, the intermediate's codes equal up to such flips, the down projection exact on the kernel's own codes."""
import numpy as np
import pytest
import torch

from _gpu_util import dev
from oracle import moe_oracle as O
from paper_2609_15627_b200 import inputs, moe

pytestmark = pytest.mark.gpu

_INVALID_ARG, _UNSUPPORTED_SHAPE, _WORKSPACE = 1, 2, 3   # moe_status_t


def _check_rows(got, want, what):
    assert not np.isnan(got).any(), what
    rms = np.sqrt((want.astype(np.float64) ** 2).mean(axis=1, keepdims=True)) + 1e-30
    rel = (np.abs(got.astype(np.float64) - want) / rms).max(axis=1)
    assert rel.max() <= 0.25, (what, float(rel.max()))
    n_off = int((rel > 1e-5).sum())
    assert n_off <= max(1, int(0.03 * len(rel))), (what, n_off, len(rel))


def _problem(T, H, I, E, k, seed, logits=None):
    w = inputs.make_expert_weights(H, I, E, seed=seed)
    x = inputs.make_x(T, H, seed + 1)
    lg = inputs.make_logits(T, E, seed + 2) if logits is None else logits
    ids, wt, off = O.route(lg, k)
    xp, perm, inv = O.permute(x, ids, off)
    return w, xp, off


def _run(w_dev, xp, off, sh, status=True):
    ws = moe.alloc_ffn_q_workspace(sh)
    y = torch.full((sh.T * sh.k, sh.H), float("nan"), dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda") if status else None
    moe.moe_expert_ffn_q(dev(xp), dev(off), w_dev, sh, y, st, ws)
    torch.cuda.synchronize()
    if status:
        assert int(st.item()) == 0
    return y.cpu().numpy()


# (T, H, I, E, k): one row; ragged small batch; an expert with three passes of 128 rows (large-batch schedule: one launch per
# projection); many experts, most of them empty; H != 2I and a long reduction; rows per expert straddling the 64-row
# boundary between the two schedules
_CASES = [(1, 512, 512, 4, 2), (7, 512, 1024, 8, 2), (300, 512, 512, 2, 2), (3, 1024, 512, 200, 2), (5, 4096, 1024, 16, 4),
          (129, 512, 512, 4, 2), (65, 1024, 512, 2, 2), (9, 768, 256, 4, 2), (200, 1280, 256, 2, 1)]


@pytest.mark.parametrize("case", _CASES)
@pytest.mark.parametrize("packed", [False, True])
def test_ffn_q_matches_its_oracle(case, packed):
    T, H, I, E, k = case
    w, xp, off = _problem(T, H, I, E, k, seed=sum(case))
    sh = moe.shape(T, H, I, E, k)
    wd = tuple(dev(a) for a in w)
    got = _run(moe.moe_prepack(*wd, sh) if packed else wd, xp, off, sh)
    _check_rows(got, O.expert_ffn_q(xp, off, *w, k), (case, packed))


def test_ffn_q_all_rows_on_one_expert_and_empty_batch_edges():
    T, H, I, E, k = 200, 512, 512, 6, 1
    lg = np.full((T, E), -5.0, np.float32)
    lg[:, 4] = 5.0                                   # every row on expert 4: two passes there, five experts empty
    w, xp, off = _problem(T, H, I, E, k, seed=3, logits=lg)
    assert off.tolist() == [0, 0, 0, 0, 0, T, T]
    sh = moe.shape(T, H, I, E, k)
    got = _run(tuple(dev(a) for a in w), xp, off, sh)
    _check_rows(got, O.expert_ffn_q(xp, off, *w, k), "one expert")


def test_ffn_q_structured_scales_and_zero_blocks():
    # scale bytes that depend on (expert, row, block); token rows with all-zero blocks and with one huge element per block
    T, H, I, E, k = 9, 512, 512, 3, 2
    w13, s13, w2, s2 = inputs.make_expert_weights(H, I, E, seed=12)
    s13 = inputs.index_scales(2 * I, H, E)
    s2 = inputs.index_scales(H, I, E, lo=117)
    x = inputs.bf16_bits_to_f32(inputs.make_x(T, H, 13)).copy()
    x[:, 64:96] = 0.0
    x[2, 128] = 3.0e4
    x[3, :] = 0.0
    xb = inputs.f32_to_bf16_bits(x.astype(np.float32))
    ids, wt, off = O.route(inputs.make_logits(T, E, 14), k)
    xp, _, _ = O.permute(xb, ids, off)
    sh = moe.shape(T, H, I, E, k)
    got = _run(tuple(dev(a) for a in (w13, s13, w2, s2)), xp, off, sh)
    _check_rows(got, O.expert_ffn_q(xp, off, w13, s13, w2, s2, k), "structured")


@pytest.mark.parametrize("T,H,I,E,k", [(33, 512, 512, 4, 2),      # one launch for both projections
                                       (300, 512, 512, 2, 2)])    # large-batch schedule: one launch per projection
def test_ffn_q_without_a_status_word_and_replayed_as_a_graph(T, H, I, E, k):
    w, xp, off = _problem(T, H, I, E, k, seed=5)
    sh = moe.shape(T, H, I, E, k)
    wd = tuple(dev(a) for a in w)
    first = _run(wd, xp, off, sh, status=False)
    _check_rows(first, O.expert_ffn_q(xp, off, *w, k), "no status word")
    ws = moe.alloc_ffn_q_workspace(sh)
    xd, od = dev(xp), dev(off)
    y = torch.empty((T * k, H), dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        moe.moe_expert_ffn_q(xd, od, wd, sh, y, st, ws, side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        moe.moe_expert_ffn_q(xd, od, wd, sh, y, st, ws, torch.cuda.current_stream())
    for _ in range(20):
        y.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy(), first)
    assert int(st.item()) == 0


def test_ffn_q_argument_checks():
    T, H, I, E, k = 4, 512, 512, 2, 1
    w, xp, off = _problem(T, H, I, E, k, seed=1)
    sh = moe.shape(T, H, I, E, k)
    wd = tuple(dev(a) for a in w)
    ws = moe.alloc_ffn_q_workspace(sh)
    y = torch.empty((T * k, H), dtype=torch.float32, device="cuda")
    xd, od = dev(xp), dev(off)
    lib, C = moe.lib(), __import__("ctypes")
    p = lambda t: None if t is None else C.c_void_p(t.data_ptr())
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    packed = moe.moe_prepack(*wd, sh)

    def call(weights4, pk, shape, ws_t=ws, n=None):
        return lib.moe_expert_ffn_q(p(xd), p(od), *(p(t) for t in weights4), p(pk), C.byref(shape), p(y), None, p(ws_t),
                                    ws_t.numel() if n is None else n, stream)

    none4 = (None, None, None, None)
    assert call(wd, None, sh) == 0 and call(none4, packed, sh) == 0
    assert call(wd, packed, sh) == _INVALID_ARG          # both forms of the weights
    assert call(none4, None, sh) == _INVALID_ARG        # neither
    assert call((wd[0], None, wd[2], wd[3]), None, sh) == _INVALID_ARG
    assert call(wd, None, sh, n=ws.numel() // 2) == _WORKSPACE
    assert call(wd, None, moe.shape(T, 384, I, E, k)) == _UNSUPPORTED_SHAPE   # H not a multiple of 256
    assert call(wd, None, moe.shape(T, H, 128, E, k)) == _UNSUPPORTED_SHAPE
    torch.cuda.synchronize()


@pytest.mark.parametrize("name", ["decode_c64", "prefill_8k", "prefill_32k_skewed"])
def test_ffn_q_at_the_benchmark_shapes_on_sampled_rows(name):
    """The launch configuration bench.py times (prepacked weights, the library's own routing and permutation), checked on
    sampled sorted rows: first and last row, rows either side of expert boundaries, random rows."""
    wl = inputs.WORKLOADS[name]
    T, H, I, E, k = wl.T, wl.H, wl.I, wl.E, wl.k
    w = inputs.make_expert_weights(H, I, E, seed=0)
    sh = moe.shape(T, H, I, E, k)
    wd = tuple(dev(a) for a in w)
    packed = moe.moe_prepack(*wd, sh)
    del wd
    buf = moe.LayerBuffers(sh)
    moe.moe_route(dev(inputs.make_logits(T, E, 1, wl.skew)), k, buf.topk_ids, buf.topk_w, buf.expert_offsets, buf.ws)
    moe.moe_permute(dev(inputs.make_x(T, H, 1)), buf.topk_ids, buf.expert_offsets, sh, buf.x_perm, buf.perm, buf.inv_perm, buf.ws)
    ws = moe.alloc_ffn_q_workspace(sh)
    buf.y_perm.fill_(float("nan"))
    moe.moe_expert_ffn_q(buf.x_perm, buf.expert_offsets, packed, sh, buf.y_perm, buf.status, ws)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    assert not torch.isnan(buf.y_perm).any()
    off = buf.expert_offsets.cpu().numpy()
    S = T * k
    rng = np.random.default_rng(0)
    heavy = int(np.argmax(np.diff(off)))                      # the expert with the most rows: the most passes
    edges = np.concatenate([off[np.r_[1:4, E // 2, E - 2]], [off[heavy], off[heavy + 1] - 130]])
    rows = np.unique(np.clip(np.concatenate([rng.integers(0, S, 40), [0, S - 1], edges - 1, edges, edges + 127, edges + 128]), 0, S - 1))
    expert_of = np.searchsorted(off, rows, side="right") - 1
    idx = torch.from_numpy(rows).cuda()
    xs = np.ascontiguousarray(buf.x_perm[idx].cpu().view(torch.int16).numpy().view(np.uint16))
    so = np.zeros(E + 1, np.int64)
    np.add.at(so, expert_of + 1, 1)
    want = O.expert_ffn_q(xs, np.cumsum(so).astype(np.int32), *w, 1)
    _check_rows(buf.y_perm[idx].cpu().numpy(), want, name)


def test_ffn_q_whole_tensor_agrees_between_weight_layouts_at_prefill_8k():
    """Every row of the output, not a sample: the call on the checkpoint's row layout and the call on moe_prepack's tiles
    read different bytes through different tensor maps and must give the same bits (the sampled rows above tie one of
    them to the oracle)."""
    wl = inputs.WORKLOADS["prefill_8k"]
    T, H, I, E, k = wl.T, wl.H, wl.I, wl.E, wl.k
    sh = moe.shape(T, H, I, E, k)
    wd = tuple(dev(a) for a in inputs.make_expert_weights(H, I, E, seed=0))
    packed = moe.moe_prepack(*wd, sh)
    buf = moe.LayerBuffers(sh)
    moe.moe_route(dev(inputs.make_logits(T, E, 2, wl.skew)), k, buf.topk_ids, buf.topk_w, buf.expert_offsets, buf.ws)
    moe.moe_permute(dev(inputs.make_x(T, H, 2)), buf.topk_ids, buf.expert_offsets, sh, buf.x_perm, buf.perm, buf.inv_perm, buf.ws)
    ws = moe.alloc_ffn_q_workspace(sh)
    y2 = torch.full_like(buf.y_perm, float("nan"))
    buf.y_perm.fill_(float("nan"))
    moe.moe_expert_ffn_q(buf.x_perm, buf.expert_offsets, wd, sh, buf.y_perm, buf.status, ws)
    moe.moe_expert_ffn_q(buf.x_perm, buf.expert_offsets, packed, sh, y2, buf.status, ws)
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    assert not torch.isnan(y2).any()
    assert torch.equal(buf.y_perm, y2)


def _unpack_codes(packed):
    return np.stack([packed & 0xF, packed >> 4], axis=-1).reshape(packed.shape[0], -1)


@pytest.mark.parametrize("T,H,I,E,k", [(129, 256, 1024, 32, 6), (64, 512, 512, 8, 2), (300, 512, 256, 2, 2)])
def test_ffn_q_stage_by_stage(T, H, I, E, k):
    """The call taken apart through its scratch (layout of the variant's workspace: codes of the intermediate [S, I/2],
    its scale bytes [S, I/32], codes of the token rows [S, H/2], their scale bytes [S, H/32], each region padded to 256
    bytes).  (1) The token rows' quantisation involves no sum: bit-exact against the oracle's quantiser.  (2) The
    intermediate's codes: equal to the oracle's except where a last-bit difference before the rounding to bf16 moved
    a value across a rounding boundary - a handful of elements, each one code step away.  (3) The down projection on
    the kernel's OWN codes, recomputed in float64: equal to the kernel's output to fp32 rounding."""
    w, xp, off = _problem(T, H, I, E, k, seed=7)
    sh = moe.shape(T, H, I, E, k)
    S = T * k
    ws = moe.alloc_ffn_q_workspace(sh)
    y = torch.empty((S, H), dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    moe.moe_expert_ffn_q(dev(xp), dev(off), tuple(dev(a) for a in w), sh, y, st, ws)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    al = lambda n: (n + 255) // 256 * 256
    raw = ws.cpu().numpy()
    o = 0
    aq2 = raw[o:o + S * I // 2].reshape(S, I // 2); o += al(S * I // 2)
    sf2 = raw[o:o + S * I // 32].reshape(S, I // 32); o += al(S * I // 32)
    aq1 = raw[o:o + S * H // 2].reshape(S, H // 2); o += al(S * H // 2)
    sf1 = raw[o:o + S * H // 32].reshape(S, H // 32)
    # (1)
    q1, s1, _ = O.quant_act(xp)
    assert np.array_equal(aq1, q1) and np.array_equal(sf1, s1)
    # (2)
    want, act = O.expert_ffn_q(xp, off, *w, k, want_act=True)
    q2, s2, _ = O.quant_act(act)
    same_scale = sf2 == s2
    c_gpu, c_ref = _unpack_codes(aq2).astype(np.int64), _unpack_codes(q2).astype(np.int64)
    diff = (c_gpu != c_ref) & np.repeat(same_scale, 32, axis=1)
    n_elem = S * I
    assert (~same_scale).sum() <= max(1, n_elem // 32 // 20000)          # a block's largest value crossing a scale boundary
    assert diff.sum() <= max(2, n_elem // 20000), int(diff.sum())
    mag = lambda c: np.where(c >= 8, c - 8, c)
    assert np.all(np.abs(mag(c_gpu[diff]) - mag(c_ref[diff])) <= 1)       # one step of the 4-bit format
    # (3)
    mags = np.array([0, .5, 1, 1.5, 2, 3, 4, 6], np.float64)
    table = np.concatenate([mags, -mags])
    a_gpu = table[c_gpu] * np.repeat(np.ldexp(1.0, sf2.astype(np.int64) - 127), 32, axis=1)
    w2, s2w = w[2], w[3]
    expert_of = np.repeat(np.arange(E), np.diff(off))
    got = y.cpu().numpy()
    for e in np.unique(expert_of):
        rows = np.nonzero(expert_of == e)[0]
        W2 = table[_unpack_codes(w2[e]).astype(np.int64)] * np.repeat(np.ldexp(1.0, s2w[e].astype(np.int64) - 127), 32, axis=1)
        ref = a_gpu[rows] @ W2.T
        assert np.allclose(got[rows], ref, rtol=2e-6, atol=2e-6 * np.abs(ref).max())
