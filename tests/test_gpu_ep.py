"""Expert-parallel sharding on ONE GPU: the ranks run one after the other in one process, each with its own buffers (no
kernel of a rank waits for another rank, so this is the same computation as one process per GPU; the peers' pointers are
ordinary device pointers here).  The sharded result must equal the unsharded layer bit for bit: the owners combine the
same fp32 rows in the same slot order."""
import numpy as np
import pytest
import torch

from _gpu_util import dev
from oracle import moe_oracle as O
from paper_2609_15627_b200 import ep, inputs, moe

pytestmark = pytest.mark.gpu


def _layer(T, H, I, E, k, seed, skew=False):
    w = inputs.make_expert_weights(H, I, E, seed=seed)
    return w, inputs.make_logits(T, E, seed + 1, skew), inputs.make_x(T, H, seed + 2)


# (T, H, I, E, k, world, kernel of a rank's expert FFN)
_CASES = [
    (64, 512, 512, 32, 4, 4, "ffn_native_mxf4_block_scaled"),     # decode-sized: 8 experts per rank
    (7, 512, 512, 16, 4, 4, "ffn_native_mxf4_block_scaled"),      # 2 tokens per rank, the last rank has one
    (3, 512, 512, 8, 4, 2, "ffn_native_mxf4_block_scaled"),       # more ranks' worth of buffer than tokens on rank 1
    (600, 512, 512, 8, 2, 2, "ffn_umma_tcgen05_grouped"),         # prefill-sized: the grouped bf16 GEMM's epilogue
    (48, 256, 128, 16, 2, 2, "ffn_stream_bulk_ring_mma16816"),    # a shape only the streaming kernel takes
    (40, 512, 256, 8, 4, 2, "ffn_native_mxf4_block_scaled"),      # I = 256
]


@pytest.mark.parametrize("T,H,I,E,k,world,kernel", _CASES)
def test_sharded_layer_is_bit_identical_to_the_unsharded_one(T, H, I, E, k, world, kernel):
    w, logits, x = _layer(T, H, I, E, k, seed=T + world)
    sh = moe.shape(T, H, I, E, k)
    wd = tuple(dev(a) for a in w)
    buf = moe.LayerBuffers(sh)
    want = moe.moe_layer(dev(logits), dev(x), wd, buf).clone()
    torch.cuda.synchronize()
    out, ranks = ep.run_emulated(torch, moe, sh, world, dev(logits), dev(x), wd)
    assert all(int(b.layer.status.item()) == 0 for b in ranks)
    assert moe.moe_last_kernel_name() == "combine_slot_order_fma"
    assert torch.equal(out, want)
    # and against the oracle, through the layer's usual tolerance (the unsharded layer is tested against it elsewhere)
    r = O.forward_staged(logits, x, *w, k)
    got = out.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.mean(got != r["out"]) < 0.05


def test_the_kernel_a_rank_runs_and_the_rows_it_writes():
    """One rank alone: the expert FFN on the shifted offsets runs the kernel the shape selects, writes exactly the rows
    of its own experts (through the table) and leaves every other row of every owner's buffer alone."""
    T, H, I, E, k, world = 64, 512, 512, 32, 4, 4
    w, logits, x = _layer(T, H, I, E, k, seed=3)
    sh = moe.shape(T, H, I, E, k)
    ranks = [ep.RankBuffers(torch, moe, sh, world, r) for r in range(world)]
    ptrs = torch.tensor([b.y_own.data_ptr() for b in ranks], dtype=torch.int64, device="cuda")
    for b in ranks:
        b.owner_y.copy_(ptrs)
        b.y_own.fill_(float("nan"))
    me = ranks[1]
    wd = tuple(dev(a) for a in w)
    ep.compute(moe, me, dev(logits), dev(x), ep.slice_weights(wd, me.e_begin, me.e_end))
    torch.cuda.synchronize()
    assert moe.moe_last_kernel_name() == "ffn_native_mxf4_block_scaled"
    ids, tw, off = O.route(logits, k)
    _, perm, _ = O.permute(x, ids, off)
    p, owner, row = ep.row_destinations(perm, off, k, me.e_begin, me.e_end, me.tpr)
    written = [torch.isnan(b.y_own).any(dim=1).logical_not().cpu().numpy() for b in ranks]
    for r in range(world):
        expect = np.zeros(ranks[r].y_own.shape[0], bool)
        expect[row[owner == r]] = True
        assert np.array_equal(written[r], expect), r
    # the table itself: addresses of exactly those rows
    table = me.row_dst.cpu().numpy()
    want_addr = ptrs.cpu().numpy()[owner] + row * H * 4
    assert np.array_equal(table[p], want_addr)


def test_production_decode_shape_on_eight_ranks():
    wl = inputs.WORKLOADS["decode_c64"]
    w, logits, x = _layer(wl.T, wl.H, wl.I, wl.E, wl.k, seed=0)
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    wd = tuple(dev(a) for a in w)
    buf = moe.LayerBuffers(sh)
    want = moe.moe_layer(dev(logits), dev(x), wd, buf).clone()
    torch.cuda.synchronize()
    out, ranks = ep.run_emulated(torch, moe, sh, 8, dev(logits), dev(x), wd)
    assert all(int(b.layer.status.item()) == 0 for b in ranks)
    assert torch.equal(out, want)


def test_argument_checks():
    T, H, I, E, k = 8, 512, 512, 16, 2
    sh = moe.shape(T, H, I, E, k)
    b = ep.RankBuffers(torch, moe, sh, 2, 0)
    with pytest.raises(moe.MoeError):   # expert range not starting on a multiple of 4
        moe.moe_ep_row_table(b.layer.perm, b.layer.expert_offsets, sh, 2, 10, b.owner_y, 2, b.row_dst)
    with pytest.raises(moe.MoeError):   # empty range
        moe.moe_ep_row_table(b.layer.perm, b.layer.expert_offsets, sh, 8, 8, b.owner_y, 2, b.row_dst)
    with pytest.raises(ValueError):
        ep.partition(T, 12, 2, 0)       # 6 experts per rank: not a multiple of 4
