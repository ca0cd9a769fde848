"""Expert-parallel sharding of the routed layer: orchestration of the C-ABI calls (no arithmetic here).

Rank r of `world` holds the experts [e_begin, e_end) and finishes the tokens [t_begin, t_end).  Every rank routes and
sorts all tokens; its experts' rows are one contiguous range of the sorted order; the expert FFN's down projection
stores each output row straight into the buffer of the rank that finishes the row's token (moe_ep_row_table,
moe_ep_expert_ffn); after a barrier each rank combines its own tokens.  The result is bit-identical to the unsharded
layer.

Two drivers:
  - `run_emulated`: all ranks one after the other in ONE process on ONE GPU, every rank with buffers of its own; the
    "peer" pointers are then ordinary device pointers.  No kernel of a rank waits for another rank, so running the ranks
    in sequence is the same computation.  This is what the GPU tests run.
  - `EpProcess`: one process per GPU under torch.distributed; the ranks' output buffers live in symmetric memory, whose
    peer pointers go into the row table.  Needs more than one GPU.
`partition` and `row_destinations` are the host-side logic, shared by both and tested on CPU ranks.
"""
import numpy as np


def partition(T, E, world, rank):
    """(e_begin, e_end, t_begin, t_end, tokens_per_rank) of `rank`: equal expert ranges (whole multiples of 4, so that
    the shifted offsets array stays 16-byte aligned) and ceil(T / world) tokens per rank (the last ranks may get fewer,
    or none)."""
    if E % world != 0 or (E // world) % 4 != 0:
        raise ValueError("expert-parallel sharding needs E / world to be a whole multiple of 4")
    per = E // world
    tpr = (T + world - 1) // world
    t0 = min(rank * tpr, T)
    return rank * per, (rank + 1) * per, t0, min(t0 + tpr, T), tpr


def row_destinations(perm, offsets, k, e_begin, e_end, tokens_per_rank):
    """Host restatement of the row table: for the sorted rows of the experts [e_begin, e_end), arrays (sorted row,
    owner rank, row inside the owner's buffer)."""
    p = np.arange(int(offsets[e_begin]), int(offsets[e_end]), dtype=np.int64)
    slot = perm[p].astype(np.int64)
    token, j = slot // k, slot % k
    owner = token // tokens_per_rank
    return p, owner, (token - owner * tokens_per_rank) * k + j


class RankBuffers:
    """Device buffers of one rank (allocation only)."""

    def __init__(self, torch, moe, sh, world, rank, device="cuda"):
        self.e_begin, self.e_end, self.t_begin, self.t_end, self.tpr = partition(sh.T, sh.E, world, rank)
        self.sh, self.world, self.rank = sh, world, rank
        self.layer = moe.LayerBuffers(sh, device)            # routing, order, sorted rows, workspace, status
        S = sh.T * sh.k
        self.y_own = torch.zeros((self.tpr * sh.k, sh.H), dtype=torch.float32, device=device)
        self.row_dst = torch.zeros(S, dtype=torch.int64, device=device)
        self.owner_y = torch.zeros(world, dtype=torch.int64, device=device)
        self.identity = torch.arange(self.tpr * sh.k, dtype=torch.int32, device=device)


def compute(moe, buf, logits, x, w_local, stream=None):
    """Everything up to the barrier: route and sort all tokens, build the row table, run this rank's experts (whose
    epilogue stores into the owners' buffers)."""
    sh, L = buf.sh, buf.layer
    moe.moe_route(logits, sh.k, L.topk_ids, L.topk_w, L.expert_offsets, L.ws, stream)
    moe.moe_ep_permute(x, L.topk_ids, L.expert_offsets, sh, buf.e_begin, buf.e_end, L.x_perm, L.perm, L.inv_perm, L.ws, stream)
    moe.moe_ep_row_table(L.perm, L.expert_offsets, sh, buf.e_begin, buf.e_end, buf.owner_y, buf.world, buf.row_dst, stream)
    moe.moe_ep_expert_ffn(L.x_perm, L.expert_offsets, w_local, sh, buf.e_begin, buf.e_end, buf.row_dst, L.status, L.ws, stream)


def finish(moe, buf, out, stream=None):
    """After the barrier: the slot-ordered combine of this rank's tokens into rows [t_begin, t_end) of `out` [T, H]."""
    sh, L = buf.sh, buf.layer
    n = buf.t_end - buf.t_begin
    if n <= 0:
        return
    local = moe.shape(n, sh.H, sh.I, sh.E, sh.k)
    moe.moe_combine(buf.y_own, buf.identity, L.topk_w[buf.t_begin:buf.t_end], local, out[buf.t_begin:buf.t_end], stream)


def slice_weights(weights, e_begin, e_end):
    """The four weight tensors of the experts [e_begin, e_end) (views: the expert is the leading dimension)."""
    return tuple(w[e_begin:e_end] for w in weights)


def run_emulated(torch, moe, sh, world, logits, x, weights):
    """All ranks in sequence on one GPU; returns (out [T, H] bf16, the ranks' buffers)."""
    ranks = [RankBuffers(torch, moe, sh, world, r) for r in range(world)]
    ptrs = torch.tensor([b.y_own.data_ptr() for b in ranks], dtype=torch.int64, device="cuda")
    for b in ranks:
        b.owner_y.copy_(ptrs)
    for b in ranks:
        compute(moe, b, logits, x, slice_weights(weights, b.e_begin, b.e_end))
    torch.cuda.synchronize()                                 # the barrier: every rank's stores are complete
    out = torch.empty((sh.T, sh.H), dtype=torch.bfloat16, device="cuda")
    for b in ranks:
        finish(moe, b, out)
    torch.cuda.synchronize()
    return out, ranks


class EpProcess:
    """One rank of a torch.distributed job (backend nccl, one process per GPU).  The output buffers are symmetric
    memory, so that every rank holds the peers' addresses; the barrier between the expert FFN and the combine is the
    process group's.  `out` of step() holds this rank's tokens only (rows [t_begin, t_end) of the layer's output)."""

    def __init__(self, torch, moe, sh, weights_local, group=None):
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm
        self.torch, self.moe, self.dist, self.group = torch, moe, dist, group
        world, rank = dist.get_world_size(group), dist.get_rank(group)
        self.buf = RankBuffers(torch, moe, sh, world, rank)
        y = symm.empty((self.buf.tpr * sh.k, sh.H), dtype=torch.float32, device="cuda")
        handle = symm.rendezvous(y, group if group is not None else dist.group.WORLD)
        self.buf.y_own = y
        self.buf.owner_y.copy_(torch.tensor([int(p) for p in handle.buffer_ptrs], dtype=torch.int64))
        self.weights_local = weights_local
        self.out = torch.empty((sh.T, sh.H), dtype=torch.bfloat16, device="cuda")

    def step(self, logits, x):
        compute(self.moe, self.buf, logits, x, self.weights_local)
        self.torch.cuda.synchronize()
        self.dist.barrier(self.group)                        # all ranks' stores into this rank's buffer are complete
        finish(self.moe, self.buf, self.out)
        return self.out[self.buf.t_begin:self.buf.t_end]
