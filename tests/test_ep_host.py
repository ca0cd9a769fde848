"""Host side of the expert-parallel sharding on CPU ranks (gloo, world size 2 and 4): every rank computes its own slice
and its own row destinations from the oracle's routing; together they must cover every expert, every token and every
slot's row in exactly one owner's buffer, and the owners' slot-ordered combine of those rows must be the layer.  No GPU."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import moe_oracle as O
from paper_2609_15627_b200 import ep, inputs


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank_main(rank, world, port, T, H, I, E, k, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = inputs.make_expert_weights(H, I, E, seed=1)
        logits, x = inputs.make_logits(T, E, 2), inputs.make_x(T, H, 3)
        ids, tw, off = O.route(logits, k)
        x_perm, perm, inv = O.permute(x, ids, off)
        e0, e1, t0, t1, tpr = ep.partition(T, E, world, rank)
        # this rank's experts on its range of the sorted order (the oracle as the stand-in for the kernels)
        y = O.expert_ffn(x_perm, off, *w, k)
        p, owner, row = ep.row_destinations(perm, off, k, e0, e1, tpr)
        # "peer stores": contributions per owner, exchanged with all_gather_object
        mine = [(int(o), int(r), y[int(pp)].copy()) for pp, o, r in zip(p, owner, row)]
        everything = [None] * world
        dist.all_gather_object(everything, (e0, e1, t0, t1, mine))
        # the slices tile the experts and the tokens
        assert sorted((a, b) for a, b, _, _, _ in everything) == [(i * (E // world), (i + 1) * (E // world)) for i in range(world)]
        tok = sorted((c, d) for _, _, c, d, _ in everything)
        assert tok[0][0] == 0 and tok[-1][1] == T and all(tok[i][1] == tok[i + 1][0] for i in range(world - 1))
        # this owner's buffer: every row of its tokens written exactly once, by whichever rank holds the expert
        n_own = (t1 - t0) * k
        buf = np.full((max(n_own, 1), H), np.nan, np.float32)
        count = np.zeros(max(n_own, 1), np.int64)
        for _, _, _, _, rows in everything:
            for o, r, v in rows:
                if o == rank:
                    buf[r] = v
                    count[r] += 1
        assert np.all(count[:n_own] == 1)
        if n_own:
            out, _ = O.combine(buf[:n_own], np.arange(n_own, dtype=np.int32), np.ascontiguousarray(tw[t0:t1]))
            ref = O.forward_staged(logits, x, *w, k)["out"]
            assert np.array_equal(out, ref[t0:t1])
        ret[rank] = 1
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,T,E,k", [(2, 9, 8, 2), (4, 6, 16, 4)])
def test_partition_and_row_destinations_over_cpu_ranks(world, T, E, k):
    H, I = 128, 128
    ret = mp.Manager().dict()
    mp.spawn(_rank_main, args=(world, _free_port(), T, H, I, E, k, ret), nprocs=world, join=True)
    assert sorted(ret.keys()) == list(range(world))


def test_partition_rules():
    assert ep.partition(64, 256, 8, 3) == (96, 128, 24, 32, 8)
    assert ep.partition(7, 16, 4, 3) == (12, 16, 6, 7, 2)
    assert ep.partition(3, 8, 2, 1) == (4, 8, 2, 3, 2)
    assert ep.partition(1, 8, 2, 1)[2:4] == (1, 1)          # a rank with no token
    with pytest.raises(ValueError):
        ep.partition(8, 12, 2, 0)
