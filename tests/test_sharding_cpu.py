"""The multi-GPU side of the path on CPU: the batch split and the max-over-ranks timing reduce,
run as two gloo ranks; and the oracle agrees that sharding sequences changes nothing."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import psattn_oracle as orc
from paper_2106_09236_b200 import sharding
from paper_2106_09236_b200 import workloads as wl


def test_shard_range_covers_everything_once():
    for n in (0, 1, 7, 16, 64, 65):
        for world in (1, 2, 3, 8):
            got = []
            for r in range(world):
                lo, hi = sharding.shard_range(n, world, r)
                assert 0 <= lo <= hi <= n
                got += list(range(lo, hi))
            assert got == list(range(n))
            sizes = [sharding.shard_range(n, world, r) for r in range(world)]
            assert max(h - l for l, h in sizes) - min(h - l for l, h in sizes) <= 1


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # each rank runs its shard of a ragged batch through the oracle; rank 0 compares with the whole
        w = wl.WORKLOADS["ragged_bf16"]
        n = max(orc.count(w.c, L) for L in range(1, w.T + 1))
        inp = wl.make_inputs(w, n, B=4)
        lo, hi = sharding.shard_range(4, world, rank)
        O, sel, M = orc.forward(inp["Q"][lo:hi], inp["K"][lo:hi], inp["V"][lo:hi], inp["sample_idx"][lo:hi],
                                inp["lengths"][lo:hi], c=w.c)
        queries = float(inp["lengths"][lo:hi].sum() * w.H)
        total_q = sharding.sum_over_ranks(queries)
        slow = sharding.max_over_ranks(1.0 + rank)          # the slowest rank sets the step time
        gathered = [None] * world
        dist.all_gather_object(gathered, (lo, hi, O, sel))
        if rank == 0:
            Of, self_, _ = orc.forward(inp["Q"], inp["K"], inp["V"], inp["sample_idx"], inp["lengths"], c=w.c)
            for lo_, hi_, O_, sel_ in gathered:
                np.testing.assert_array_equal(O_, Of[lo_:hi_])
                np.testing.assert_array_equal(sel_, self_[lo_:hi_])
            out.put((total_q, slow, float(inp["lengths"].sum() * w.H)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_the_batch_with_no_exchange():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=180)
        assert p.exitcode == 0
    total_q, slow, want_q = out.get(timeout=10)
    assert total_q == want_q
    assert slow == 2.0


def test_reduces_are_identity_without_a_process_group():
    assert sharding.max_over_ranks(3.5) == 3.5
    assert sharding.sum_over_ranks(2.0) == 2.0
    assert sharding.rank_seed(100, 2, 3) == 100 + 2000 + 51
