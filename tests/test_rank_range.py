"""Shares of data-parallel ranks (host only): every rank gets the same number of equally long blocks, which is what
keeps gradient synchronisation from stalling (paper, section "Problem Statement and Current Limitations")."""
import os
import sys

import pytest
import torch.multiprocessing as mp

import paper_2310_10879_b200 as B
from paper_2310_10879_b200 import _lib

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_ranges_are_equal_disjoint_and_cover_all_blocks():
    for n_blocks in (1, 7, 116, 213658):
        for world in (1, 2, 3, 8):
            for batch in (1, 4, 64):
                ranges = [B.bload_rank_range(n_blocks, world, r, batch) for r in range(world)]
                counts = {c for _, c in ranges}
                assert len(counts) == 1 and next(iter(counts)) % batch == 0          # same work everywhere, whole batches
                assert [b for b, _ in ranges] == [r * ranges[0][1] for r in range(world)]  # contiguous, disjoint
                assert ranges[-1][0] + ranges[-1][1] >= n_blocks                      # every block belongs to some rank
                assert (ranges[0][1] - batch) * world < n_blocks                       # and not a batch more than needed
    # the deadlock example of the paper: 8 videos of 2..6 frames in blocks of 6 -> both GPUs run the same iterations
    assert B.bload_rank_range(6, 2, 0, 1) == (0, 3) and B.bload_rank_range(6, 2, 1, 1) == (3, 3)
    for bad in [(0, 2, 0, 1), (5, 0, 0, 1), (5, 2, 2, 1), (5, 2, -1, 1), (5, 2, 0, 0), (2**31, 8, 0, 1)]:
        with pytest.raises(B.BloadError) as ei:
            B.bload_rank_range(*bad)
        assert ei.value.code == _lib.ERR_ARG


def _rank(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist

    import paper_2310_10879_b200 as Bl
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    begin, count = Bl.bload_rank_range(37, world, rank, 4)
    t = torch.tensor([count], dtype=torch.int64)
    lo, hi = t.clone(), t.clone()
    dist.all_reduce(lo, op=dist.ReduceOp.MIN); dist.all_reduce(hi, op=dist.ReduceOp.MAX)
    gathered = [torch.zeros(2, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(gathered, torch.tensor([begin, count], dtype=torch.int64))
    q.put((rank, int(lo), int(hi), [tuple(int(x) for x in g) for g in gathered]))
    dist.destroy_process_group()


def test_two_ranks_agree_without_exchanging_anything_but_the_check():
    ctx = mp.get_context("spawn")
    q = ctx.SimpleQueue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    for rank, lo, hi, ranges in (q.get() for _ in range(2)):
        assert lo == hi == 20                       # ceil(37 / 2) = 19 -> 20 blocks = 5 batches of 4 on both ranks
        assert ranges == [(0, 20), (20, 20)]
