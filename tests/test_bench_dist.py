"""The multi-GPU path of bench.py is 'replicas only': every rank runs the same work and the only
exchange is the max-over-ranks of the measured time.  Checked here with two gloo ranks on CPU."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist

    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_seconds = 1.0 + rank          # rank 1 is the slow one
    worst = bench.dist_max(local_seconds)
    dist.barrier()
    q.put((rank, worst, bench.aggregate(10.0, world, worst)))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_throughput():
    ctx = mp.get_context("spawn")
    q = ctx.SimpleQueue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    got = sorted(q.get() for _ in range(2))
    for rank, worst, value in got:
        assert worst == 2.0                 # both ranks agree on the slowest rank's time
        assert value == 10.0 * 2 / 2.0      # units of ALL ranks over that time


def test_single_process_helpers_and_byte_formulas():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.dist_max(3.5) == 3.5
    b = bench.algorithmic_bytes(sum_t=100, n_blocks=3, t_block=40, fb=8, ofb=16)
    assert b == dict(pack=100 * 8 + 3 * 40 * 8, unpack=2 * 100 * 16, meta=10 * 120)
    peak, kind = bench.measured_peak()
    assert peak > 1000 and kind in ("measured", "fallback")
