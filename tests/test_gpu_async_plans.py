"""Several plans in flight: bload_plan_async / bload_plan_finish on different streams, and a plan that is
built while another plan's pack and unpack are running.  Every result is compared with the oracle."""
import ctypes as C

import numpy as np
import pytest
import torch

import gpu_util as G
import paper_2310_10879_b200 as B
from oracle import bload_oracle as O
from paper_2310_10879_b200 import _lib
from paper_2310_10879_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_eight_epochs_planned_side_by_side():
    w = W.scaled(W.WORKLOADS["heavy_tail_bf16"], 6000)
    T = W.lengths(w)
    d_len = torch.from_numpy(T).to(G.DEV)
    streams = [torch.cuda.Stream() for _ in range(8)]
    jobs = []
    for e, s in enumerate(streams):
        s.wait_stream(torch.cuda.current_stream())
        jobs.append(B.bload_plan_async(d_len, w.t_block, seed=100 + e, policy=e % 2, stream=s))
    for e, (s, (buf, work, sizes)) in enumerate(zip(streams, jobs)):
        plan = B.bload_plan_finish(buf, sizes, stream=s)
        assert plan.info.seed == 100 + e and plan.info.policy == e % 2 and plan.info.n == T.size
        G.assert_plan_equal(plan, O.plan(T, w.t_block, 100 + e, e % 2))


def test_next_epoch_is_planned_under_the_copies_of_the_current_one():
    w = W.scaled(W.WORKLOADS["tokens"], 40000)
    T = W.lengths(w)
    fb = w.frame_bytes
    d_len = torch.from_numpy(T).to(G.DEV)
    cur = B.bload_plan(d_len, w.t_block, 1)
    op = O.plan(T, w.t_block, 1)
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    dense = torch.empty(op.n_blocks * w.t_block * fb, dtype=torch.uint8, device=G.DEV)
    back = torch.empty_like(store)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    nxt = B.bload_plan_async(d_len, w.t_block, 2, stream=side)        # epoch 2 on the side stream ...
    B.bload_pack(cur, store, fb, 0, op.n_blocks, dense=dense)         # ... while epoch 1 is packed and unpacked
    B.bload_unpack(cur, dense, fb, 0, op.n_blocks, back)
    plan2 = B.bload_plan_finish(nxt[0], nxt[2], stream=side)
    torch.cuda.synchronize()
    assert np.array_equal(dense.cpu().numpy().reshape(op.n_blocks, w.t_block, fb), O.pack(op, store.cpu().numpy(), fb, 0, op.n_blocks, 0))
    assert torch.equal(back, store)
    G.assert_plan_equal(plan2, O.plan(T, w.t_block, 2))


def test_async_errors_and_unfinished_buffers():
    L = B.load()
    d_len = torch.ones(16, dtype=torch.int32, device=G.DEV)
    sz = B.bload_plan_sizes(16, 8)
    buf = torch.zeros(sz.plan_bytes, dtype=torch.uint8, device=G.DEV)
    work = torch.zeros(sz.work_bytes, dtype=torch.uint8, device=G.DEV)
    args = [d_len.data_ptr(), 16, 8, 0, 0, buf.data_ptr(), sz.plan_bytes, work.data_ptr(), sz.work_bytes, None]

    def call(i, v):
        a = list(args); a[i] = v
        return L.bload_plan_async(*a)

    assert call(0, None) == _lib.ERR_NULL and call(5, None) == _lib.ERR_NULL and call(7, None) == _lib.ERR_NULL
    assert call(1, 0) == _lib.ERR_ARG and call(2, _lib.MAX_T_BLOCK + 1) == _lib.ERR_UNSUPPORTED and call(4, 9) == _lib.ERR_UNSUPPORTED
    assert call(6, sz.plan_bytes - 1) == _lib.ERR_WORKSPACE and call(8, 1) == _lib.ERR_WORKSPACE
    assert call(5, buf.data_ptr() + 8) == _lib.ERR_ALIGN
    info = B.PlanInfo()
    assert L.bload_plan_finish(buf.data_ptr(), None, C.byref(info)) == _lib.ERR_PLAN      # zeros: not a plan
    assert L.bload_plan_finish(None, None, C.byref(info)) == _lib.ERR_NULL
    assert L.bload_plan_finish(buf.data_ptr(), None, None) == _lib.ERR_NULL
    assert L.bload_plan_async(*args) == 0
    assert L.bload_plan_finish(buf.data_ptr(), None, C.byref(info)) == 0 and info.n_blocks == 2 and info.sum_t == 16
    # bad lengths surface at finish time
    bad = torch.tensor([3, 0, 2], dtype=torch.int32, device=G.DEV)
    pb, wk, s3 = B.bload_plan_async(bad, 4, 0)
    p = B.bload_plan_finish(pb, s3, check=False)
    assert p.info.status == _lib.ERR_LENGTH and p.info.first_bad_index == 1


def test_pack_and_unpack_of_two_plans_on_two_streams_at_once():
    """Two independent epochs handled concurrently on two streams (separate plans and buffers): the kernels keep no
    state outside their arguments, so both results must be exact."""
    w = W.scaled(W.WORKLOADS["features_fp16"], 600)
    T = W.lengths(w)
    fb = 64
    d_len = torch.from_numpy(T).to(G.DEV)
    jobs = []
    for e in range(2):
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            plan = B.bload_plan(d_len, w.t_block, 50 + e, policy=e)
            op = O.plan(T, w.t_block, 50 + e, policy=e)
            store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
            dense = torch.empty(op.n_blocks * w.t_block * fb, dtype=torch.uint8, device=G.DEV)
            back = torch.empty_like(store)
        jobs.append((s, plan, op, store, dense, back))
    for _ in range(3):                       # interleave the launches of the two streams
        for s, plan, op, store, dense, back in jobs:
            with torch.cuda.stream(s):
                B.bload_pack(plan, store, fb, 0, op.n_blocks, dense=dense)
                B.bload_unpack(plan, dense, fb, 0, op.n_blocks, back)
    torch.cuda.synchronize()
    for s, plan, op, store, dense, back in jobs:
        assert np.array_equal(dense.cpu().numpy().reshape(op.n_blocks, w.t_block, fb),
                              O.pack(op, store.cpu().numpy(), fb, 0, op.n_blocks, 0))
        assert torch.equal(back, store)
