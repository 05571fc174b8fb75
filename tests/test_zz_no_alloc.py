"""The allocation-free planner entry point, bload_plan_static.

Some users of the library cannot allocate device memory when they need a plan (a loader thread
next to a training job whose allocator already owns the GPU, or code that is not allowed to call
cudaMalloc because of the device-wide stall it can cause).  For them the library carries its own
fixed scratch array.  This file checks, through the C ABI, that the variant produces exactly the
plan of the regular entry point -- all tables and scalars, bit for bit -- on two calls in a row
that share the scratch array, and that it refuses problems larger than the array.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2310_10879_b200 as B
from paper_2310_10879_b200 import _lib
from paper_2310_10879_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TABLES = ("offsets", "seg_seq", "seg_block", "seg_start", "seg_src", "block_seg_begin", "block_fill", "seq_block",
          "seq_start")
SCALARS = ("status", "t_block", "n", "n_blocks", "sum_t", "t_max", "first_bad_index", "checksum",
           "max_segs_per_block", "seed", "policy")


def _same_plan(a, b):
    for k in SCALARS:
        assert getattr(a.info, k) == getattr(b.info, k), k
    ta, tb = a.tables(), b.tables()
    for k in TABLES:
        assert torch.equal(ta[k], tb[k]), k


def _memory_state():
    """What an allocation anywhere would change: the number of blocks torch's allocator has ever handed out, the number
    of segments it has ever taken from the driver (both only grow; tensors of earlier tests that are freed meanwhile do
    not move them), and the driver's free bytes."""
    st = torch.cuda.memory_stats(DEV)
    return (st["allocation.all.allocated"], st["segment.all.allocated"], torch.cuda.mem_get_info(DEV)[0])


@pytest.mark.parametrize("policy", [0, 1])
def test_static_scratch_plan_equals_regular_plan_on_two_calls_in_a_row(policy):
    cases = [(W.lengths(W.scaled(W.WORKLOADS["heavy_tail_bf16"], 20000)), 10000, 11),   # larger problem first ...
             (W.lengths(W.scaled(W.WORKLOADS["tokens"], 3000)), 4096, 12),              # ... then a smaller one on the
             (W.TOY8_LENGTHS, W.TOY8_T_BLOCK, 13)]                                      # leftovers of the previous call
    # everything that allocates happens first: inputs, the caller's plan buffers, the regular entry point's plans
    prepared = []
    for T, tb, seed in cases:
        d_len = torch.from_numpy(np.ascontiguousarray(T, np.int32)).to(DEV)
        sizes = B.bload_plan_sizes(T.size, tb)
        plan_buf = torch.empty(sizes.plan_bytes, dtype=torch.uint8, device=DEV)   # the caller's output buffer
        prepared.append((d_len, tb, seed, plan_buf, B.bload_plan(d_len, tb, seed, policy=policy)))
    B.bload_plan_static(prepared[0][0], prepared[0][1], 0, policy=policy, plan_buf=prepared[0][3])  # first call on the device: looks the array up
    torch.cuda.synchronize()
    # then the static calls, back to back on the shared array, with no allocation by anyone in between
    before = _memory_state()
    got_all = [B.bload_plan_static(d_len, tb, seed, policy=policy, plan_buf=plan_buf)
               for d_len, tb, seed, plan_buf, _ in prepared]
    torch.cuda.synchronize()
    after = _memory_state()
    assert after[:2] == before[:2] and after[2] >= before[2], "bload_plan_static took device memory: %s -> %s" % (before, after)
    for (d_len, tb, seed, plan_buf, want), got in zip(prepared, got_all):
        _same_plan(got, want)
        # and the plan is usable by the rest of the library
        fb = 16
        if policy:
            continue
        store = torch.randint(0, 256, (got.sum_t * fb,), dtype=torch.uint8, device=DEV)
        d1 = torch.empty(got.n_blocks * tb * fb, dtype=torch.uint8, device=DEV)
        d2 = torch.empty_like(d1)
        B.bload_pack(got, store, fb, 0, got.n_blocks, dense=d1)
        B.bload_pack(want, store, fb, 0, want.n_blocks, dense=d2)
        assert torch.equal(d1, d2)


def test_static_scratch_reports_bad_lengths_like_the_regular_entry_point():
    T = np.ones(5000, np.int32); T[4321] = 9
    d_len = torch.from_numpy(T).to(DEV)
    got = B.bload_plan_static(d_len, 8, 0, check=False)
    want = B.bload_plan(d_len, 8, 0, check=False)
    assert got.info.status == want.info.status == _lib.ERR_LENGTH
    assert got.info.first_bad_index == want.info.first_bad_index == 4321


def test_static_scratch_rejects_sizes_beyond_its_array():
    n = _lib.STATIC_MAX_N + 1
    d_len = torch.ones(n, dtype=torch.int32, device=DEV)
    with pytest.raises(B.BloadError) as ei:
        B.bload_plan_static(d_len, 8, 0)
    assert ei.value.code == _lib.ERR_WORKSPACE
    # at the limit it still works
    d_len = torch.ones(_lib.STATIC_MAX_N, dtype=torch.int32, device=DEV)
    p = B.bload_plan_static(d_len, 32768, 0)
    assert p.n_blocks == 2 and p.sum_t == _lib.STATIC_MAX_N
    info = B.PlanInfo()
    L = B.load()
    assert L.bload_plan_static(None, 4, 4, 0, 0, None, 0, None, C.byref(info)) == _lib.ERR_NULL


def test_static_scratch_has_no_room_for_best_fit_decreasing():
    d_len = torch.ones(100, dtype=torch.int32, device=DEV)
    with pytest.raises(B.BloadError) as ei:
        B.bload_plan_static(d_len, 8, 0, policy=2)
    assert ei.value.code == _lib.ERR_UNSUPPORTED
