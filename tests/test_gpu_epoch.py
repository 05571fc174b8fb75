"""bload_epoch (plan, metadata, pack and unpack of a whole epoch with the copies running under the plan) against
the oracle and against the separate calls, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

import gpu_util as G
import paper_2310_10879_b200 as B
from oracle import bload_oracle as O
from paper_2310_10879_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _epoch_parity(T, tb, seed, fb, ofb, extra=2, pad=0x2D, side=True, payload_seed=1):
    T = np.ascontiguousarray(T, np.int32)
    op = O.plan(T, tb, seed)
    cap = op.n_blocks + extra
    g = torch.Generator(device=G.DEV); g.manual_seed(payload_seed)
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV, generator=g)
    dense_out = torch.randint(0, 256, (cap * tb * ofb,), dtype=torch.uint8, device=G.DEV, generator=g)
    dense = G.Guarded(cap * tb * fb)
    meta = dict(seq_id=G.Guarded(cap * tb * 4, 0x11), pos=G.Guarded(cap * tb * 4, 0x11),
                reset=G.Guarded(cap * tb, 0x11), valid=G.Guarded(cap * tb, 0x11))
    rag = G.Guarded(op.sum_t * ofb, 0x5A)
    d_len = torch.from_numpy(T).to(G.DEV)
    s2 = torch.cuda.Stream() if side else None
    plan = B.bload_epoch(d_len, tb, seed, cap, store=store, frame_bytes=fb, dense=dense.t,
                         seq_id=meta["seq_id"].t.view(torch.int32), pos=meta["pos"].t.view(torch.int32),
                         reset=meta["reset"].t, valid=meta["valid"].t, pad_byte=pad, dense_out=dense_out,
                         out_frame_bytes=ofb, ragged_out=rag.t, side_stream=s2)
    # the call has synchronised: everything is complete
    G.assert_plan_equal(plan, op)
    for x in (dense, rag, *meta.values()):
        x.check()
    d = G.first_diff(dense.t.cpu().numpy(), O.pack(op, store.cpu().numpy(), fb, 0, cap, pad))
    assert d is None, "packed bytes: " + d
    for name, want in zip(("seq_id", "pos", "reset", "valid"), O.metadata(op, 0, cap)):
        got = meta[name].t.view(torch.int32 if name in ("seq_id", "pos") else torch.uint8).cpu().numpy().reshape(cap, tb)
        assert np.array_equal(got, want), name
    want_r = np.full(op.sum_t * ofb, 0x5A, np.uint8)
    O.unpack(op, dense_out.cpu().numpy(), ofb, 0, cap, want_r)
    d = G.first_diff(rag.t.cpu().numpy(), want_r)
    assert d is None, "unpacked bytes: " + d
    return plan, op


@pytest.mark.parametrize("n,tb,fb,ofb", [(8, 6, 12288, 16), (300, 40, 64, 128), (3000, 64, 100, 36), (5000, 200, 16, 16),
                                         (20000, 100, 8, 4), (40000, 50, 4, 12), (2600, 1000, 2048, 2048)])
def test_epoch_matches_the_oracle(n, tb, fb, ofb):
    rng = np.random.default_rng(n + tb)
    T = np.minimum(rng.geometric(1.0 / max(2, tb // 5), size=n), tb)
    _epoch_parity(T, tb, 1234 + n, fb, ofb)


def test_epoch_workloads_and_single_stream():
    w = W.scaled(W.WORKLOADS["heavy_tail_bf16"], 6000)
    _epoch_parity(W.lengths(w), w.t_block, w.seed, 256, 512, extra=1)
    w = W.scaled(W.WORKLOADS["tokens"], 50000)
    _epoch_parity(W.lengths(w), w.t_block, w.seed, 4, 4)
    w = W.WORKLOADS["video_dataset_shape"]
    _epoch_parity(W.lengths(w), w.t_block, w.seed, w.frame_bytes, w.frame_bytes, side=False)
    _epoch_parity(W.TOY8_LENGTHS, W.TOY8_T_BLOCK, 3, 48, 48, extra=0)


def test_epoch_equals_the_separate_calls_and_repeats_exactly():
    w = W.scaled(W.WORKLOADS["heavy_tail_bf16"], 8000)
    T = W.lengths(w); tb = w.t_block; fb = 64
    d_len = torch.from_numpy(T).to(G.DEV)
    ref = B.bload_plan(d_len, tb, w.seed)
    cap = ref.n_blocks + 3
    store = torch.randint(0, 256, (ref.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    want = torch.empty(cap * tb * fb, dtype=torch.uint8, device=G.DEV)
    B.bload_pack(ref, store, fb, 0, cap, dense=want, pad_byte=7)
    side = torch.cuda.Stream()
    sizes = B.bload_plan_sizes(T.size, tb)
    work = torch.empty(sizes.work_bytes, dtype=torch.uint8, device=G.DEV)
    for rep in range(3):  # the same scratch and plan buffers again and again
        got = torch.full_like(want, 0xEE)
        plan = B.bload_epoch(d_len, tb, w.seed, cap, store=store, frame_bytes=fb, dense=got, pad_byte=7,
                             side_stream=side, work=work)
        assert plan.info.checksum == ref.info.checksum and plan.n_blocks == ref.n_blocks
        for name, t in plan.tables().items():
            assert torch.equal(t, ref.tables()[name]), "%s differs in repetition %d" % (name, rep)
        assert torch.equal(got, want)


def test_epoch_capacity_too_small_and_bad_arguments():
    rng = np.random.default_rng(3)
    T = rng.integers(1, 30, size=4000).astype(np.int32)
    op = O.plan(T, 30, 9)
    d_len = torch.from_numpy(T).to(G.DEV)
    fb = 16
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    cap = op.n_blocks - 5
    dense = G.Guarded(cap * 30 * fb)
    with pytest.raises(B.BloadError) as e:
        B.bload_epoch(d_len, 30, 9, cap, store=store, frame_bytes=fb, dense=dense.t, side_stream=torch.cuda.Stream())
    assert e.value.code == -4 and e.value.info.n_blocks == op.n_blocks
    torch.cuda.synchronize(); dense.check()
    # the blocks that fit were packed
    assert np.array_equal(dense.t.cpu().numpy().reshape(cap, 30, fb), O.pack(op, store.cpu().numpy(), fb, 0, cap, 0))
    with pytest.raises(B.BloadError) as e:
        B.bload_epoch(d_len, 30, 9, 0, store=store, frame_bytes=fb, dense=dense.t)
    assert e.value.code == -2
    with pytest.raises(B.BloadError) as e:
        B.bload_epoch(d_len, 30, 9, cap, store=None, frame_bytes=fb, dense=dense.t)
    assert e.value.code == -1
    bad = T.copy(); bad[77] = 31
    with pytest.raises(B.BloadError) as e:
        B.bload_epoch(torch.from_numpy(bad).to(G.DEV), 30, 9, cap, store=store, frame_bytes=fb, dense=dense.t)
    assert e.value.code == -3 and e.value.info.first_bad_index == 77


@pytest.mark.parametrize("chunks", [1, 2, 7, 32])
def test_epoch_with_any_number_of_chunks(chunks):
    # the number of launches of the fill rule changes where the chain pauses, never what it computes: few draws per
    # chunk (chunks that end after one block), chunks that find the plan already finished, a single chunk
    rng = np.random.default_rng(chunks)
    tb = 64
    T = np.minimum(rng.geometric(1.0 / 9, size=700), tb).astype(np.int32)
    op = O.plan(T, tb, 5)
    cap = op.n_blocks + 1
    fb = 32
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    dense = G.Guarded(cap * tb * fb)
    valid = torch.empty(cap * tb, dtype=torch.uint8, device=G.DEV)
    plan = B.bload_epoch(torch.from_numpy(T).to(G.DEV), tb, 5, cap, store=store, frame_bytes=fb, dense=dense.t,
                         valid=valid, side_stream=torch.cuda.Stream(), chunks=chunks)
    dense.check()
    G.assert_plan_equal(plan, op)
    assert np.array_equal(dense.t.cpu().numpy().reshape(cap, tb, fb), O.pack(op, store.cpu().numpy(), fb, 0, cap, 0))
    assert np.array_equal(valid.cpu().numpy().reshape(cap, tb), O.metadata(op, 0, cap)[3])
    # a tiny problem with more chunks than sequences
    T2 = np.array([3, 1, 2], np.int32)
    op2 = O.plan(T2, 3, 1)
    d2 = torch.empty(op2.n_blocks * 3 * 8, dtype=torch.uint8, device=G.DEV)
    s2 = torch.randint(0, 256, (op2.sum_t * 8,), dtype=torch.uint8, device=G.DEV)
    p2 = B.bload_epoch(torch.from_numpy(T2).to(G.DEV), 3, 1, op2.n_blocks, store=s2, frame_bytes=8, dense=d2, chunks=chunks)
    G.assert_plan_equal(p2, op2)
    assert np.array_equal(d2.cpu().numpy().reshape(op2.n_blocks, 3, 8), O.pack(op2, s2.cpu().numpy(), 8, 0, op2.n_blocks, 0))
