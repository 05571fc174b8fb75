"""GPU parity at the full sizes of the three large evaluation configurations, in the launch
configuration the benchmark times (one whole-epoch call per direction).  The plan is compared with
the oracle table by table; the packed bytes, the per-slot metadata and the unpacked per-frame
outputs of EVERY block are compared with the oracle, slab by slab so that host memory stays bounded
(one slab of dense blocks at a time; only the ragged arrays are held whole)."""
import numpy as np
import pytest
import torch

import gpu_util as G
import paper_2310_10879_b200 as B
from oracle import bload_oracle as O
from paper_2310_10879_b200 import workloads as W

pytestmark = pytest.mark.gpu

SLAB_BYTES = 1 << 30   # dense bytes compared per step


def _slabs(n_blocks, block_bytes):
    step = max(1, SLAB_BYTES // block_bytes)
    return [(lo, min(step, n_blocks - lo)) for lo in range(0, n_blocks, step)]


def _assert_same(got: torch.Tensor, want: np.ndarray, what: str):
    d = G.first_diff(got.cpu().numpy(), want)
    assert d is None, what + ": " + d


def _run(name):
    _run_workload(W.WORKLOADS[name])


def _run_workload(w, carry=False):
    T = W.lengths(w)
    op = O.plan(T, w.t_block, w.seed)
    plan = G.gpu_plan(T, w.t_block, w.seed)
    G.assert_plan_equal(plan, op)
    fb, ofb, tb, nb = w.frame_bytes, w.out_frame_bytes, w.t_block, op.n_blocks
    store = W.payload_torch(w, op.sum_t, G.DEV)
    store_u8 = store.view(torch.uint8).reshape(-1)
    dense = G.Guarded(nb * tb * fb)
    B.bload_pack(plan, store_u8, fb, 0, nb, dense=dense.t, pad_byte=0)
    torch.cuda.synchronize()
    dense.check()
    store_h = store_u8.cpu().numpy()
    # every block of the whole-epoch launch against the oracle (padding included: the oracle writes it too)
    d3 = dense.t.view(nb, tb * fb)
    for lo, cnt in _slabs(nb, tb * fb):
        _assert_same(d3[lo:lo + cnt], O.pack(op, store_h, fb, lo, cnt, 0), "packed bytes of blocks %d..%d" % (lo, lo + cnt))
    del store_h
    # per-slot metadata of the whole epoch in one call: every block against the oracle, and the counts
    meta = [torch.empty(nb * tb, dtype=d, device=G.DEV) for d in (torch.int32, torch.int32, torch.uint8, torch.uint8)]
    B.bload_pack(plan, None, fb, 0, nb, seq_id=meta[0], pos=meta[1], reset=meta[2], valid=meta[3])
    torch.cuda.synchronize()
    for lo, cnt in _slabs(nb, tb * 10):
        for nm, got, want in zip(("seq_id", "pos", "reset", "valid"), meta, O.metadata(op, lo, cnt)):
            _assert_same(got.view(nb, tb)[lo:lo + cnt], want, "%s of blocks %d..%d" % (nm, lo, lo + cnt))
    assert int(meta[3].sum(dtype=torch.int64)) == op.sum_t and int(meta[2].sum(dtype=torch.int64)) == op.n
    del meta
    # round trip of the input itself (same frame size): unpack(pack(x)) == x, every byte
    back = G.Guarded(op.sum_t * fb, 0x5A)
    B.bload_unpack(plan, dense.t, fb, 0, nb, back.t)
    torch.cuda.synchronize(); back.check()
    assert torch.equal(back.t, store_u8)
    del back, dense, d3, store, store_u8
    torch.cuda.empty_cache()
    # unpack of a per-frame output (fp32 of the same shape for the bf16 workload): every sequence against the oracle
    out = W.payload_torch(w, nb * tb, G.DEV, out=True)          # dense per-frame outputs
    out_u8 = out.view(torch.uint8).reshape(nb, tb * ofb)
    rag = G.Guarded(op.sum_t * ofb, 0x5A)
    B.bload_unpack(plan, out_u8, ofb, 0, nb, rag.t)
    torch.cuda.synchronize(); rag.check()
    want = np.full(op.sum_t * ofb, 0x5A, np.uint8)
    for lo, cnt in _slabs(nb, tb * ofb):
        O.unpack(op, out_u8[lo:lo + cnt].cpu().numpy(), ofb, lo, cnt, want)
    step = 1 << 30
    for lo in range(0, want.size, step):
        _assert_same(rag.t[lo:lo + step], want[lo:lo + step], "unpacked bytes from %d" % lo)
    st = B.bload_stats(plan.info)
    assert st["pad_packed"] == nb * tb - op.sum_t and st["pad_naive_tmax"] == op.n * op.t_max - op.sum_t
    if carry:  # the consumer-side shifted copy of the same per-frame outputs, every block
        del rag, want
        prev = G.Guarded(nb * tb * ofb, 0x3C)
        B.bload_carry_prev(plan, out_u8.reshape(-1), ofb, 0, nb, prev.t, fill_byte=0xE7)
        torch.cuda.synchronize(); prev.check()
        p3 = prev.t.view(nb, tb * ofb)
        for lo, cnt in _slabs(nb, tb * ofb):
            _assert_same(p3[lo:lo + cnt], O.carry_prev(op, out_u8[lo:lo + cnt].cpu().numpy().reshape(-1), ofb, lo, cnt, 0xE7),
                         "carry_prev of blocks %d..%d" % (lo, lo + cnt))


def test_full_size_raw_frames():
    _run("raw_frames")


def test_full_size_tokens():
    _run("tokens")


def test_full_size_heavy_tail_bf16_with_fp32_outputs():
    _run("heavy_tail_bf16")


@pytest.mark.parametrize("name,n,fb", [("video_dataset_shape", 1_000_000, 8), ("heavy_tail_bf16", 1_000_000, 4),
                                       ("video_dataset_shape", 600_000, 6), ("tokens", 120_000, 16),
                                       ("video_dataset_shape", 400_000, 12)])
def test_a_million_short_runs(name, n, fb):
    """The word-wise kernels at scale: a million clips of 22 frames with 8-byte records (blocks of 94 slots), a million
    heavy-tailed sequences of 4-byte frames, 6-byte and 12-byte records, 16-byte frames with token lengths.  Plan, packed
    bytes, metadata, unpacked bytes and the shifted copy of every block against the oracle; thousands of windows per
    warp, warps that begin inside runs, padding and the filler tail."""
    from dataclasses import replace
    w = replace(W.scaled(W.WORKLOADS[name], n), frame_bytes=fb, out_frame_bytes=fb, payload="u8")
    _run_workload(w, carry=True)


@pytest.mark.parametrize("name", ["tokens", "heavy_tail_bf16"])
def test_full_size_epoch_call_equals_the_separate_calls(name):
    """bload_epoch at full size, in the configuration the benchmark times (two streams, the chain's stream with the
    higher priority): every table and every output byte equals what the separate calls give, which the tests above
    compare with the oracle."""
    w = W.WORKLOADS[name]
    T = W.lengths(w)
    d_len = torch.from_numpy(T).to(G.DEV)
    fb, ofb, tb = w.frame_bytes, w.out_frame_bytes, w.t_block
    ref = B.bload_plan(d_len, tb, w.seed)
    nb = ref.n_blocks
    store = W.payload_torch(w, ref.sum_t, G.DEV).view(torch.uint8).reshape(-1)
    dense_out = torch.randint(0, 256, (nb * tb * ofb,), dtype=torch.uint8, device=G.DEV)
    want_dense = torch.empty(nb * tb * fb, dtype=torch.uint8, device=G.DEV)
    want_meta = [torch.empty(nb * tb, dtype=d, device=G.DEV) for d in (torch.int32, torch.int32, torch.uint8, torch.uint8)]
    want_rag = torch.empty(ref.sum_t * ofb, dtype=torch.uint8, device=G.DEV)
    B.bload_pack(ref, store, fb, 0, nb, dense=want_dense, seq_id=want_meta[0], pos=want_meta[1], reset=want_meta[2],
                 valid=want_meta[3])
    B.bload_unpack(ref, dense_out, ofb, 0, nb, want_rag)
    got_dense = G.Guarded(nb * tb * fb)
    got_meta = [torch.full_like(x, 0x11) for x in want_meta]
    got_rag = G.Guarded(ref.sum_t * ofb, 0x5A)
    chain, side = torch.cuda.Stream(priority=-1), torch.cuda.Stream()
    chain.wait_stream(torch.cuda.current_stream())
    plan = B.bload_epoch(d_len, tb, w.seed, nb, store=store, frame_bytes=fb, dense=got_dense.t, seq_id=got_meta[0],
                         pos=got_meta[1], reset=got_meta[2], valid=got_meta[3], dense_out=dense_out, out_frame_bytes=ofb,
                         ragged_out=got_rag.t, stream=chain, side_stream=side)
    torch.cuda.synchronize()
    got_dense.check(); got_rag.check()
    assert plan.info.checksum == ref.info.checksum and plan.n_blocks == nb
    for k, t in plan.tables().items():
        assert torch.equal(t, ref.tables()[k]), k
    assert torch.equal(got_dense.t, want_dense)
    for a, b in zip(got_meta, want_meta):
        assert torch.equal(a, b)
    assert torch.equal(got_rag.t, want_rag)


@pytest.mark.parametrize("tail", [O.KEEP_TAIL, O.DROP_TAIL])
def test_full_size_chunking_planner_on_the_token_lengths(tail):
    """The chunking planner at a million sequences (2.4 / 1.6 million chunks of 512 tokens): totals, every table and the
    digest against the oracle, and the packed bytes of every block through the ordinary pack call, slab by slab."""
    w = W.WORKLOADS["tokens"]
    T = W.lengths(w)
    c, fb = 512, w.frame_bytes
    ch = O.chunks(T, c, tail)
    plan, ci, cseq, cfirst = B.bload_plan_chunks(torch.from_numpy(T).to(G.DEV), c, tail)
    assert (ci.n_chunks, ci.frames_kept, ci.frames_deleted, ci.pad_frames, ci.sum_t) == \
        (ch.n_chunks, ch.frames_kept, ch.frames_deleted, ch.pad_frames, ch.sum_t)
    assert np.array_equal(cseq.cpu().numpy(), ch.chunk_seq) and np.array_equal(cfirst.cpu().numpy(), ch.chunk_first)
    G.assert_plan_equal(plan, ch.as_plan(), maximal=False, invariants_too=tail == O.KEEP_TAIL)
    store = W.payload_torch(w, ch.sum_t, G.DEV).view(torch.uint8).reshape(-1)
    nb = ch.n_chunks
    dense = G.Guarded(nb * c * fb)
    B.bload_pack(plan, store, fb, 0, nb, dense=dense.t)
    torch.cuda.synchronize(); dense.check()
    store_h = store.cpu().numpy()
    d2 = dense.t.view(nb, c * fb)
    for lo, cnt in _slabs(nb, c * fb):
        _assert_same(d2[lo:lo + cnt], O.chunk_pack(ch, store_h, fb, lo, cnt, 0), "chunk blocks %d..%d" % (lo, lo + cnt))
    # unpack: kept frames come back, deleted frames keep the canary value
    back = G.Guarded(ch.sum_t * fb, 0x5A)
    B.bload_unpack(plan, dense.t, fb, 0, nb, back.t)
    torch.cuda.synchronize(); back.check()
    want = np.full(ch.sum_t * fb, 0x5A, np.uint8)
    for lo, cnt in _slabs(nb, c * fb):
        O.chunk_unpack(ch, d2[lo:lo + cnt].cpu().numpy(), fb, lo, cnt, want)
    step = 1 << 30
    for lo in range(0, want.size, step):
        _assert_same(back.t[lo:lo + step], want[lo:lo + step], "unpacked bytes from %d" % lo)
