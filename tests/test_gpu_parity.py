"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, bit for bit."""
import ctypes as C

import numpy as np
import pytest
import torch

import gpu_util as G
import paper_2310_10879_b200 as B
from oracle import bload_oracle as O
from paper_2310_10879_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_toy8_of_the_paper():
    for seed in range(20):
        for fb in (12288, 1):
            G.full_parity(W.TOY8_LENGTHS, W.TOY8_T_BLOCK, seed, fb, payload_seed=seed)


def test_config_toy_video():
    w = W.WORKLOADS["toy_video"]
    plan, op = G.full_parity(W.lengths(w), w.t_block, w.seed, w.frame_bytes)
    # batches of 8 blocks, the last one rounded up with filler blocks
    store = W.payload_torch(w, op.sum_t, G.DEV).view(torch.uint8).reshape(-1)
    store_h = store.cpu().numpy()
    for b0 in range(0, op.n_blocks, w.batch_blocks):
        res, _ = G.gpu_pack_all(plan, store, w.frame_bytes, b0, w.batch_blocks, 0)
        assert np.array_equal(res["dense"], O.pack(op, store_h, w.frame_bytes, b0, w.batch_blocks, 0))
        for name, want in zip(("seq_id", "pos", "reset", "valid"), O.metadata(op, b0, w.batch_blocks)):
            assert np.array_equal(res[name], want)


def test_config_features_fp16():
    w = W.WORKLOADS["features_fp16"]
    G.full_parity(W.lengths(w), w.t_block, w.seed, w.frame_bytes)


def test_config_raw_frames_scaled():
    w = W.scaled(W.WORKLOADS["raw_frames"], 40)
    G.full_parity(W.lengths(w), w.t_block, w.seed, w.frame_bytes, extra_blocks=1)


def test_config_tokens_scaled():
    w = W.scaled(W.WORKLOADS["tokens"], 30000)
    G.full_parity(W.lengths(w), w.t_block, w.seed, w.frame_bytes)


def test_config_heavy_tail_scaled_with_fp32_outputs():
    w = W.scaled(W.WORKLOADS["heavy_tail_bf16"], 1200)
    G.full_parity(W.lengths(w), w.t_block, w.seed, w.frame_bytes, out_fb=w.out_frame_bytes, extra_blocks=1)


def test_dataset_shaped_lengths():
    w = W.WORKLOADS["video_dataset_shape"]
    plan, op = G.full_parity(W.lengths(w), w.t_block, w.seed, w.frame_bytes)
    s = B.bload_stats(plan.info)
    assert s == {**O.stats(op.n, op.sum_t, op.t_max, op.t_block, op.n_blocks),
                 "max_segs_per_block": op.max_segs_per_block, "frames_deleted": 0}


@pytest.mark.parametrize("fb", [1, 2, 3, 4, 6, 8, 12, 20, 24, 48, 100, 1000, 4100])
@pytest.mark.parametrize("pad", [0, 0x7F])
def test_frame_sizes_and_alignments(fb, pad):
    """Frame sizes that are not multiples of 16 exercise every relative misalignment of source and
    destination runs (byte, 2-, 4-, 8-byte granules) and the head/tail handling."""
    rng = np.random.default_rng(fb * 31 + pad)
    tb = int(rng.integers(5, 200))
    T = rng.integers(1, tb + 1, size=int(rng.integers(1, 300))).astype(np.int32)
    G.full_parity(T, tb, int(rng.integers(0, 1 << 40)), fb, out_fb=fb + (fb % 3), pad=pad)


@pytest.mark.parametrize("case", ["one", "all_full", "all_ones", "block_of_one", "max_t_block", "many_short",
                                  "two_lengths"])
def test_degenerate_plans(case):
    rng = np.random.default_rng(1)
    if case == "one":
        T, tb = np.array([5], np.int32), 9
    elif case == "all_full":
        T, tb = np.full(300, 17, np.int32), 17
    elif case == "all_ones":
        T, tb = np.ones(5000, np.int32), 33
    elif case == "block_of_one":
        T, tb = np.ones(70, np.int32), 1
    elif case == "max_t_block":
        tb = 32768
        T = np.concatenate([rng.integers(1, tb + 1, size=40), [tb, tb, 1, 1, 255, 256, 257]]).astype(np.int32)
    elif case == "many_short":
        T, tb = rng.integers(1, 4, size=9000).astype(np.int32), 4096      # thousands of segments per block
    else:
        T, tb = rng.choice([3, 700], size=4097).astype(np.int32), 1000
    G.full_parity(T, tb, 77, 8 if case in ("max_t_block", "many_short") else 20)


@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 255, 256, 257, 2047, 2048, 2049, 4096, 70001])
def test_plan_sizes_around_tile_boundaries(n):
    rng = np.random.default_rng(n)
    tb = 300
    T = rng.integers(1, tb + 1, size=n).astype(np.int32)
    for seed in (0, 2**63 + 11):
        G.assert_plan_equal(G.gpu_plan(T, tb, seed), O.plan(T, tb, seed))


def test_many_seeds_small():
    T = W.lengths(W.WORKLOADS["features_fp16"])[:200]
    for seed in range(40):
        G.assert_plan_equal(G.gpu_plan(T, 1000, seed), O.plan(T, 1000, seed))


def test_block_ranges_and_partial_unpack():
    w = W.scaled(W.WORKLOADS["features_fp16"], 400)
    T = W.lengths(w)
    op = O.plan(T, w.t_block, 9)
    plan = G.gpu_plan(T, w.t_block, 9)
    fb = 40
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    store_h = store.cpu().numpy()
    for b0, cnt in [(0, 1), (3, 4), (op.n_blocks - 1, 1), (op.n_blocks - 1, 3), (op.n_blocks + 5, 2), (2, 0)]:
        res, _ = G.gpu_pack_all(plan, store, fb, b0, cnt, 0x33)
        assert np.array_equal(res["dense"], O.pack(op, store_h, fb, b0, cnt, 0x33))
        for name, want in zip(("seq_id", "pos", "reset", "valid"), O.metadata(op, b0, cnt)):
            assert np.array_equal(res[name], want)
        dense_out = torch.randint(0, 256, (cnt * w.t_block * fb,), dtype=torch.uint8, device=G.DEV)
        rag = G.Guarded(op.sum_t * fb, 0x5A)
        B.bload_unpack(plan, dense_out, fb, b0, cnt, rag.t)
        torch.cuda.synchronize(); rag.check()
        want = np.full(op.sum_t * fb, 0x5A, np.uint8)
        O.unpack(op, dense_out.cpu().numpy(), fb, b0, cnt, want)
        assert np.array_equal(rag.t.cpu().numpy(), want)


def test_metadata_only_and_dense_only_calls():
    T = W.lengths(W.scaled(W.WORKLOADS["features_fp16"], 100))
    op = O.plan(T, 1000, 4); plan = G.gpu_plan(T, 1000, 4)
    valid = torch.zeros(op.n_blocks * 1000, dtype=torch.uint8, device=G.DEV)
    B.bload_pack(plan, None, 16, 0, op.n_blocks, valid=valid)
    assert np.array_equal(valid.cpu().numpy().reshape(op.n_blocks, 1000), O.metadata(op, 0, op.n_blocks)[3])
    # odd t_block and unaligned metadata pointers take the scalar path
    T = np.array([3, 4, 2, 7, 1, 6], np.int32)
    op = O.plan(T, 7, 1); plan = G.gpu_plan(T, 7, 1)
    raw = torch.zeros(op.n_blocks * 7 + 3, dtype=torch.uint8, device=G.DEV)
    B.bload_pack(plan, None, 16, 0, op.n_blocks, reset=raw[1:1 + op.n_blocks * 7])
    assert np.array_equal(raw[1:1 + op.n_blocks * 7].cpu().numpy().reshape(op.n_blocks, 7),
                          O.metadata(op, 0, op.n_blocks)[2])


@pytest.mark.parametrize("tb", [1, 2, 3, 5, 6, 94, 96, 777, 1023, 1024, 1025, 1300, 2500, 4097, 10001])
def test_metadata_for_blocks_of_any_length(tb):
    """Metadata-only calls over block lengths around the kernels' shapes: blocks shorter than a CTA's 1,024 slots and blocks
    whose length is not a multiple of 4 take the kernel that treats the call's blocks as one array (quads that run through
    the ends of one to four blocks), the others the chunked kernel; whole plans with filler blocks, sub-ranges that start
    anywhere, unaligned output pointers, a subset of the four arrays; canaries around every output."""
    rng = np.random.default_rng(tb)
    n = int(min(4000, max(6, 400_000 // tb)))
    T = rng.integers(1, tb + 1, size=n).astype(np.int32)
    op = O.plan(T, tb, 12); plan = G.gpu_plan(T, tb, 12)
    nb = op.n_blocks
    for b0, cnt in [(0, nb + 3), (1, max(nb - 2, 1)), (nb // 2, 1), (nb - 1, 3), (nb + 1, 2)]:
        slots = cnt * tb
        outs = dict(seq_id=G.Guarded(slots * 4, 0x11), pos=G.Guarded(slots * 4, 0x11), reset=G.Guarded(slots, 0x11),
                    valid=G.Guarded(slots, 0x11))
        B.bload_pack(plan, None, 8, b0, cnt, seq_id=outs["seq_id"].t.view(torch.int32), pos=outs["pos"].t.view(torch.int32),
                     reset=outs["reset"].t, valid=outs["valid"].t)
        torch.cuda.synchronize()
        want = O.metadata(op, b0, cnt)
        for (name, g), w in zip(outs.items(), want):
            g.check()
            got = g.t.view(torch.int32) if name in ("seq_id", "pos") else g.t
            assert np.array_equal(got.cpu().numpy().reshape(cnt, tb), w), (name, b0, cnt)
    # two of the four arrays at addresses that rule out vector stores
    cnt = min(nb, 7)
    raw_pos = torch.full((cnt * tb + 3,), 77, dtype=torch.int32, device=G.DEV)
    raw_reset = torch.full((cnt * tb + 3,), 77, dtype=torch.uint8, device=G.DEV)
    B.bload_pack(plan, None, 8, 0, cnt, pos=raw_pos[1:1 + cnt * tb], reset=raw_reset[1:1 + cnt * tb])
    want = O.metadata(op, 0, cnt)
    assert np.array_equal(raw_pos[1:1 + cnt * tb].cpu().numpy().reshape(cnt, tb), want[1])
    assert np.array_equal(raw_reset[1:1 + cnt * tb].cpu().numpy().reshape(cnt, tb), want[2])
    assert int(raw_pos[0]) == 77 and int(raw_pos[-1]) == 77 and int(raw_reset[0]) == 77 and int(raw_reset[-2]) == 77


def test_bad_lengths_are_reported_not_faulted():
    for T, tb, bad in [([3, 0, 2], 4, 1), ([3, 4, 5, 2], 4, 2), ([3, -1], 4, 1)]:
        plan = G.gpu_plan(np.array(T, np.int32), tb, 0, check=False)
        op = O.plan(np.array(T, np.int32), tb, 0)
        assert plan.info.status == B._lib.ERR_LENGTH and op.status != 0
        assert plan.info.first_bad_index == bad == op.first_bad
        with pytest.raises(B.BloadError):
            B.bload_pack(plan, torch.zeros(64, dtype=torch.uint8, device=G.DEV), 1, 0, 1,
                         dense=torch.zeros(64, dtype=torch.uint8, device=G.DEV))
    big = np.ones(5000, np.int32); big[4321] = 9
    plan = G.gpu_plan(big, 8, 0, check=False)
    assert plan.info.first_bad_index == 4321
    # the context is still healthy
    G.assert_plan_equal(G.gpu_plan(np.ones(10, np.int32), 8, 0), O.plan(np.ones(10, np.int32), 8, 0))


def test_host_detected_errors_launch_nothing():
    L = B.load()
    e = B._lib
    d_len = torch.ones(16, dtype=torch.int32, device=G.DEV)
    sz = B.bload_plan_sizes(16, 8)
    plan_buf = torch.zeros(sz.plan_bytes + 256, dtype=torch.uint8, device=G.DEV)
    work = torch.zeros(sz.work_bytes + 256, dtype=torch.uint8, device=G.DEV)
    info = B.PlanInfo()

    def call(lengths=d_len.data_ptr(), n=16, tb=8, policy=0, plan=plan_buf.data_ptr(), pb=sz.plan_bytes,
             wk=work.data_ptr(), wb=sz.work_bytes):
        return L.bload_plan(lengths, n, tb, 0, policy, plan, pb, wk, wb, None, C.byref(info))

    assert call(lengths=None) == e.ERR_NULL and call(plan=None) == e.ERR_NULL and call(wk=None) == e.ERR_NULL
    assert call(n=0) == e.ERR_ARG and call(tb=0) == e.ERR_ARG
    assert call(tb=e.MAX_T_BLOCK + 1) == e.ERR_UNSUPPORTED and call(policy=3) == e.ERR_UNSUPPORTED
    assert call(policy=1) == 0
    assert call(pb=sz.plan_bytes - 1) == e.ERR_WORKSPACE and call(wb=sz.work_bytes - 1) == e.ERR_WORKSPACE
    assert call(plan=plan_buf.data_ptr() + 8) == e.ERR_ALIGN and call(wk=work.data_ptr() + 16) == e.ERR_ALIGN
    assert call() == 0
    p = B.Plan(plan_buf, info, sz)
    x = torch.zeros(4096, dtype=torch.uint8, device=G.DEV)
    for kwargs, code in [(dict(frame_bytes=0), e.ERR_ARG), (dict(block_begin=-1), e.ERR_ARG),
                         (dict(block_count=-1), e.ERR_ARG), (dict(block_begin=2**31 - 1, block_count=1), e.ERR_ARG)]:
        a = dict(frame_bytes=1, block_begin=0, block_count=1); a.update(kwargs)
        with pytest.raises(B.BloadError) as ei:
            B.bload_pack(p, x, a["frame_bytes"], a["block_begin"], a["block_count"], dense=x)
        assert ei.value.code == code
        with pytest.raises(B.BloadError) as ei:
            B.bload_unpack(p, x, a["frame_bytes"], a["block_begin"], a["block_count"], x)
        assert ei.value.code == code
    with pytest.raises(B.BloadError) as ei:
        B.bload_pack(p, x[4:], 1, 0, 1, dense=x)
    assert ei.value.code == e.ERR_ALIGN
    with pytest.raises(B.BloadError) as ei:
        B.bload_unpack(p, x, 1, 0, 1, x[8:])
    assert ei.value.code == e.ERR_ALIGN
    with pytest.raises(B.BloadError) as ei:
        B.bload_pack(p, None, 1, 0, 1, dense=x)
    assert ei.value.code == e.ERR_NULL
    torch.cuda.synchronize()


def test_plan_on_a_side_stream_and_reuse_of_buffers():
    T = W.lengths(W.scaled(W.WORKLOADS["tokens"], 5000))
    d_len = torch.from_numpy(T).to(G.DEV)
    sz = B.bload_plan_sizes(T.size, 4096)
    plan_buf = torch.empty(sz.plan_bytes, dtype=torch.uint8, device=G.DEV)
    work = torch.empty(sz.work_bytes, dtype=torch.uint8, device=G.DEV)
    s = torch.cuda.Stream()
    for seed in (1, 2, 1):
        with torch.cuda.stream(s):
            plan = B.bload_plan(d_len, 4096, seed, work=work, plan_buf=plan_buf)
        G.assert_plan_equal(plan, O.plan(T, 4096, seed))


@pytest.mark.parametrize("tb,fb,tmax", [(4, 4, 4), (64, 4, 64), (1000, 16, 9), (4096, 4, 4096), (4096, 8, 40),
                                        (20000, 36, 3000), (20000, 4, 20000), (700, 256, 300), (32768, 12, 5000),
                                        (5000, 64, 2), (2048, 20, 2048), (64, 1024, 8), (100, 4096, 3), (37, 16384, 1),
                                        (300, 2052, 6)])
def test_small_word_sized_frames_take_the_staged_path(tb, fb, tmax):
    """Word-sized frames whose runs are short on average (up to 16 KB) and whose blocks are multiples of 16 bytes go
    through the shared-memory staged kernels, the rest through the register path: many sub-tiles per block, runs cut by sub-tile ends, more than 32 runs per sub-tile,
    pad-only sub-tiles, filler blocks, a non-zero pad byte."""
    assert (tb * fb) % 16 == 0
    rng = np.random.default_rng(tb * 131 + fb)
    n = int(min(4000, max(3, 6_000_000 // (tmax * fb))))
    T = rng.integers(1, tmax + 1, size=n).astype(np.int32)
    T[rng.integers(0, n)] = tmax
    plan, op = G.full_parity(T, tb, 5, fb, out_fb=fb, pad=0xA7, extra_blocks=2)
    # a sub-range in the middle, as a training loop would request batch by batch
    if op.n_blocks > 3:
        store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
        res, _ = G.gpu_pack_all(plan, store, fb, 1, 2, 0, meta=False)
        assert np.array_equal(res["dense"], O.pack(op, store.cpu().numpy(), fb, 1, 2, 0))


@pytest.mark.parametrize("tb,fb,kind", [(4096, 4, "ones"), (4096, 4, "few_words"), (10000, 4, "heavy_tail"), (94, 8, "clips"),
                                        (94, 12, "clips"), (512, 36, "few_words"), (64, 256, "ones"), (4096, 4, "some_long"),
                                        (33, 4, "few_words"), (1000, 16, "one_sequence")])
def test_runs_of_a_few_words(tb, fb, kind):
    """Calls whose runs are short on average take the word-wise kernels (a lane finds the run of each of its words
    in a window of 32 runs): runs of one word (a window lasts 31 words), a few words, clip- and sentence-like lengths, a
    few runs as long as a block among thousands of tiny ones, windows that end inside a sub-tile and at its end, warps
    that start inside padding and inside filler blocks, totals that are not multiples of 16 bytes, sub-ranges."""
    rng = np.random.default_rng(tb * 31 + fb)
    if kind == "ones":
        T = np.ones(30011, np.int64)
    elif kind == "few_words":
        T = rng.integers(1, 6, size=40003)
    elif kind == "heavy_tail":
        T = W.lengths(W.scaled(W.WORKLOADS["heavy_tail_bf16"], 60000))
    elif kind == "clips":
        T = W.lengths(W.scaled(W.WORKLOADS["video_dataset_shape"], 50000))
    elif kind == "some_long":
        T = np.concatenate([rng.integers(1, 9, size=60000), np.full(25, tb), rng.integers(tb // 2, tb, size=20)])
    else:
        T = np.array([7])
    T = rng.permutation(np.minimum(T, tb)).astype(np.int32)
    want_k = G.expected_copy_kernels(int(T.sum()), len(T), fb, tb)
    assert want_k["pack_meta"] == "k17_pack_short_runs<metadata>"
    plan, op = G.full_parity(T, tb, 21, fb, out_fb=fb, pad=0xE1, extra_blocks=3)
    assert B.bload_last_copy_kernel("pack") == want_k["pack_meta"]
    assert B.bload_last_copy_kernel("unpack") == want_k["unpack"]
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    store_h = store.cpu().numpy()
    nb = op.n_blocks
    for b0, cnt in [(0, 1), (nb // 2, 3), (nb - 1, 3), (nb + 2, 2), (1, max(nb - 2, 1))]:
        res, _ = G.gpu_pack_all(plan, store, fb, b0, cnt, 0x4D, meta=False)
        assert B.bload_last_copy_kernel("pack") == want_k["pack"]
        d = G.first_diff(res["dense"].reshape(-1), O.pack(op, store_h, fb, b0, cnt, 0x4D).reshape(-1))
        assert d is None, "blocks [%d, +%d): %s" % (b0, cnt, d)
        # the same range back: the word-wise walk along the dense side, canaries around the output
        dense_out = torch.randint(0, 256, (cnt * tb * fb,), dtype=torch.uint8, device=G.DEV)
        rag = G.Guarded(op.sum_t * fb, 0x5A)
        B.bload_unpack(plan, dense_out, fb, b0, cnt, rag.t)
        torch.cuda.synchronize(); rag.check()
        assert B.bload_last_copy_kernel("unpack") == (want_k["unpack"] if b0 == 0 and cnt >= nb else want_k["unpack_range"])
        want = np.full(op.sum_t * fb, 0x5A, np.uint8)
        O.unpack(op, dense_out.cpu().numpy(), fb, b0, cnt, want)
        d = G.first_diff(rag.t.cpu().numpy(), want)
        assert d is None, "unpack of blocks [%d, +%d): %s" % (b0, cnt, d)


@pytest.mark.parametrize("tb,fb,tmax", [(94, 6, 94), (94, 3, 94), (4096, 2, 300), (4096, 1, 200), (1000, 30, 40), (33, 10, 33),
                                        (7, 1, 7), (1, 3, 1), (5000, 2, 1500), (640, 6, 400), (2000, 1, 700), (3000, 3, 600)])
def test_frames_that_are_not_multiples_of_4_bytes(tb, fb, tmax):
    """Even frame sizes that are not multiples of 4 take the unstaged walks with 2-byte words while their runs average at
    most 1.5 KB (pack) or 1 KB (unpack), odd sizes with 1-byte words up to 384 bytes; above that the register path.
    Blocks of 3 bytes to 30 KB, runs of 1 byte and up, padding, filler blocks, sub-ranges, canaries around every output;
    the last three cases sit at and above the cross-overs."""
    rng = np.random.default_rng(tb * 53 + fb)
    n = int(min(8000, max(3, 3_000_000 // (tmax * fb))))
    T = rng.integers(1, tmax + 1, size=n).astype(np.int32)
    T[rng.integers(0, n)] = tmax
    want_k = G.expected_copy_kernels(int(T.sum()), n, fb, tb)
    plan, op = G.full_parity(T, tb, 33, fb, out_fb=fb, pad=0x9C, extra_blocks=2)
    assert B.bload_last_copy_kernel("pack") == want_k["pack"] and B.bload_last_copy_kernel("unpack") == want_k["unpack"]
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    store_h = store.cpu().numpy()
    nb = op.n_blocks
    for b0, cnt in [(0, 1), (nb // 2, 2), (nb - 1, 3), (nb, 2)]:
        res, _ = G.gpu_pack_all(plan, store, fb, b0, cnt, 0x21, meta=False)
        d = G.first_diff(res["dense"].reshape(-1), O.pack(op, store_h, fb, b0, cnt, 0x21).reshape(-1))
        assert d is None, "blocks [%d, +%d): %s" % (b0, cnt, d)
        rag = G.Guarded(op.sum_t * fb, 0x5A)
        # (a block range must start 16-byte aligned in the caller's buffer: a fresh buffer per range)
        dense_out = torch.randint(0, 256, (cnt * tb * fb,), dtype=torch.uint8, device=G.DEV)
        B.bload_unpack(plan, dense_out, fb, b0, cnt, rag.t)
        torch.cuda.synchronize(); rag.check()
        assert B.bload_last_copy_kernel("unpack") == (want_k["unpack"] if b0 == 0 and cnt >= nb else want_k["unpack_range"])
        want = np.full(op.sum_t * fb, 0x5A, np.uint8)
        O.unpack(op, dense_out.cpu().numpy(), fb, b0, cnt, want)
        d = G.first_diff(rag.t.cpu().numpy(), want)
        assert d is None, "unpack of blocks [%d, +%d): %s" % (b0, cnt, d)


@pytest.mark.parametrize("tb,fb,tmax", [(94, 12, 94), (7, 12, 7), (94, 20, 94), (94, 100, 60), (5, 4, 5), (1, 4, 1), (3, 4, 3),
                                        (1234, 36, 600), (4097, 4, 4097), (10001, 12, 2000), (2049, 8, 2049)])
def test_pack_of_small_frames_in_blocks_of_any_size(tb, fb, tmax):
    """The staged pack kernel cuts the dense side of a call into sub-tiles as one array, so blocks need not be multiples
    of 16 bytes: blocks of 4 to 120,012 bytes that begin at every 4-byte offset, hundreds of blocks per sub-tile, blocks
    cut by sub-tile ends inside their frames and inside their padding, calls whose total is not a multiple of 16 bytes
    (the last words leave with plain stores), filler blocks, sub-ranges."""
    assert (tb * fb) % 16 != 0
    rng = np.random.default_rng(tb * 977 + fb)
    n = int(min(6000, max(3, 6_000_000 // (tmax * fb))))
    T = rng.integers(1, tmax + 1, size=n).astype(np.int32)
    T[rng.integers(0, n)] = tmax
    plan, op = G.full_parity(T, tb, 8, fb, out_fb=fb, pad=0x6B, extra_blocks=3)
    want_k = G.expected_copy_kernels(op.sum_t, len(T), fb, tb)
    assert B.bload_last_copy_kernel("pack") == want_k["pack_meta"] and want_k["pack"] != "k7_copy<pack>"
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    store_h = store.cpu().numpy()
    nb = op.n_blocks
    for b0, cnt in [(0, 1), (1, 1), (nb // 2, 3), (nb - 1, 2), (0, nb), (nb // 3, nb // 2 + 1), (nb, 1)]:
        res, _ = G.gpu_pack_all(plan, store, fb, b0, cnt, 0xD2, meta=False)
        assert B.bload_last_copy_kernel("pack") == want_k["pack"]
        d = G.first_diff(res["dense"].reshape(-1), O.pack(op, store_h, fb, b0, cnt, 0xD2).reshape(-1))
        assert d is None, "blocks [%d, +%d): %s" % (b0, cnt, d)


@pytest.mark.parametrize("tb,fb,tmax", [(4096, 4, 4096), (64, 4, 64), (1000, 16, 9), (700, 256, 60), (36, 12, 36), (94, 12, 94),
                                        (5, 4, 5)])
def test_one_launch_for_dense_blocks_and_metadata_of_small_frames(tb, fb, tmax):
    """A pack call that asks for dense blocks and metadata of small word-sized frames is ONE launch (some CTAs pack, the
    others write metadata).  Its outputs equal those of the two separate calls and the oracle's: sub-ranges, filler
    blocks behind the plan, a metadata array left out, metadata pointers that force the scalar stores."""
    rng = np.random.default_rng(tb * 7 + fb)
    n = int(min(3000, max(3, 3_000_000 // (tmax * fb))))
    T = rng.integers(1, tmax + 1, size=n).astype(np.int32)
    op = O.plan(T, tb, 17); plan = G.gpu_plan(T, tb, 17)
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    store_h = store.cpu().numpy()
    nb = op.n_blocks
    for b0, cnt in [(0, nb + 2), (0, 1), (max(nb // 2, 0), min(3, nb)), (nb - 1, 4), (nb + 1, 2)]:
        before = B.bload_kernel_launches()
        res, _ = G.gpu_pack_all(plan, store, fb, b0, cnt, 0x3C)
        assert B.bload_kernel_launches() - before == 1
        assert B.bload_last_copy_kernel("pack") == G.expected_copy_kernels(op.sum_t, len(T), fb, tb)["pack_meta"]
        assert np.array_equal(res["dense"], O.pack(op, store_h, fb, b0, cnt, 0x3C))
        for name, want in zip(("seq_id", "pos", "reset", "valid"), O.metadata(op, b0, cnt)):
            assert np.array_equal(res[name], want), name
    # only two of the four arrays, at addresses that are not vector aligned
    cnt = min(nb, 5)
    raw_pos = torch.full((cnt * tb + 3,), 77, dtype=torch.int32, device=G.DEV)
    raw_valid = torch.full((cnt * tb + 3,), 77, dtype=torch.uint8, device=G.DEV)
    dense = G.Guarded(cnt * tb * fb)
    B.bload_pack(plan, store, fb, 0, cnt, dense=dense.t, pos=raw_pos[1:1 + cnt * tb], valid=raw_valid[1:1 + cnt * tb])
    torch.cuda.synchronize(); dense.check()
    want = O.metadata(op, 0, cnt)
    assert np.array_equal(raw_pos[1:1 + cnt * tb].cpu().numpy().reshape(cnt, tb), want[1])
    assert np.array_equal(raw_valid[1:1 + cnt * tb].cpu().numpy().reshape(cnt, tb), want[3])
    assert int(raw_pos[0]) == 77 and int(raw_pos[-1]) == 77 and int(raw_valid[0]) == 77 and int(raw_valid[-1]) == 77
    assert np.array_equal(dense.t.cpu().numpy().reshape(cnt, tb, fb), O.pack(op, store_h, fb, 0, cnt, 0))


@pytest.mark.parametrize("tb,fb,kind", [(4096, 4, "tokens"), (2048, 8, "half"), (3072, 4, "half"), (1024, 16, "few_long"),
                                        (4096, 4, "all_long"), (8192, 4, "four_per_block"), (1000, 20, "around_512"),
                                        (333, 48, "half")])
def test_unpack_of_block_ranges_of_small_frames(tb, fb, kind):
    """Unpack of a block sub-range of small word-sized frames (the staged kernel over the dense side or, for short runs
    and for frames that are multiples of 16 bytes, the word-wise walk along it).  Plans that mix
    runs as long as a block and runs of a few frames in every proportion, runs around 512 bytes, runs cut by sub-tile
    ends, ranges that start and end anywhere, filler blocks; every byte against the oracle, canaries around the output."""
    rng = np.random.default_rng(tb * 3 + fb)
    blocks = (24 << 20) // (tb * fb)
    if kind == "tokens":
        T = W.lengths(W.scaled(W.WORKLOADS["tokens"], int(blocks * 4.7)))
    elif kind == "half":
        T = np.where(rng.random(blocks) < 0.5, tb, rng.integers(1, 40, size=blocks))
        T = np.concatenate([T, rng.integers(1, 40, size=blocks * 20)])
    elif kind == "few_long":
        T = np.concatenate([rng.integers(1, 24, size=blocks * 90), np.full(blocks // 50, tb)])
    elif kind == "all_long":
        T = np.full(blocks, tb)
    elif kind == "four_per_block":
        T = np.full(4 * blocks, tb // 4)
    else:                                                   # run lengths around 512 bytes
        T = rng.integers(max(1, 480 // fb), 560 // fb + 1, size=blocks * (tb * fb // 520))
    T = rng.permutation(np.minimum(np.asarray(T), tb)).astype(np.int32)
    op = O.plan(T, tb, 6); plan = G.gpu_plan(T, tb, 6)
    nb = op.n_blocks
    g = torch.Generator(device=G.DEV); g.manual_seed(tb)
    for b0, cnt in ((1, nb - 2), (0, 3), (nb // 3, nb // 2), (nb - 2, 5)):
        cnt = max(cnt, 1)
        dense_out = torch.randint(0, 256, (cnt * tb * fb,), dtype=torch.uint8, device=G.DEV, generator=g)
        rag = G.Guarded(op.sum_t * fb, 0x5A)
        B.bload_unpack(plan, dense_out, fb, b0, cnt, rag.t)
        torch.cuda.synchronize(); rag.check()
        assert B.bload_last_copy_kernel("unpack") == G.expected_copy_kernels(op.sum_t, len(T), fb, tb)["unpack_range"]
        want = np.full(op.sum_t * fb, 0x5A, np.uint8)
        O.unpack(op, dense_out.cpu().numpy(), fb, b0, cnt, want)
        d = G.first_diff(rag.t.cpu().numpy(), want)
        assert d is None, "blocks [%d, +%d): %s" % (b0, cnt, d)


@pytest.mark.parametrize("tb,fb,lengths", [(6, 4, [2, 2, 3, 3, 4, 5, 6, 6]), (7, 12, [1]), (9, 20, [9, 1, 1]),
                                           (5, 4, [1, 1, 1]), (3000, 4, None), (1234, 36, None)])
def test_whole_plan_unpack_of_word_sized_frames(tb, fb, lengths):
    """Unpacking every block of a plan with small word-sized frames takes the ragged-side tiled kernel:
    totals that are not multiples of 16 bytes, totals below one vector, block sizes that are not
    multiples of 16 bytes, many warps with one sub-tile each."""
    rng = np.random.default_rng(tb + fb)
    T = np.array(lengths, np.int32) if lengths else rng.integers(1, tb + 1, size=5000).astype(np.int32)
    G.full_parity(T, tb, 3, fb, out_fb=fb, pad=0x11, extra_blocks=0)
    G.full_parity(T, tb, 4, fb, out_fb=fb, pad=0, extra_blocks=3)


# ---- policy 1: uniform over the lengths that fit ----

@pytest.mark.parametrize("name,n", [("toy_video", None), ("features_fp16", None), ("tokens", 30000),
                                    ("heavy_tail_bf16", 20000), ("video_dataset_shape", None)])
def test_policy1_plans_match_the_oracle(name, n):
    w = W.WORKLOADS[name]
    if n:
        w = W.scaled(w, n)
    T = W.lengths(w)
    for seed in (w.seed, 7):
        G.assert_plan_equal(G.gpu_plan(T, w.t_block, seed, policy=1), O.plan(T, w.t_block, seed, policy=1))


def test_policy1_small_and_degenerate_cases():
    rng = np.random.default_rng(3)
    G.full_parity(W.TOY8_LENGTHS, W.TOY8_T_BLOCK, 2, 8, policy=1)
    for T, tb in [(np.array([5], np.int32), 9), (np.full(300, 17, np.int32), 17), (np.ones(5000, np.int32), 33),
                  (np.ones(70, np.int32), 1), (rng.integers(1, 4, size=9000).astype(np.int32), 4096),
                  (np.concatenate([rng.integers(1, 32769, size=40), [32768, 32768, 1, 1, 1024, 1025]]).astype(np.int32), 32768),
                  (rng.choice([3, 700], size=4097).astype(np.int32), 1000)]:
        for seed in (0, 11):
            G.assert_plan_equal(G.gpu_plan(T, tb, seed, policy=1), O.plan(T, tb, seed, policy=1))
    for n in (1, 31, 32, 33, 2049, 70001):
        T = rng.integers(1, 301, size=n).astype(np.int32)
        G.assert_plan_equal(G.gpu_plan(T, 300, 5, policy=1), O.plan(T, 300, 5, policy=1))


# ---- policy 2: best fit decreasing (deterministic comparison strategy) ----

@pytest.mark.parametrize("name,n", [("toy_video", None), ("features_fp16", None), ("raw_frames", None), ("tokens", 50000),
                                    ("heavy_tail_bf16", 20000), ("video_dataset_shape", None)])
def test_policy2_plans_match_the_oracle(name, n):
    w = W.WORKLOADS[name]
    if n:
        w = W.scaled(w, n)
    T = W.lengths(w)
    for seed in (w.seed, 7):
        G.assert_plan_equal(G.gpu_plan(T, w.t_block, seed, policy=2), O.plan(T, w.t_block, seed, policy=2))


def test_policy2_small_and_degenerate_cases():
    rng = np.random.default_rng(4)
    G.full_parity(W.TOY8_LENGTHS, W.TOY8_T_BLOCK, 2, 8, policy=2)
    G.full_parity(rng.integers(1, 60, size=700).astype(np.int32), 64, 3, 20, policy=2)
    for T, tb in [(np.array([5], np.int32), 9), (np.full(300, 17, np.int32), 17), (np.ones(5000, np.int32), 33),
                  (np.ones(70, np.int32), 1), (rng.integers(1, 4, size=9000).astype(np.int32), 4096),
                  (np.concatenate([rng.integers(1, 32769, size=40), [32768, 32768, 1, 1, 1024, 1025]]).astype(np.int32), 32768),
                  (rng.choice([3, 700], size=4097).astype(np.int32), 1000), (np.array([2, 1, 1], np.int32), 2)]:
        for seed in (0, 11):
            G.assert_plan_equal(G.gpu_plan(T, tb, seed, policy=2), O.plan(T, tb, seed, policy=2))
    for n in (1, 31, 32, 33, 2049, 70001):
        T = rng.integers(1, 301, size=n).astype(np.int32)
        G.assert_plan_equal(G.gpu_plan(T, 300, 5, policy=2), O.plan(T, 300, 5, policy=2))


def test_policy2_full_size_tokens():
    w = W.WORKLOADS["tokens"]
    T = W.lengths(w)
    G.assert_plan_equal(G.gpu_plan(T, w.t_block, w.seed, policy=2), O.plan(T, w.t_block, w.seed, policy=2))


def test_rank_ranges_pack_and_unpack_like_the_whole():
    """Three data-parallel ranks, emulated one after the other on one GPU (they share nothing and wait for nothing):
    each packs its equal share of blocks, filler blocks included; together the shares are the whole epoch."""
    w = W.scaled(W.WORKLOADS["features_fp16"], 500)
    T = W.lengths(w)
    fb, tb, world, batch = 48, w.t_block, 3, 4
    op = O.plan(T, tb, 21)
    plan = G.gpu_plan(T, tb, 21)
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    store_h = store.cpu().numpy()
    back = torch.full((op.sum_t * fb,), 0x5A, dtype=torch.uint8, device=G.DEV)
    covered = 0
    for rank in range(world):
        b0, cnt = B.bload_rank_range(op.n_blocks, world, rank, batch)
        res, dense = G.gpu_pack_all(plan, store, fb, b0, cnt, 0)
        assert np.array_equal(res["dense"], O.pack(op, store_h, fb, b0, cnt, 0))
        assert np.array_equal(res["valid"], O.metadata(op, b0, cnt)[3])
        B.bload_unpack(plan, dense.t, fb, b0, cnt, back)
        covered += cnt
    torch.cuda.synchronize()
    assert covered >= op.n_blocks and torch.equal(back, store)


def test_reader_behind_a_pack_of_large_frames_sees_dense_blocks_and_metadata():
    """Large frames: the pack kernel is launched beside the call's metadata kernel, not behind it.  Whatever the stream
    runs next must still find both outputs complete -- here copies enqueued on the same side stream straight after
    the call, with no synchronisation in between, call after call on the same output buffers (so a late metadata
    kernel of call i would also be caught overwriting the results of call i+1)."""
    rng = np.random.default_rng(99)
    tb, fb = 2000, 4096
    T = rng.integers(1, 40, size=6000).astype(np.int32)
    plan = G.gpu_plan(T, tb, 3)
    op = O.plan(T, tb, 3)
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    assert G.expected_copy_kernels(op.sum_t, T.size, fb, tb)["pack"] == "k7_copy<pack>"
    cnt = 3
    dense = torch.empty(cnt * tb * fb, dtype=torch.uint8, device=G.DEV)
    seq_id = torch.empty(cnt * tb, dtype=torch.int32, device=G.DEV)
    pos = torch.empty_like(seq_id)
    reset = torch.empty(cnt * tb, dtype=torch.uint8, device=G.DEV)
    valid = torch.empty_like(reset)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    got = []
    with torch.cuda.stream(s):
        for b0 in range(0, min(op.n_blocks, 4 * cnt), cnt):
            B.bload_pack(plan, store, fb, b0, cnt, dense=dense, seq_id=seq_id, pos=pos, reset=reset, valid=valid, pad_byte=0x5C)
            got.append((b0, dense.clone(), seq_id.clone(), pos.clone(), reset.clone(), valid.clone()))
    s.synchronize()
    assert B.bload_last_copy_kernel("pack") == "k7_copy<pack>"
    h_store = store.cpu().numpy()
    for b0, d, si, po, re, va in got:
        assert np.array_equal(d.cpu().numpy().reshape(cnt, tb, fb), O.pack(op, h_store, fb, b0, cnt, 0x5C)), b0
        for name, arr, want in zip(("seq_id", "pos", "reset", "valid"), (si, po, re, va), O.metadata(op, b0, cnt)):
            assert np.array_equal(arr.cpu().numpy().reshape(cnt, tb), want), (b0, name)


@pytest.mark.parametrize("tb,fb,kind", [(4096, 1, "token_like"), (4096, 2, "token_like"), (4096, 3, "token_like"),
                                        (333, 3, "uniform"), (2047, 2, "uniform"), (5000, 1, "ones_and_long"),
                                        (3100, 1, "ones_and_long"), (901, 3, "uniform")])
def test_frames_of_one_to_three_bytes_in_runs_up_to_4_kb_move_in_granules(tb, fb, kind):
    """Frames shorter than a word (masks, 16-bit ids) in runs beyond the word-wise walks: the pack and whole-plan unpack
    kernels that move 16-byte granules.  Lengths with the shape of the token workload (many runs of 8 frames between runs as long as a
    block), blocks whose size is not a multiple of 16 bytes (the last granule of the call is partial), and thousands of
    one-frame runs between long ones, which the fill rule collects at the ends of the blocks: dozens of runs inside one
    granule, more than a window of 32 holds.  Whole plan with filler blocks, sub-ranges, a non-zero pad byte."""
    rng = np.random.default_rng(tb * 7 + fb)
    if kind == "token_like":
        T = np.concatenate([np.full(900, 8), np.full(350 // fb, tb), rng.integers(9, tb // fb, size=900)]).astype(np.int32)
    elif kind == "uniform":
        T = rng.integers(1, tb + 1, size=2500).astype(np.int32)
    else:
        T = np.concatenate([np.ones(3000, np.int32), np.full(900, tb, np.int32), rng.integers(2, 40, size=300).astype(np.int32)])
    rng.shuffle(T)
    want_k = G.expected_copy_kernels(int(T.sum()), T.size, fb, tb)
    assert want_k["pack"] == "k24_pack_granules", (int(T.sum()) * fb // T.size)
    plan, op = G.full_parity(T, tb, 41, fb, out_fb=fb, pad=0xC3, extra_blocks=3)
    assert B.bload_last_copy_kernel("pack") == "k24_pack_granules" and B.bload_last_copy_kernel("unpack") == "k25_unpack_granules"
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
    store_h = store.cpu().numpy()
    nb = op.n_blocks
    for b0, cnt in [(0, 1), (1, 1), (nb // 3, 5), (nb - 2, 4), (nb, 1)]:
        res, _ = G.gpu_pack_all(plan, store, fb, b0, cnt, 0x3D, meta=True)
        d = G.first_diff(res["dense"].reshape(-1), O.pack(op, store_h, fb, b0, cnt, 0x3D).reshape(-1))
        assert d is None, "blocks [%d, +%d): %s" % (b0, cnt, d)
    assert B.bload_last_copy_kernel("pack") == "k24_pack_granules"
