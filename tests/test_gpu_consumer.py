"""GPU parity of the consumer-side calls (bload_carry_prev, bload_reset_state, bload_valid_sum) and of repeat-last padding,
through the C ABI, against the CPU oracle: bytes bit for bit, sums within a stated bound."""
import numpy as np
import pytest
import torch

import gpu_util as G
import paper_2310_10879_b200 as B
from oracle import bload_oracle as O
from paper_2310_10879_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _both_plans(T, tb, seed, policy=0):
    op = O.plan(T, tb, seed, policy)
    plan = G.gpu_plan(T, tb, seed, policy=policy)
    assert plan.info.checksum == op.checksum
    return plan, op


def _carry_prev_parity(plan, op, fb, b0, cnt, fill, seed=3):
    tb = op.t_block
    g = torch.Generator(device=G.DEV); g.manual_seed(seed)
    dense = torch.randint(0, 256, (cnt * tb * fb,), dtype=torch.uint8, device=G.DEV, generator=g)
    prev = G.Guarded(cnt * tb * fb, 0x3C)
    B.bload_carry_prev(plan, dense, fb, b0, cnt, prev.t, fill_byte=fill)
    torch.cuda.synchronize()
    prev.check()
    want = O.carry_prev(op, dense.cpu().numpy(), fb, b0, cnt, fill)
    d = G.first_diff(prev.t.cpu().numpy(), want)
    assert d is None, "carry_prev fb=%d blocks [%d,+%d): %s" % (fb, b0, cnt, d)


@pytest.mark.parametrize("fb", [1, 3, 4, 12, 16, 20, 64, 100, 4096, 4100, 20000])
def test_carry_prev_frame_sizes(fb):
    rng = np.random.default_rng(fb)
    tb = int(rng.integers(5, 120))
    T = rng.integers(1, tb + 1, size=int(rng.integers(1, 200))).astype(np.int32)
    plan, op = _both_plans(T, tb, int(rng.integers(0, 1 << 40)))
    _carry_prev_parity(plan, op, fb, 0, op.n_blocks + 2, 0x00)
    if op.n_blocks > 3:
        _carry_prev_parity(plan, op, fb, 2, op.n_blocks - 3, 0xA7)


def test_carry_prev_workloads():
    for name, n, fb in (("toy_video", 0, None), ("features_fp16", 0, None), ("tokens", 20000, None),
                        ("heavy_tail_bf16", 1000, None), ("raw_frames", 30, None)):
        w = W.WORKLOADS[name]
        if n:
            w = W.scaled(w, n)
        plan, op = _both_plans(W.lengths(w), w.t_block, w.seed)
        _carry_prev_parity(plan, op, fb or w.frame_bytes, 0, op.n_blocks + 1, 0)


def test_carry_prev_other_policies_and_single_frame_sequences():
    T = np.ones(500, np.int32)  # every frame is a first frame: nothing is ever carried over
    plan, op = _both_plans(T, 37, 5)
    _carry_prev_parity(plan, op, 8, 0, op.n_blocks, 0x55)
    rng = np.random.default_rng(9)
    T = rng.integers(1, 50, size=400).astype(np.int32)
    for policy in (1, 2):
        plan, op = _both_plans(T, 64, 11, policy)
        _carry_prev_parity(plan, op, 24, 0, op.n_blocks + 1, 0)


def test_carry_prev_of_a_packed_batch_is_the_previous_frame_of_the_same_sequence():
    # a property that holds at any size, checked without the oracle: pack frame numbers, shift, compare with pos - 1
    w = W.scaled(W.WORKLOADS["heavy_tail_bf16"], 3000)
    T = W.lengths(w)
    plan = G.gpu_plan(T, w.t_block, w.seed)
    nb, tb = plan.n_blocks, plan.t_block
    off = plan.tables()["offsets"]
    frame_no = torch.arange(plan.sum_t, device=G.DEV, dtype=torch.int64)
    frame_no -= torch.repeat_interleave(off[:-1], torch.from_numpy(T).to(G.DEV).long())
    store = frame_no.to(torch.int32)
    dense = torch.empty(nb * tb, dtype=torch.int32, device=G.DEV)
    pos = torch.empty(nb * tb, dtype=torch.int32, device=G.DEV)
    B.bload_pack(plan, store, 4, 0, nb, dense=dense, pos=pos, pad_byte=0xFF)
    prev = torch.empty_like(dense)
    B.bload_carry_prev(plan, dense, 4, 0, nb, prev, fill_byte=0xFF)
    torch.cuda.synchronize()
    assert torch.equal(dense, pos)
    assert torch.equal(prev, torch.where(pos > 0, pos - 1, torch.full_like(pos, -1)))


@pytest.mark.parametrize("sb", [1, 7, 16, 100, 4096, 40000])
def test_reset_state_against_the_oracle(sb):
    rng = np.random.default_rng(sb)
    tb = 40
    T = rng.integers(1, tb + 1, size=300).astype(np.int32)
    plan, op = _both_plans(T, tb, 77)
    b0, cnt = 1, op.n_blocks + 1  # reaches one filler block
    init_h = rng.integers(0, 256, size=sb, dtype=np.uint8)
    init_d = torch.from_numpy(init_h).to(G.DEV)
    for slot in (0, 1, 5, tb - 1):
        for init in (None, init_h):
            state_h = rng.integers(0, 256, size=(cnt, sb), dtype=np.uint8)
            st = G.Guarded(cnt * sb)
            st.t.copy_(torch.from_numpy(state_h.reshape(-1)).to(G.DEV))
            B.bload_reset_state(plan, b0, cnt, slot, st.t, sb, init=None if init is None else init_d)
            torch.cuda.synchronize()
            st.check()
            want = O.reset_state(op, b0, cnt, slot, state_h.copy(), init)
            assert np.array_equal(st.t.cpu().numpy().reshape(cnt, sb), want), (sb, slot, init is None)


def test_reset_state_drives_a_recurrence_to_per_sequence_cumsums():
    # the whole loop on the GPU: h <- reset(h); h += x[:, s]; y[:, s] = h, then unpack and compare with numpy
    rng = np.random.default_rng(4)
    tb, d = 48, 6
    T = rng.integers(1, tb + 1, size=200).astype(np.int32)
    plan, op = _both_plans(T, tb, 123)
    nb = op.n_blocks
    x = torch.from_numpy(rng.integers(0, 100, size=(op.sum_t, d)).astype(np.int32)).to(G.DEV)
    dense = torch.empty(nb, tb, d, dtype=torch.int32, device=G.DEV)
    B.bload_pack(plan, x, 4 * d, 0, nb, dense=dense)
    h = torch.full((nb, d), 99, dtype=torch.int32, device=G.DEV)
    y = torch.empty_like(dense)
    for s in range(tb):
        B.bload_reset_state(plan, 0, nb, s, h, 4 * d)
        h += dense[:, s, :]
        y[:, s, :] = h
    out = torch.empty(op.sum_t, d, dtype=torch.int32, device=G.DEV)
    B.bload_unpack(plan, y, 4 * d, 0, nb, out)
    torch.cuda.synchronize()
    xh, got = x.cpu().numpy(), out.cpu().numpy()
    for i in range(op.n):
        a, b = int(op.offsets[i]), int(op.offsets[i + 1])
        assert np.array_equal(got[a:b], np.cumsum(xh[a:b], axis=0)), i


@pytest.mark.parametrize("tb,n", [(6, 8), (37, 300), (64, 500), (1000, 1000), (4096, 3000)])
def test_valid_sum_against_the_oracle(tb, n):
    rng = np.random.default_rng(tb + n)
    T = rng.integers(1, tb + 1, size=n).astype(np.int32)
    plan, op = _both_plans(T, tb, 31)
    for b0, cnt in ((0, op.n_blocks + 2), (1, max(op.n_blocks - 1, 1))):
        vals_h = rng.standard_normal(cnt * tb).astype(np.float32) * 1000.0
        vals_h[rng.integers(0, vals_h.size, size=10)] = 1e30  # some land on padding and must not be seen ...
        _, _, _, valid = O.metadata(op, b0, cnt)
        vals_h[(valid.reshape(-1) == 1) & (np.abs(vals_h) > 1e29)] = 3.0  # ... none on a frame
        vals = torch.from_numpy(vals_h).to(G.DEV)
        bs = torch.full((cnt,), -1.0, dtype=torch.float64, device=G.DEV)
        tot = torch.full((2,), -1.0, dtype=torch.float64, device=G.DEV)
        B.bload_valid_sum(plan, vals, b0, cnt, bs, tot)
        bs2 = torch.empty_like(bs); tot2 = torch.empty_like(tot)
        B.bload_valid_sum(plan, vals, b0, cnt, bs2, tot2)
        torch.cuda.synchronize()
        assert torch.equal(bs, bs2) and torch.equal(tot, tot2)  # fixed summation order: identical bits
        want_sum, want_cnt = O.valid_sum(op, b0, cnt, vals_h)
        assert int(tot[1].item()) == want_cnt
        # double-precision sums in two different orders, each within n * 2^-53 * (sum of magnitudes) of the exact sum
        mag = float(np.abs(vals_h.astype(np.float64))[valid.reshape(-1) == 1].sum())
        bound = 2 * max(want_cnt, 1) * 2.0 ** -53 * mag
        assert abs(tot[0].item() - want_sum) <= bound, (tot[0].item(), want_sum, bound)
        per_block = bs.cpu().numpy()
        for q in range(cnt):
            w, c = O.valid_sum(op, b0 + q, 1, vals_h[q * tb:(q + 1) * tb])
            m = float(np.abs(vals_h[q * tb:(q + 1) * tb].astype(np.float64))[valid[q] == 1].sum())
            assert abs(per_block[q] - w) <= 2 * max(c, 1) * 2.0 ** -53 * m, q


def test_valid_sum_is_exact_on_integers_and_skips_total_when_null():
    rng = np.random.default_rng(8)
    T = rng.integers(1, 30, size=1000).astype(np.int32)
    plan, op = _both_plans(T, 30, 2)
    nb = op.n_blocks
    v = torch.from_numpy(rng.integers(-1000, 1000, size=op.sum_t).astype(np.float32)).to(G.DEV)
    dense = torch.empty(nb * 30, dtype=torch.float32, device=G.DEV)
    B.bload_pack(plan, v, 4, 0, nb, dense=dense, pad_byte=0x7F)
    bs = torch.empty(nb, dtype=torch.float64, device=G.DEV)
    B.bload_valid_sum(plan, dense, 0, nb, bs, None)
    torch.cuda.synchronize()
    assert float(bs.sum().item()) == float(v.double().sum().item())


def test_consumer_calls_reject_bad_arguments():
    T = np.array([3, 4, 5], np.int32)
    plan, _ = _both_plans(T, 8, 1)
    buf = torch.zeros(1 << 12, dtype=torch.uint8, device=G.DEV)
    E = B.BloadError
    with pytest.raises(E) as e:
        B.bload_carry_prev(plan, buf, 4, 0, 1, buf)
    assert e.value.code == -2  # same buffer
    with pytest.raises(E) as e:
        B.bload_carry_prev(plan, buf[1:], 4, 0, 1, buf[2048:])
    assert e.value.code == -5
    with pytest.raises(E) as e:
        B.bload_carry_prev(plan, None, 4, 0, 1, buf)
    assert e.value.code == -1
    for slot in (-1, 8):
        with pytest.raises(E) as e:
            B.bload_reset_state(plan, 0, 1, slot, buf, 16)
        assert e.value.code == -2
    with pytest.raises(E) as e:
        B.bload_reset_state(plan, 0, 1, 0, buf, 16, init=buf[8:])
    assert e.value.code == -5
    with pytest.raises(E) as e:
        B.bload_reset_state(plan, 0, 1, 0, buf, 0)
    assert e.value.code == -2
    f = torch.zeros(64, dtype=torch.float32, device=G.DEV)
    d = torch.zeros(8, dtype=torch.float64, device=G.DEV)
    with pytest.raises(E) as e:
        B.bload_valid_sum(plan, None, 0, 1, d)
    assert e.value.code == -1
    with pytest.raises(E) as e:
        B.bload_valid_sum(plan, f, -1, 1, d)
    assert e.value.code == -2
    # an empty range: total is (0, 0), nothing else is written
    tot = torch.full((2,), 5.0, dtype=torch.float64, device=G.DEV)
    B.bload_valid_sum(plan, f, 0, 0, d, tot)
    torch.cuda.synchronize()
    assert tot.tolist() == [0.0, 0.0]


@pytest.mark.parametrize("fb", [1, 4, 6, 16, 100, 4096, 40000])
def test_pack_repeat_last_against_the_oracle(fb):
    rng = np.random.default_rng(fb + 1)
    tb = int(rng.integers(5, 90))
    T = rng.integers(1, tb + 1, size=int(rng.integers(2, 150))).astype(np.int32)
    plan, op = _both_plans(T, tb, int(rng.integers(0, 1 << 40)))
    g = torch.Generator(device=G.DEV); g.manual_seed(fb)
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV, generator=g)
    store_h = store.cpu().numpy()
    for b0, cnt in ((0, op.n_blocks + 2), (1, max(op.n_blocks - 1, 1))):
        dense = G.Guarded(cnt * tb * fb)
        valid = torch.empty(cnt * tb, dtype=torch.uint8, device=G.DEV)
        B.bload_pack(plan, store, fb, b0, cnt, dense=dense.t, valid=valid, pad_byte=0x33, repeat_last=True)
        torch.cuda.synchronize()
        dense.check()
        d = G.first_diff(dense.t.cpu().numpy(), O.pack_repeat_last(op, store_h, fb, b0, cnt, 0x33))
        assert d is None, "repeat-last fb=%d: %s" % (fb, d)
        assert np.array_equal(valid.cpu().numpy().reshape(cnt, tb), O.metadata(op, b0, cnt)[3])


def test_pack_repeat_last_workloads():
    for name, n in (("toy_video", 0), ("features_fp16", 0), ("tokens", 20000), ("heavy_tail_bf16", 1000)):
        w = W.WORKLOADS[name]
        if n:
            w = W.scaled(w, n)
        plan, op = _both_plans(W.lengths(w), w.t_block, w.seed)
        store = W.payload_torch(w, op.sum_t, G.DEV).view(torch.uint8).reshape(-1)
        cnt = op.n_blocks + 1
        dense = G.Guarded(cnt * w.t_block * w.frame_bytes)
        B.bload_pack(plan, store, w.frame_bytes, 0, cnt, dense=dense.t, repeat_last=True)
        torch.cuda.synchronize()
        dense.check()
        d = G.first_diff(dense.t.cpu().numpy(), O.pack_repeat_last(op, store.cpu().numpy(), w.frame_bytes, 0, cnt, 0))
        assert d is None, name + ": " + d


@pytest.mark.parametrize("fb,tb", [(4, 16), (4, 4096), (8, 64), (12, 1000), (16, 64), (32, 500), (100, 64), (256, 48),
                                   (4, 8192)])
def test_carry_prev_small_word_sized_frames_take_the_staged_kernel(fb, tb):
    # (the name is historical: these cases used to go through the staged pack kernel; short runs now take the shifted
    # copy, k11_carry_shift)  frame sizes that are multiples of 4 in short runs with 16-byte block rows: several
    # sub-tiles per block or several blocks per sub-tile, segments that start inside a sub-tile, first frames that
    # straddle two sub-tiles
    rng = np.random.default_rng(fb * 1000 + tb)
    n = int(rng.integers(50, 600))
    T = np.minimum(rng.geometric(1.0 / max(2, tb // 6), size=n), tb).astype(np.int32)
    plan, op = _both_plans(T, tb, int(rng.integers(0, 1 << 40)))
    _carry_prev_parity(plan, op, fb, 0, op.n_blocks + 2, 0x00)
    _carry_prev_parity(plan, op, fb, 0, op.n_blocks, 0xC3, seed=9)
    if op.n_blocks > 4:
        _carry_prev_parity(plan, op, fb, 3, op.n_blocks - 4, 0x5E)
        _carry_prev_parity(plan, op, fb, op.n_blocks - 1, 5, 0x01)


def _expected_carry_kernel(sum_t, n, fb, tb):
    """The rule stated beside launch_carry_prev: the word-wise walk for blocks of at most 1 KB (4 KB when the frames are
    multiples of 4 bytes) and, when the frames are multiples of 8 bytes, for runs of at most 8 KB (or blocks of at most 32 KB) on average; else the shifted copy per
    sub-tile up to 16 KB runs; else the segment-by-segment kernel."""
    run, block = sum_t * fb // n, tb * fb
    if block <= 1024 or (block <= 4096 and fb % 4 == 0) or (fb % 8 == 0 and (run <= 8192 or block <= 32768) and run <= 16384):
        return "k23_carry_walk"
    return "k11_carry_shift" if run <= 16384 else "k11_carry_prev"


@pytest.mark.parametrize("fb,tb,tmax", [(8, 94, 94), (16, 94, 94), (64, 94, 94), (6, 94, 94), (1, 7, 7), (12, 94, 94), (256, 94, 60),
                                        (32, 10000, 300), (8, 4096, 2000), (4, 1, 1), (2, 500, 300)])
def test_carry_prev_by_the_word_wise_walk(fb, tb, tmax):
    """Small blocks (the paper's own block of 94 frames with per-frame records of a few bytes) and short runs of frames
    that are multiples of 8 bytes take the word-wise walk: words of 16, 8, 4, 2 and 1 bytes, blocks of 4 bytes to 320 KB,
    runs that begin before the warp's piece, pieces that begin in padding and in filler blocks, sub-ranges; the
    previous frame of every frame, the fill byte on first frames and padding."""
    rng = np.random.default_rng(fb * 19 + tb)
    n = int(min(6000, max(4, 3_000_000 // (tmax * fb))))
    T = rng.integers(1, tmax + 1, size=n).astype(np.int32)
    T[rng.integers(0, n)] = tmax
    plan, op = _both_plans(T, tb, 13)
    assert _expected_carry_kernel(op.sum_t, n, fb, tb) == "k23_carry_walk"
    _carry_prev_parity(plan, op, fb, 0, op.n_blocks + 3, 0x00)
    assert B.bload_last_copy_kernel("carry_prev") == "k23_carry_walk"
    _carry_prev_parity(plan, op, fb, 0, op.n_blocks, 0xB4, seed=3)
    if op.n_blocks > 3:
        _carry_prev_parity(plan, op, fb, 1, op.n_blocks - 2, 0x5E)
        _carry_prev_parity(plan, op, fb, op.n_blocks // 2, 2, 0x01)
    _carry_prev_parity(plan, op, fb, op.n_blocks - 1, 4, 0x77)
    _carry_prev_parity(plan, op, fb, op.n_blocks + 1, 2, 0x12)


@pytest.mark.parametrize("fb,tb,tmax", [(1, 40, 9), (3, 50, 50), (7, 3000, 40), (10, 64, 8), (130, 64, 20), (1000, 12, 5),
                                        (4096, 30, 3), (20, 20000, 600), (6, 16384, 300)])
def test_carry_prev_short_runs_take_the_shifted_copy(fb, tb, tmax):
    """Short runs (16 KB or less on average), any frame size: one shifted copy per sub-tile and fill patches at the first
    frame of every segment -- one lane per segment for frames up to 64 bytes, the whole warp per segment above; frame
    sizes that are not multiples of 4 or 16, first frames that straddle sub-tiles, more than 32 segments per sub-tile,
    blocks that end inside a sub-tile, filler blocks, sub-ranges."""
    rng = np.random.default_rng(fb * 77 + tb)
    n = int(min(3000, max(4, 4_000_000 // (tmax * fb))))
    T = rng.integers(1, tmax + 1, size=n).astype(np.int32)
    plan, op = _both_plans(T, tb, 31)
    _carry_prev_parity(plan, op, fb, 0, op.n_blocks + 2, 0x00)
    assert B.bload_last_copy_kernel("carry_prev") == _expected_carry_kernel(op.sum_t, n, fb, tb)
    _carry_prev_parity(plan, op, fb, 0, op.n_blocks, 0xC3, seed=9)
    if op.n_blocks > 3:
        _carry_prev_parity(plan, op, fb, 1, op.n_blocks - 2, 0x5E)
