"""Pins for the oracle's metadata, pack, unpack and statistics (no GPU)."""
import os

import numpy as np
import pytest

import invariants
from oracle import bload_oracle as O
from paper_2310_10879_b200 import workloads as W


def _golden(name):
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, *v = line.split()
                out[k] = [int(x) for x in v]
    return out


def test_naive_padding_reproduces_the_paper_table():
    g = _golden("paper_table1_padding.txt")
    n, s, tmax = g["n_videos"][0], g["n_frames"][0], g["t_max"][0]
    st = O.stats(n, s, tmax, tmax, -(-s // tmax))
    assert st["pad_naive_tmax"] == g["padding_zero_pad"][0] == 534831
    # "almost 4x the original data size" / "over 500k": 3.2x
    assert 3.0 < st["pad_naive_tmax"] / s < 4.0
    # the lower bound on blocks gives the least padding any packing into blocks of 94 could have
    assert st["min_blocks"] == 1775 and st["pad_packed"] == 1775 * 94 - s
    # reduction reported in the paper: more than 100x with 3,695 padding frames
    assert g["padding_zero_pad"][0] / g["padding_block_pad"][0] > 100


def test_stats_closed_forms():
    rng = np.random.default_rng(3)
    for _ in range(50):
        n = int(rng.integers(1, 500)); tb = int(rng.integers(1, 300))
        T = rng.integers(1, tb + 1, size=n).astype(np.int32)
        p = O.plan(T, tb, int(rng.integers(0, 1 << 30)))
        s = O.stats(p.n, p.sum_t, p.t_max, tb, p.n_blocks)
        assert s["pad_packed"] == int((tb - p.block_fill.astype(np.int64)).sum())
        assert s["pad_naive_tmax"] == int((int(T.max()) - T.astype(np.int64)).sum())
        assert s["pad_naive_tblock"] == int((tb - T.astype(np.int64)).sum())
        assert s["min_blocks"] == -(-int(T.sum()) // tb)
        assert abs(s["frac_packed"] - s["pad_packed"] / (p.n_blocks * tb)) < 1e-15
        assert abs(s["frac_naive_tmax"] - s["pad_naive_tmax"] / (n * int(T.max()))) < 1e-15
        if s["pad_packed"]:
            assert abs(s["reduction_vs_tmax"] - s["pad_naive_tmax"] / s["pad_packed"]) < 1e-9


def test_padding_reduction_on_dataset_shaped_input_is_of_the_papers_order():
    w = W.WORKLOADS["video_dataset_shape"]
    T = W.lengths(w)
    p = O.plan(T, w.t_block, w.seed)
    s = O.stats(p.n, p.sum_t, p.t_max, w.t_block, p.n_blocks)
    assert s["reduction_vs_tmax"] > 50          # paper: 144.7x on the real lengths
    assert s["frac_packed"] < 0.05


def _plan(name, n=None, seed=None):
    w = W.WORKLOADS[name]
    if n:
        w = W.scaled(w, n)
    T = W.lengths(w)
    return w, O.plan(T, w.t_block, w.seed if seed is None else seed)


@pytest.mark.parametrize("name,n", [("toy_video", None), ("features_fp16", None), ("heavy_tail_bf16", 900),
                                    ("tokens", 3000)])
def test_metadata_matches_slotwise_construction(name, n):
    w, p = _plan(name, n)
    extra = 3                                   # filler blocks past the end are all padding
    got = O.metadata(p, 0, p.n_blocks + extra)
    want = invariants.slot_maps(p.lengths, p.t_block, p.n_blocks, p.seg_seq, p.seg_start, p.block_seg_begin,
                                0, p.n_blocks + extra)
    for a, b in zip(got, want):
        assert np.array_equal(a, b)
    seq_id, pos, reset, valid = got
    # I1 at frame level: every (sequence, frame) exactly once
    flat = p.offsets[seq_id[valid == 1].astype(np.int64)] + pos[valid == 1]
    assert np.array_equal(np.sort(flat), np.arange(p.sum_t))
    # I4: a reset flag exactly at every sequence start
    assert int(reset.sum()) == p.n and np.all(pos[reset == 1] == 0) and np.all(reset[pos == 0] == 1)
    assert np.all(reset[:p.n_blocks, 0] == 1)
    # I6: pad slots
    assert np.all(seq_id[valid == 0] == -1) and np.all(pos[valid == 0] == -1) and np.all(reset[valid == 0] == 0)
    assert np.all(valid[p.n_blocks:] == 0)
    # a sub-range equals the slice of the full result
    sub = O.metadata(p, 2, 3)
    for a, b in zip(sub, got):
        assert np.array_equal(a, b[2:5])


@pytest.mark.parametrize("name,n,fb", [("toy_video", None, 12288), ("toy_video", None, 1), ("features_fp16", 300, 2048),
                                       ("tokens", 3000, 4), ("heavy_tail_bf16", 500, 24), ("raw_frames", 40, 7)])
@pytest.mark.parametrize("pad", [0, 0xA5])
def test_pack_is_a_gather_and_unpack_its_inverse(name, n, fb, pad):
    w, p = _plan(name, n)
    store = W.payload_bytes_numpy(p.sum_t * fb, seed=17)
    nb = p.n_blocks + 2
    dense = O.pack(p, store, fb, 0, nb, pad)
    seq_id, pos, reset, valid = invariants.slot_maps(p.lengths, p.t_block, p.n_blocks, p.seg_seq, p.seg_start,
                                                     p.block_seg_begin, 0, nb)
    frames = store.reshape(p.sum_t, fb)
    src = np.where(valid == 1, p.offsets[np.maximum(seq_id, 0).astype(np.int64)] + pos, 0)
    want = np.where((valid == 1)[..., None], frames[src], np.uint8(pad))
    assert np.array_equal(dense, want)
    # frame order inside every sequence survives (I2): check one sequence directly
    s = int(p.seg_seq[p.n // 2]); b, st = int(p.seq_block[s]), int(p.seq_start[s])
    assert np.array_equal(dense[b, st:st + p.lengths[s]], frames[p.offsets[s]:p.offsets[s + 1]])
    # round trip
    out = np.full(p.sum_t * fb, 0x3C, np.uint8)
    O.unpack(p, dense, fb, 0, nb, out)
    assert np.array_equal(out, store)
    # a block range touches only its own sequences
    out = np.full(p.sum_t * fb, 0x3C, np.uint8)
    lo, cnt = 1, min(2, p.n_blocks - 1)
    O.unpack(p, dense[lo:lo + cnt], fb, lo, cnt, out)
    touched = np.zeros(p.sum_t, bool)
    for k in range(p.block_seg_begin[lo], p.block_seg_begin[lo + cnt]):
        s = p.seg_seq[k]; touched[p.offsets[s]:p.offsets[s + 1]] = True
    o2 = out.reshape(p.sum_t, fb)
    assert np.array_equal(o2[touched], frames[touched]) and np.all(o2[~touched] == 0x3C)
    # packing a sub-range equals the slice
    assert np.array_equal(O.pack(p, store, fb, lo, cnt, pad), dense[lo:lo + cnt])


def test_pack_repeat_last_against_a_numpy_gather():
    rng = np.random.default_rng(12)
    for n, tb, fb in ((8, 6, 3), (60, 25, 16), (200, 64, 5)):
        T = rng.integers(1, tb + 1, size=n).astype(np.int32)
        p = O.plan(T, tb, 1000 + n)
        store = rng.integers(0, 256, size=(p.sum_t, fb), dtype=np.uint8)
        nb = p.n_blocks + 1
        seq_id, pos, _, valid = O.metadata(p, 0, nb)
        src = np.where(valid == 1, p.offsets[np.maximum(seq_id, 0)] + pos, -1)
        want = np.full((nb, tb, fb), 0x42, np.uint8)
        for q in range(nb):
            fill = int(valid[q].sum())
            if fill:
                idx = src[q].copy()
                idx[fill:] = idx[fill - 1]
                want[q] = store[idx]
        got = O.pack_repeat_last(p, store, fb, 0, nb, 0x42)
        assert np.array_equal(got, want)
        assert np.array_equal(O.pack_repeat_last(p, store, fb, 1, 2, 0x42), want[1:3])


def test_pack_repeat_last_with_one_sequence_per_block_is_the_naive_padding_of_the_paper():
    # lengths above half a block cannot share a block: every sample is padded on its own by repeating its last frame
    rng = np.random.default_rng(13)
    tb = 20
    T = rng.integers(11, tb + 1, size=30).astype(np.int32)
    p = O.plan(T, tb, 5)
    assert p.n_blocks == T.size
    store = rng.integers(0, 256, size=(p.sum_t, 7), dtype=np.uint8)
    got = O.pack_repeat_last(p, store, 7, 0, p.n_blocks)
    for b in range(p.n_blocks):
        i = int(p.seg_seq[p.block_seg_begin[b]])
        x = store[p.offsets[i]:p.offsets[i + 1]]
        assert np.array_equal(got[b], np.concatenate([x, np.repeat(x[-1:], tb - len(x), axis=0)]))
