"""Pins of the oracle's chunking strategy (the comparison system of the paper's section "Problem Statement and Current
Limitations": each sample is broken into chunks of a fixed number of frames and each chunk is treated as a sample).
Closed forms, the numpy construction of the chunk list, the reduction to naive padding, and the chunk-wise pack /
unpack / metadata against the ordinary oracle functions run on the derived one-chunk-per-block plan."""
import os

import numpy as np
import pytest

from oracle import bload_oracle as O
from paper_2310_10879_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _numpy_chunks(T, c, tail):
    """The chunk list by array arithmetic: counts per sequence, then repeat / arange."""
    T = T.astype(np.int64)
    cnt = (T + c - 1) // c if tail == O.KEEP_TAIL else T // c
    seq = np.repeat(np.arange(T.size), cnt)
    base = np.cumsum(cnt) - cnt
    idx = np.arange(int(cnt.sum())) - np.repeat(base, cnt)
    first = idx * c
    ln = np.minimum(c, T[seq] - first)
    return seq, first, ln


@pytest.mark.parametrize("tail", [O.KEEP_TAIL, O.DROP_TAIL])
@pytest.mark.parametrize("name,c", [("toy_video", 7), ("features_fp16", 30), ("features_fp16", 1), ("raw_frames", 60),
                                    ("heavy_tail_bf16", 128), ("video_dataset_shape", 22), ("tokens", 512)])
def test_chunk_list_and_closed_forms(name, c, tail):
    w = W.WORKLOADS[name]
    T = W.lengths(w) if name != "tokens" else W.lengths(W.scaled(w, 50_000))
    ch = O.chunks(T, c, tail)
    assert ch.status == 0
    seq, first, ln = _numpy_chunks(T, c, tail)
    assert np.array_equal(ch.chunk_seq, seq) and np.array_equal(ch.chunk_first, first) and np.array_equal(ch.chunk_len, ln)
    T64 = T.astype(np.int64)
    if tail == O.KEEP_TAIL:
        assert ch.n_chunks == int(((T64 + c - 1) // c).sum())
        assert ch.pad_frames == int(((-T64) % c).sum()) and ch.frames_deleted == 0 and ch.frames_kept == int(T64.sum())
    else:
        assert ch.n_chunks == int((T64 // c).sum())
        assert ch.pad_frames == 0 and ch.frames_deleted == int((T64 % c).sum())
        assert ch.frames_kept == ch.n_chunks * c and bool((ch.chunk_len == c).all())
    assert ch.frames_kept + ch.frames_deleted == ch.sum_t == int(T64.sum()) and ch.t_max == int(T.max())
    assert ch.n_chunks * c == ch.frames_kept + ch.pad_frames
    # every kept frame lies in exactly one chunk; the chunks of a sequence follow one another from its first frame
    hit = np.zeros(ch.sum_t, np.int32)
    start = ch.offsets[ch.chunk_seq.astype(np.int64)] + ch.chunk_first
    np.add.at(hit, np.concatenate([np.arange(a, a + l) for a, l in zip(start[:20000], ch.chunk_len[:20000])]) if ch.n_chunks else [], 1)
    assert hit.max(initial=0) <= 1
    if ch.n_chunks <= 20000:
        assert int(hit.sum()) == ch.frames_kept
        kept_per_seq = np.bincount(ch.chunk_seq, weights=ch.chunk_len, minlength=T.size).astype(np.int64)
        want = T64 if tail == O.KEEP_TAIL else (T64 // c) * c
        assert np.array_equal(kept_per_seq, want)


def test_a_chunk_that_covers_every_sequence_is_the_naive_padding_of_the_paper():
    # Table I, column "0 padding": 7,464 videos, 166,785 frames, longest 94 -> 534,831 padding frames.  Any lengths with
    # those three figures give it; chunks of 94 frames then are the samples themselves, each padded to 94.
    with open(os.path.join(GOLDEN, "paper_table1_padding.txt")) as f:
        gold = dict(line.split() for line in f if line.strip() and not line.startswith("#"))
    n, sum_t, t_min, t_max, pad = (int(gold[k]) for k in ("n_videos", "n_frames", "t_min", "t_max", "padding_zero_pad"))
    T = np.full(n, sum_t // n, np.int32)                    # 22 or 23 frames each ...
    T[: sum_t - int(T.sum())] += 1
    move = t_max - int(T[0])                                # ... except one of the longest and some of the shortest length
    T[0] += move
    for i in range(1, n):
        take = min(move, int(T[i]) - t_min)
        T[i] -= take; move -= take
        if move == 0:
            break
    assert int(T.sum()) == sum_t and int(T.max()) == t_max and int(T.min()) == t_min
    for tail in (O.KEEP_TAIL,):
        ch = O.chunks(T, t_max, tail)
        assert ch.n_chunks == n and ch.pad_frames == pad == n * t_max - sum_t and ch.frames_deleted == 0
        assert np.array_equal(ch.chunk_seq, np.arange(n)) and not ch.chunk_first.any() and np.array_equal(ch.chunk_len, T)
    # with only full chunks kept nothing is padded and everything shorter than the chunk is deleted
    ch = O.chunks(T, t_max, O.DROP_TAIL)
    assert ch.n_chunks == int((T == t_max).sum()) and ch.pad_frames == 0 and ch.frames_deleted == sum_t - ch.n_chunks * t_max


@pytest.mark.parametrize("tail", [O.KEEP_TAIL, O.DROP_TAIL])
@pytest.mark.parametrize("c,fb", [(5, 3), (16, 8), (1, 4), (64, 20)])
def test_chunk_pack_unpack_metadata(c, fb, tail):
    rng = np.random.default_rng(c * 10 + fb + tail)
    T = rng.integers(1, 4 * c + 2, size=60).astype(np.int32)
    ch = O.chunks(T, c, tail)
    store = rng.integers(0, 256, size=ch.sum_t * fb, dtype=np.uint8)
    nb = ch.n_chunks + 2                                     # two filler blocks behind the last chunk
    dense = O.chunk_pack(ch, store, fb, 0, nb, 0xAB)
    # numpy: frame numbers of every slot, -1 on padding
    frame = np.full((nb, c), -1, np.int64)
    start = ch.offsets[ch.chunk_seq.astype(np.int64)] + ch.chunk_first
    for j in range(ch.n_chunks):
        frame[j, :ch.chunk_len[j]] = start[j] + np.arange(ch.chunk_len[j])
    want = np.where((frame >= 0)[:, :, None], store.reshape(-1, fb)[np.maximum(frame, 0)], 0xAB).astype(np.uint8)
    assert np.array_equal(dense, want)
    sid, pos, reset, valid = O.chunk_metadata(ch, 0, nb)
    assert np.array_equal(valid, (frame >= 0).astype(np.uint8))
    assert np.array_equal(sid, np.where(frame >= 0, np.arange(nb)[:, None], -1))
    assert np.array_equal(pos, np.where(frame >= 0, np.arange(c)[None, :], -1))
    assert np.array_equal(reset, ((frame >= 0) & (np.arange(c)[None, :] == 0)).astype(np.uint8))
    # unpack: kept frames come back, deleted frames are not touched
    out = rng.integers(0, 256, size=nb * c * fb, dtype=np.uint8)
    rag = np.full(ch.sum_t * fb, 0x5A, np.uint8)
    O.chunk_unpack(ch, out, fb, 0, nb, rag)
    want_r = np.full((ch.sum_t, fb), 0x5A, np.uint8)
    want_r[frame[frame >= 0]] = out.reshape(nb, c, fb)[frame >= 0]
    assert np.array_equal(rag.reshape(-1, fb), want_r)
    assert int((rag.reshape(-1, fb) == 0x5A).all(axis=1).sum()) >= ch.frames_deleted - 1
    # the same chunks as an ordinary plan (chunk j = sequence j = block j): the general oracle functions agree
    p = ch.as_plan()
    if tail == O.KEEP_TAIL:      # only then do the chunks tile the store, which the general functions assume
        assert np.array_equal(O.pack(p, store, fb, 0, nb, 0xAB), dense)
        for a, b in zip(O.metadata(p, 0, nb), (sid, pos, reset, valid)):
            assert np.array_equal(a, b)
        rag2 = np.full(ch.sum_t * fb, 0x5A, np.uint8)
        O.unpack(p, out, fb, 0, nb, rag2)
        assert np.array_equal(rag2, rag)
    # partial ranges
    if ch.n_chunks > 3:
        assert np.array_equal(O.chunk_pack(ch, store, fb, 2, 2, 1), np.where((frame[2:4] >= 0)[:, :, None],
                              store.reshape(-1, fb)[np.maximum(frame[2:4], 0)], 1).astype(np.uint8))


def test_chunk_arguments():
    assert O.chunks(np.array([3, 0, 2], np.int32), 2).status != 0 and O.chunks(np.array([3, 0, 2], np.int32), 2).first_bad == 1
    assert O.chunks(np.array([3], np.int32), 0).status != 0
    assert O.chunks(np.array([3], np.int32), 2, tail=2).status != 0
    ch = O.chunks(np.array([1, 1, 1], np.int32), 5, O.DROP_TAIL)       # everything deleted
    assert ch.status == 0 and ch.n_chunks == 0 and ch.frames_deleted == 3
