"""Property tests of the oracle (hypothesis): any lengths, block length, seed and policy give a plan that
passes the independent validity checker, and pack/unpack round-trip for any frame size."""
import numpy as np
from hypothesis import given, settings, strategies as st

import invariants
from oracle import bload_oracle as O


@settings(max_examples=150, deadline=None)
@given(st.integers(1, 60), st.data(), st.integers(0, 2**64 - 1), st.integers(0, 1))
def test_any_plan_is_valid(t_block, data, seed, policy):
    T = np.array(data.draw(st.lists(st.integers(1, t_block), min_size=1, max_size=80)), np.int32)
    p = O.plan(T, t_block, seed, policy)
    assert p.status == 0
    invariants.check_plan(p.lengths, p.t_block, p.n_blocks, p.offsets, p.seg_seq, p.seg_block, p.seg_start,
                          p.block_seg_begin, p.block_fill, p.seq_block, p.seq_start)
    s = O.stats(p.n, p.sum_t, p.t_max, t_block, p.n_blocks)
    assert s["pad_packed"] == p.n_blocks * t_block - int(T.sum()) >= 0
    assert s["pad_naive_tmax"] == T.size * int(T.max()) - int(T.sum())


@settings(max_examples=60, deadline=None)
@given(st.integers(1, 30), st.data(), st.integers(0, 2**32), st.integers(1, 40), st.integers(0, 255))
def test_pack_unpack_round_trip(t_block, data, seed, fb, pad):
    T = np.array(data.draw(st.lists(st.integers(1, t_block), min_size=1, max_size=40)), np.int32)
    p = O.plan(T, t_block, seed)
    store = np.random.default_rng(seed).integers(0, 256, size=p.sum_t * fb, dtype=np.uint8)
    dense = O.pack(p, store, fb, 0, p.n_blocks + 1, pad)
    seq_id, pos, reset, valid = O.metadata(p, 0, p.n_blocks + 1)
    assert np.all(dense[valid == 0] == pad) and int(valid.sum()) == p.sum_t and int(reset.sum()) == p.n
    out = np.zeros_like(store)
    O.unpack(p, dense, fb, 0, p.n_blocks + 1, out)
    assert np.array_equal(out, store)


@settings(max_examples=60, deadline=None)
@given(st.integers(1, 30), st.data(), st.integers(0, 2**32), st.integers(1, 24), st.integers(0, 255))
def test_carry_prev_and_repeat_last_properties(t_block, data, seed, fb, fill):
    T = np.array(data.draw(st.lists(st.integers(1, t_block), min_size=1, max_size=40)), np.int32)
    p = O.plan(T, t_block, seed)
    nb = p.n_blocks + 1
    store = np.random.default_rng(seed).integers(0, 256, size=(p.sum_t, fb), dtype=np.uint8)
    dense = O.pack(p, store, fb, 0, nb, fill)
    seq_id, pos, reset, valid = O.metadata(p, 0, nb)
    # what a slot receives is the frame before it in the ragged store, or the fill byte at a sequence start / padding
    prev = O.carry_prev(p, dense, fb, 0, nb, fill)
    cont = (valid == 1) & (reset == 0)
    src = p.offsets[np.maximum(seq_id, 0)] + pos - 1
    assert np.array_equal(prev[cont], store[src[cont]]) and np.all(prev[~cont] == fill)
    # repeat-last padding changes nothing but the padding of blocks that hold a frame
    rep = O.pack_repeat_last(p, store, fb, 0, nb, fill)
    assert np.array_equal(rep[valid == 1], dense[valid == 1])
    for q in range(nb):
        k = int(valid[q].sum())
        want = dense[q, k - 1] if k else np.full(fb, fill, np.uint8)
        assert np.all(rep[q, k:] == want)


@settings(max_examples=60, deadline=None)
@given(st.integers(1, 20), st.data(), st.integers(0, 2**32), st.integers(0, 255))
def test_var_frames_round_trip_and_padding(t_block, data, seed, pad):
    n = data.draw(st.integers(1, 30))
    T = np.array(data.draw(st.lists(st.integers(1, t_block), min_size=n, max_size=n)), np.int32)
    F = np.array(data.draw(st.lists(st.integers(1, 20), min_size=n, max_size=n)), np.int32)
    slot = int(F.max()) + data.draw(st.integers(0, 5))
    p = O.plan(T, t_block, seed)
    boff = O.byte_offsets(T, F)
    store = np.random.default_rng(seed).integers(0, 256, size=int(boff[-1]), dtype=np.uint8)
    nb = p.n_blocks + 1
    dense = O.pack_var(p, store, F, slot, 0, nb, pad)
    seq_id, _, _, valid = O.metadata(p, 0, nb)
    used = np.where(valid == 1, F[np.maximum(seq_id, 0)], 0)               # bytes of every slot that hold a frame
    is_pad = np.arange(slot)[None, None, :] >= used[:, :, None]
    assert np.all(dense[is_pad] == pad) and int((~is_pad).sum()) == int(boff[-1])
    back = np.zeros_like(store)
    O.unpack_var(p, dense, F, slot, 0, nb, back)
    assert np.array_equal(back, store)


@settings(max_examples=120, deadline=None)
@given(st.integers(1, 40), st.data(), st.integers(0, 1), st.integers(1, 12), st.integers(0, 2**32))
def test_chunking_strategy_properties(t_chunk, data, tail, fb, seed):
    """Any lengths and chunk length: every kept frame sits in exactly one chunk at the slot its position says, chunks
    never cross a sequence, the two tails differ exactly by the short last chunks, and pack followed by unpack returns
    the kept frames and leaves the deleted ones alone."""
    T = np.array(data.draw(st.lists(st.integers(1, 3 * t_chunk + 2), min_size=1, max_size=40)), np.int32)
    ch = O.chunks(T, t_chunk, tail)
    assert ch.status == 0
    T64 = T.astype(np.int64)
    assert ch.frames_kept + ch.frames_deleted == int(T64.sum()) and ch.n_chunks * t_chunk == ch.frames_kept + ch.pad_frames
    assert bool((ch.chunk_len >= 1).all()) and bool((ch.chunk_len <= t_chunk).all()) if ch.n_chunks else True
    assert bool((ch.chunk_first % t_chunk == 0).all()) and bool((ch.chunk_first + ch.chunk_len <= T[ch.chunk_seq]).all())
    if tail == O.DROP_TAIL:
        assert ch.pad_frames == 0 and ch.frames_deleted == int((T64 % t_chunk).sum())
    else:
        assert ch.frames_deleted == 0 and ch.pad_frames == int(((-T64) % t_chunk).sum())
    store = np.random.default_rng(seed).integers(0, 256, size=ch.sum_t * fb, dtype=np.uint8)
    dense = O.chunk_pack(ch, store, fb, 0, ch.n_chunks + 1, 0xEE)
    sid, pos, reset, valid = O.chunk_metadata(ch, 0, ch.n_chunks + 1)
    assert int(valid.sum()) == ch.frames_kept and int(reset.sum()) == ch.n_chunks
    assert np.all(dense[valid == 0] == 0xEE)
    back = np.full(ch.sum_t * fb, 0x5A, np.uint8)
    O.chunk_unpack(ch, dense, fb, 0, ch.n_chunks + 1, back)
    kept = np.zeros(ch.sum_t, bool)
    for j in range(ch.n_chunks):
        a = int(ch.offsets[ch.chunk_seq[j]]) + int(ch.chunk_first[j])
        assert not kept[a:a + ch.chunk_len[j]].any()
        kept[a:a + ch.chunk_len[j]] = True
    assert int(kept.sum()) == ch.frames_kept
    b2, s2 = back.reshape(-1, fb), store.reshape(-1, fb)
    assert np.array_equal(b2[kept], s2[kept]) and bool((b2[~kept] == 0x5A).all())
