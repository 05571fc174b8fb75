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
