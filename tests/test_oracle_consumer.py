"""Pins for the oracle's consumer-side functions (carry_prev, reset_state, valid_sum); no GPU.

Each pin reaches the same result by a route that does not go through the function under test: the
operation is carried out per sequence in the ragged store with numpy, and the already pinned
pack / unpack move the result between the two layouts.
"""
import numpy as np
import pytest

from oracle import bload_oracle as O

CASES = [(8, 6, 1), (40, 17, 3), (200, 64, 16), (150, 50, 5), (64, 64, 12)]


def _plan(n, tb, seed):
    rng = np.random.default_rng(seed)
    T = rng.integers(1, tb + 1, size=n).astype(np.int32)
    return O.plan(T, tb, seed), rng


@pytest.mark.parametrize("n,tb,fb", CASES)
def test_carry_prev_equals_shifting_each_sequence_in_the_ragged_store(n, tb, fb):
    p, rng = _plan(n, tb, 100 + n)
    store = rng.integers(0, 256, size=(p.sum_t, fb), dtype=np.uint8)
    fill = 0xA5
    shifted = np.empty_like(store)
    for i in range(p.n):
        a, b = int(p.offsets[i]), int(p.offsets[i + 1])
        shifted[a] = fill
        shifted[a + 1:b] = store[a:b - 1]
    nb = p.n_blocks + 2  # two filler blocks
    want = O.pack(p, shifted, fb, 0, nb, pad_byte=fill)
    dense = O.pack(p, store, fb, 0, nb, pad_byte=0x11)
    got = O.carry_prev(p, dense, fb, 0, nb, fill)
    assert np.array_equal(got, want)
    # a sub-range of blocks gives the same rows
    if p.n_blocks >= 3:
        sub = O.carry_prev(p, dense[1:3], fb, 1, 2, fill)
        assert np.array_equal(sub, want[1:3])


def test_carry_prev_never_crosses_a_sequence_boundary():
    # frames carry their sequence id: whatever a slot receives must come from its own sequence
    p, _ = _plan(300, 40, 7)
    ids = np.repeat(np.arange(p.n, dtype=np.int32), p.lengths)
    dense = O.pack(p, ids.view(np.uint8).reshape(p.sum_t, 4), 4, 0, p.n_blocks, pad_byte=0xFF)
    prev = O.carry_prev(p, dense, 4, 0, p.n_blocks, 0xFF).reshape(-1, 4).view(np.int32).reshape(p.n_blocks, p.t_block)
    seq_id, pos, reset, valid = O.metadata(p, 0, p.n_blocks)
    cont = (valid == 1) & (reset == 0)
    assert np.array_equal(prev[cont], seq_id[cont])
    assert np.all(prev[~cont] == -1)
    assert int(cont.sum()) == p.sum_t - p.n


@pytest.mark.parametrize("n,tb,fb", CASES)
def test_reset_state_turns_a_running_sum_into_per_sequence_cumsums(n, tb, fb):
    p, rng = _plan(n, tb, 200 + n)
    x = rng.integers(0, 1000, size=(p.sum_t, 2)).astype(np.int64)
    nb = p.n_blocks + 1
    dense = O.pack(p, x.view(np.uint8).reshape(p.sum_t, 16), 16, 0, nb).reshape(nb, tb, 16).view(np.int64)
    init = np.array([5, -7], np.int64)
    state = rng.integers(-99, 99, size=(nb, 2)).astype(np.int64)  # garbage carried in from a previous batch
    out = np.zeros((nb, tb, 2), np.int64)
    for s in range(tb):
        sb = state.view(np.uint8).reshape(nb, 16)
        O.reset_state(p, 0, nb, s, sb, init)
        state = sb.view(np.int64).reshape(nb, 2) + dense[:, s, :]
        out[:, s, :] = state
    got = np.zeros((p.sum_t, 16), np.uint8).reshape(-1)
    O.unpack(p, out.view(np.uint8), 16, 0, nb, got)
    got = got.view(np.int64).reshape(p.sum_t, 2)
    want = np.empty_like(x)
    for i in range(p.n):
        a, b = int(p.offsets[i]), int(p.offsets[i + 1])
        want[a:b] = init + np.cumsum(x[a:b], axis=0)
    assert np.array_equal(got, want)
    # the filler block's state is the initial state at every slot
    assert np.array_equal(out[nb - 1] - dense[nb - 1], np.broadcast_to(init, (tb, 2)))


def test_reset_state_defaults_to_zeros_and_leaves_continuing_rows_alone():
    p, rng = _plan(50, 20, 9)
    nb = p.n_blocks
    _, _, reset, valid = O.metadata(p, 0, nb)
    for s in (0, 1, 7, 19):
        state = rng.integers(1, 256, size=(nb, 24), dtype=np.uint8)
        before = state.copy()
        O.reset_state(p, 0, nb, s, state)
        cont = (valid[:, s] == 1) & (reset[:, s] == 0)
        assert np.array_equal(state[cont], before[cont])
        assert np.all(state[~cont] == 0)
    assert not np.any((valid[:, 0] == 1) & (reset[:, 0] == 0))  # slot 0 always starts a sequence


@pytest.mark.parametrize("n,tb,fb", CASES)
def test_valid_sum_equals_the_sum_over_the_ragged_values(n, tb, fb):
    p, rng = _plan(n, tb, 300 + n)
    v = rng.integers(-2 ** 20, 2 ** 20, size=p.sum_t).astype(np.float32)  # integers: every partial sum is exact
    nb = p.n_blocks + 1
    dense = O.pack(p, v.view(np.uint8).reshape(p.sum_t, 4), 4, 0, nb, pad_byte=0x7F)  # padding decodes to a huge float
    s, c = O.valid_sum(p, 0, nb, dense.reshape(-1).view(np.float32))
    assert c == p.sum_t
    assert s == float(v.astype(np.float64).sum())
    # sub-ranges add up
    if p.n_blocks >= 2:
        s1, c1 = O.valid_sum(p, 0, 1, dense[:1].reshape(-1).view(np.float32))
        s2, c2 = O.valid_sum(p, 1, nb - 1, dense[1:].reshape(-1).view(np.float32))
        assert c1 + c2 == c and s1 + s2 == s
