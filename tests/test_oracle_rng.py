"""Pins for the oracle's random numbers and integer helpers (no GPU)."""
import numpy as np
from numpy.random import Philox

from oracle import bload_oracle as O

MASK = (1 << 64) - 1


def _numpy_philox(ctr, key):
    # numpy advances the counter by one before it produces a block of four words
    c = (int(ctr[0]) - 1) & MASK
    assert ctr[0] != 0
    bg = Philox(counter=np.array([c, ctr[1], ctr[2], ctr[3]], dtype=np.uint64), key=np.array(key, dtype=np.uint64))
    return bg.random_raw(4)


def test_philox_matches_numpy_bit_generator():
    rng = np.random.default_rng(5)
    for _ in range(200):
        ctr = [int(x) for x in rng.integers(1, 1 << 63, size=4, dtype=np.uint64)]
        key = [int(x) for x in rng.integers(0, 1 << 63, size=2, dtype=np.uint64)]
        assert np.array_equal(O.philox4x64_10(ctr, key), _numpy_philox(ctr, key))
    # the two streams the planner uses
    for seed in (0, 1, 2**63 + 5, MASK):
        for i in (1, 2, 77, 10**6, 2**31 - 2):
            assert O.seq_key(seed, i) == int(_numpy_philox([i, 0, 0, 0], [seed, 1])[0]) >> 32
            assert O.draw_word(seed, i) == int(_numpy_philox([i, 0, 0, 0], [seed, 2])[0])


def test_philox_counter_zero_is_consistent_with_numpy_wraparound():
    # counter 0 is reached by numpy from the all-ones counter (carry into the next word)
    bg = Philox(counter=np.array([MASK, MASK, MASK, MASK], dtype=np.uint64), key=np.array([9, 1], dtype=np.uint64))
    assert np.array_equal(O.philox4x64_10([0, 0, 0, 0], [9, 1]), bg.random_raw(4))


def test_pick_is_floor_of_u_times_m_over_2_64():
    rng = np.random.default_rng(6)
    for _ in range(2000):
        u = int(rng.integers(0, 1 << 63, dtype=np.uint64)) * 2 + int(rng.integers(0, 2))
        m = int(rng.integers(1, 1 << 31))
        j = O.pick(u, m)
        assert j == (u * m) >> 64 and 0 <= j < m
    assert O.pick(MASK, 7) == 6 and O.pick(0, 7) == 0 and O.pick(1 << 63, 2) == 1


def test_pick_is_uniform():
    # 60000 draw words of one stream mapped onto 6 bins: fixed seeds, so the statistic is a constant
    from scipy.stats import chi2
    counts = np.zeros(6)
    for k in range(60000):
        counts[O.pick(O.draw_word(12345, k), 6)] += 1
    stat = float(((counts - 10000.0) ** 2 / 10000.0).sum())
    assert stat < chi2.ppf(0.9999, 5)


def test_offsets_are_exclusive_prefix_sums():
    rng = np.random.default_rng(7)
    for n in (1, 2, 31, 1000, 70001):
        T = rng.integers(1, 5000, size=n).astype(np.int32)
        off = O.offsets(T)
        assert off.dtype == np.int64 and off[0] == 0
        assert np.array_equal(off[1:], np.cumsum(T, dtype=np.int64))
    # sums beyond 32 bits
    T = np.full(3_000_000, 2_000, np.int32)
    assert O.offsets(T)[-1] == 6_000_000_000
