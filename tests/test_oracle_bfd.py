"""Pins for the oracle's best-fit-decreasing strategy (policy 2; a textbook bin-packing heuristic used as a
deterministic low-padding comparison, not the paper's random rule)."""
import bisect

import numpy as np
import pytest

import brute
import invariants
from oracle import bload_oracle as O
from paper_2310_10879_b200 import workloads as W


def _check(p):
    assert p.status == 0
    invariants.check_plan(p.lengths, p.t_block, p.n_blocks, p.offsets, p.seg_seq, p.seg_block, p.seg_start,
                          p.block_seg_begin, p.block_fill, p.seq_block, p.seq_start, maximal=False)


def textbook_bfd_fills(lengths, t_block):
    """Best fit decreasing with a sorted list of free rooms (bisect): the multiset of final fills does not depend
    on which of several equally full blocks is taken."""
    rooms = []                                   # sorted free room of every open block
    for l in sorted((int(x) for x in lengths), reverse=True):
        i = bisect.bisect_left(rooms, l)
        if i == len(rooms):
            new = t_block - l
        else:
            new = rooms.pop(i) - l
        bisect.insort(rooms, new)
    return sorted(t_block - r for r in rooms)


def replay_best_fit(p):
    """Walk the placements in the order the strategy made them (decreasing length, ties in reverse L_dict order) and
    check at every step: the chosen block had the smallest room that fits; a new block was opened only when no
    open block had room; among equally full candidates the one that reached that room first was taken."""
    T = p.lengths
    order = sorted(range(p.n), key=lambda i: (int(T[i]), O.seq_key(p.seed, i), i), reverse=True)
    room, since, clock = {}, {}, 0                # per open block: free room, time it got that room
    for s in order:
        l, b, st = int(T[s]), int(p.seq_block[s]), int(p.seq_start[s])
        fits = [(r, since[q], q) for q, r in room.items() if r >= l]
        if b not in room:
            assert not fits, "opened a block although one had room"
            assert b == len(room) and st == 0      # blocks are numbered in opening order
            room[b] = p.t_block
        else:
            assert st == p.t_block - room[b]
            assert (room[b], since[b], b) == min(fits), "not the best fit / not the oldest of the best"
        room[b] -= l
        clock += 1
        since[b] = clock
    assert sorted(p.t_block - r for r in room.values()) == sorted(int(x) for x in p.block_fill)


@pytest.mark.parametrize("seed", [0, 5])
def test_bfd_small_cases_step_by_step(seed):
    rng = np.random.default_rng(40 + seed)
    for _ in range(60):
        n = int(rng.integers(1, 40)); tb = int(rng.integers(1, 30))
        T = rng.integers(1, tb + 1, size=n).astype(np.int32)
        p = O.plan(T, tb, seed, policy=2)
        _check(p)
        replay_best_fit(p)
        assert sorted(int(x) for x in p.block_fill) == textbook_bfd_fills(T, tb)


def test_bfd_against_the_exhaustive_optimum():
    rng = np.random.default_rng(7)
    for _ in range(80):
        n = int(rng.integers(1, 9)); tb = int(rng.integers(2, 12))
        T = rng.integers(1, tb + 1, size=n).astype(np.int32)
        p = O.plan(T, tb, 1, policy=2)
        opt = brute.min_blocks([int(x) for x in T], tb)
        assert opt <= p.n_blocks <= (11 * opt + 6) // 9 + 1     # the classical 11/9 OPT + 6/9 guarantee
    # the toy dataset of the paper, stand-in lengths: 31 frames in blocks of 6 need 6 blocks, BFD finds them
    p = O.plan(W.TOY8_LENGTHS, W.TOY8_T_BLOCK, 0, policy=2)
    assert p.n_blocks == 6 and sorted(p.block_fill) == [2, 5, 6, 6, 6, 6]


@pytest.mark.parametrize("name", ["toy_video", "features_fp16", "raw_frames", "heavy_tail_bf16", "video_dataset_shape", "tokens"])
def test_bfd_on_workloads(name):
    w = W.WORKLOADS[name]
    T = W.lengths(w)
    p = O.plan(T, w.t_block, w.seed, policy=2)
    _check(p)
    assert sorted(int(x) for x in p.block_fill) == textbook_bfd_fills(T, w.t_block)
    assert -(-p.sum_t // w.t_block) <= p.n_blocks <= O.plan(T, w.t_block, w.seed, policy=0).n_blocks
    if name != "tokens":
        replay_best_fit(p)


def test_bfd_is_deterministic_up_to_ties():
    T = W.lengths(W.WORKLOADS["features_fp16"])
    a, b = O.plan(T, 1000, 1, policy=2), O.plan(T, 1000, 2, policy=2)
    assert a.n_blocks == b.n_blocks and np.array_equal(np.sort(a.block_fill), np.sort(b.block_fill))
    assert np.array_equal(a.lengths[a.seg_seq], b.lengths[b.seg_seq])      # same lengths in the same places
